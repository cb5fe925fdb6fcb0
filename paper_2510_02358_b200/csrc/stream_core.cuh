// Streaming pass for rows whose start, strides and length are multiples of 16 bytes, and the
// selection of the exact top-K from what it leaves behind.
//
// Pass 1 (stream_slice, one CTA per row slice): the slice streams through a ring of
// shared-memory stages by bulk asynchronous copies (cp.async.bulk, completion counted on an
// mbarrier per stage, no multicast) that one thread issues ahead; all kThreads threads read each
// stage with one 128-bit shared load per vector and do the arithmetic from registers.  The loop
// has no block-wide barrier.  It leaves in global memory, per row: a table with, for every tile
// and thread, the largest logit of the thread's kVpt vectors of that tile, and per slice and
// warp the log-sum-exp terms.
//
// Pass 2 (one CTA per row, run by the kernels in lattice.cu / verify.cu): merge_warp_partials
// adds up the sums, select_from_table picks the exact top-K: a threshold with at least K
// logits at or above it, the exact K-th largest table entry among those that reach it, and a
// second look (L2 hits) at the few (tile, thread) shares whose maximum reaches that value.
// Results are the same as scan_slice's (scan_core.cuh).
#pragma once

#include "scan_core.cuh"

namespace dsp {

constexpr int kTileBytes = kThreads * kVpt * 16;     // one ring stage = one tile of either dtype
constexpr int kStages = 3;
constexpr int kRingBytes = kStages * kTileBytes;     // dynamic shared memory of a streaming kernel
constexpr long long kWaitCycles = 400000000LL;       // every wait gives up after this many SM clocks (~0.2 s)

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Bounded wait for the phase with the given parity: gives up after kWaitCycles, or at once when
// another wait of this CTA has already given up (`abort` non-zero).  False if it gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort) {
    const uint32_t a = smem_addr(bar);
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}"
            : "=r"(ok)
            : "r"(a), "r"(parity)
            : "memory");
        if (ok) return true;
        if (*abort || clock64() - t0 > kWaitCycles) return false;
    }
}
// Bulk copy global -> this CTA's shared memory; both addresses and the size are multiples of 16.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Two fp32 operations in one instruction on a register pair (Blackwell's packed fp32 pipe).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Static shared state of a streaming kernel.
struct StreamBars {
    uint64_t full[kStages];      // stage filled by its bulk copy
    uint64_t empty[kStages];     // stage released by all warps
    int timed_out;               // non-zero once a bounded wait gave up
};

// Called by every thread before the scan starts (ends with a CTA-wide barrier).
__device__ __forceinline__ void stream_begin(StreamBars &bars) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars.full[s], 1);
            mbar_init(&bars.empty[s], kWarps);
        }
        mbar_init_fence();
        bars.timed_out = 0;
    }
    __syncthreads();
}

// Issue the bulk copy of tile t of the slice at `src` into its ring stage (one thread).
__device__ __forceinline__ void issue_tile(const char *src, int nbytes, int t, unsigned char *ring,
                                           StreamBars &bars) {
    const int s = t % kStages;
    const uint32_t bytes = (uint32_t)min(kTileBytes, nbytes - t * kTileBytes);
    mbar_expect_tx(&bars.full[s], bytes);
    bulk_load(ring + (size_t)s * kTileBytes, src + (size_t)t * kTileBytes, bytes, &bars.full[s]);
}

// Padding for the vectors past the end of a ragged last tile: -2^124, below every finite
// logit the interface allows, finite when scaled by log2(e), never a candidate (its index is
// past the row).
template <typename DT> struct Pad;
template <> struct Pad<__nv_bfloat16> { static constexpr uint32_t kWord = 0xFD80FD80u; };
template <> struct Pad<float> { static constexpr uint32_t kWord = 0xFD800000u; };

// Entry of the table of per-thread tile maxima, stored in the row's own element type (exact).
__device__ __forceinline__ void table_store(__nv_bfloat16 *tab, int i, float v) {
    reinterpret_cast<unsigned short *>(tab)[i] = (unsigned short)(__float_as_uint(v) >> 16);
}
__device__ __forceinline__ void table_store(float *tab, int i, float v) { tab[i] = v; }

// First threshold from one value per thread (its largest logit): with r = ceil(K / #warps), the
// smallest over the warps of each warp's r-th largest value has K distinct logits at or above
// it.  One barrier; every thread derives the value itself.  If some warp has fewer than r finite
// values (masked rows) the general rule of bootstrap_threshold applies (two more barriers).
template <typename SY>
__device__ __forceinline__ float bootstrap_threshold_fast(ScanSmem &sm, float tm, int K) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float s = bitonic_desc(tm == tm ? tm : -CUDART_INF_F, lane);
    sm.wsorted[warp][lane] = s;
    SY::sync();
    const int r = (K + kWarps - 1) / kWarps;
    float t = CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t = fminf(t, sm.wsorted[w][r - 1]);
    if (t > -CUDART_INF_F) return t;
    SY::sync();
    if (tid == 0) {
        float g = -CUDART_INF_F;
        for (int rr = 1; rr <= 32; ++rr) {
            int nw = 0;
            float lo = CUDART_INF_F;
            for (int w = 0; w < kWarps; ++w) {
                const float x = sm.wsorted[w][rr - 1];
                if (x > -CUDART_INF_F) { ++nw; lo = fminf(lo, x); }
            }
            if (nw == 0) break;
            if (rr * nw >= K) { g = lo; break; }
        }
        sm.thr_v = g;
    }
    SY::sync();
    return sm.thr_v;
}

// Exact top-K of [s0, s1) of `row` from its table of per-thread tile maxima (`tab`, ntiles x
// kThreads, entry [t][thread], in global memory).  On return sm.cand[0 .. sm.cnt) holds the best
// min(K, #finite) keys, sorted (after a barrier).  Rows with very many equal top values overflow
// the lists and take topk_careful instead.  Block-wide; sm.cnt and sm.flag must be 0 on entry
// (before a barrier).
template <typename DT, typename SY>
__device__ void select_from_table(const DT *__restrict__ row, int s0, int s1, int K, int ntiles,
                                  const DT *tab, ScanSmem &sm) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    constexpr int kHalf = kCandCap / 2;              // element keys first, table entries in the upper half
    const int tid = threadIdx.x;
    // 1. a threshold with at least K table entries at or above it, from each thread's largest
    float rm = -CUDART_INF_F;
    for (int t = 0; t < ntiles; ++t) rm = fmaxf(rm, Elem<DT>::load1(tab + t * kThreads + tid));
    const float t0 = bootstrap_threshold_fast<SY>(sm, rm, K);
    // 2. the table entries that reach it (each thread looks at its own column)
    for (int t = 0; t < ntiles; ++t) {
        const float v = Elem<DT>::load1(tab + t * kThreads + tid);
        if (v >= t0 && v > -CUDART_INF_F) {
            const int pos = atomicAdd(&sm.cnt, 1);
            if (pos < kHalf) sm.cand[kHalf + pos] = make_key(v, t * kThreads + tid);
        }
    }
    SY::sync();
    const int n = sm.cnt;
    if (n > kHalf) {                                 // block-uniform
        topk_careful<DT, SY>(row, s0, s1, K, sm);
        return;
    }
    // 3. the K-th largest of them (all of them if there are fewer than K), by counting
    const int kk = min(K, n);
    const unsigned long long *entries = sm.cand + kHalf;
    for (int i = tid; i < n; i += kThreads) {
        const unsigned long long key = entries[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += entries[j] > key;
        if (rank == kk - 1) sm.thrkey = key;
    }
    SY::sync();
    // 4. the shares whose maximum reaches that value hold every logit of the slice's top K:
    //    look at their logits again and list those that reach it
    if (n > 0) {
        // with fewer than K entries (the threshold was -inf: every finite entry is listed) every
        // finite logit of the listed shares is wanted
        const float tk = n >= K ? key_value(sm.thrkey) : -CUDART_INF_F;
        for (int i = tid; i < n; i += kThreads) {
            const unsigned long long key = entries[i];
            if (key_value(key) >= tk) {
                const int id = key_id(key);
                const int e00 = s0 + (id / kThreads) * TE + (id % kThreads) * N;
#pragma unroll
                for (int j = 0; j < kVpt; ++j) {
                    const int e0 = e00 + j * kThreads * N;
                    if (e0 < s1) {                   // vectors are whole: the row length is a multiple of N
                        const uint4 v = ldg_stream(row + e0);
#pragma unroll
                        for (int e = 0; e < N; ++e) {
                            const float x = Elem<DT>::get(v, e);
                            if (x >= tk && x > -CUDART_INF_F) {
                                const int pos = atomicAdd(&sm.flag, 1);
                                if (pos < kHalf) sm.cand[pos] = make_key(x, e0 + e);
                            }
                        }
                    }
                }
            }
        }
    }
    SY::sync();
    const int n2 = sm.flag;
    if (n2 > kHalf) {                                // block-uniform
        topk_careful<DT, SY>(row, s0, s1, K, sm);
        return;
    }
    // 5. the best K of the listed logits, sorted, to the front
    if (tid == 0) sm.cnt = n2;
    prune<SY>(sm, K);
}

// Log-sum-exp terms of one warp of one slice, as pass 1 leaves them.
struct WarpPartial {
    double S, T;
    float c;
    int pad;
};

// Pass 1 over [s0, s1) of `row` (all kThreads threads of the CTA).  Writes the slice's part of
// the row's table of per-thread tile maxima (`tab` points at the slice's first tile: entry
// [t][thread]) and, with `sums` (block-uniform), this warp's sums relative to its own reference
// exponent into wpart[warp] (c = kRefFloor, S = 0 if the warp saw no finite logit).
template <typename DT>
__device__ void stream_slice(const DT *__restrict__ row, int s0, int s1, bool sums, StreamBars &bars,
                             unsigned char *ring, DT *__restrict__ tab, WarpPartial *wpart) {
    constexpr int N = Elem<DT>::N;
    constexpr int VT = kTileBytes / 16;
    static_assert(VT == kThreads * kVpt && tile_elems<DT>() * (int)sizeof(DT) == kTileBytes, "tile geometry");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nbytes = (s1 - s0) * (int)sizeof(DT);
    const int ntiles = (nbytes + kTileBytes - 1) / kTileBytes;
    volatile int *abort = &bars.timed_out;

    float c = kRefFloor, S = 0.f, T = 0.f;

    // Thread 0 also issues the copies, kStages - 1 tiles ahead of the tile being scanned.
    const char *src = reinterpret_cast<const char *>(row + s0);
    if (tid == 0) {
        for (int tt = 0; tt < min(kStages, ntiles); ++tt) issue_tile(src, nbytes, tt, ring, bars);
    }
    for (int t = 0; t < ntiles; ++t) {
        if (tid == 0 && t >= 1 && t + kStages - 1 < ntiles) {
            const int tt = t + kStages - 1;           // its stage held tile t - 1
            if (!mbar_wait(&bars.empty[tt % kStages], ((tt / kStages) - 1) & 1, abort)) bars.timed_out = 1;
            issue_tile(src, nbytes, tt, ring, bars);
        }
        const int s = t % kStages;
        if (!mbar_wait(&bars.full[s], (t / kStages) & 1, abort)) bars.timed_out = 1;
        const int nvec = min(kTileBytes, nbytes - t * kTileBytes) >> 4;
        const uint4 *sp = reinterpret_cast<const uint4 *>(ring + (size_t)s * kTileBytes);
        uint4 v[kVpt];
        if (nvec == VT) {
#pragma unroll
            for (int j = 0; j < kVpt; ++j) v[j] = sp[j * kThreads + tid];
        } else {
            const uint32_t pw = Pad<DT>::kWord;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                const int vi = j * kThreads + tid;
                v[j] = vi < nvec ? sp[vi] : make_uint4(pw, pw, pw, pw);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.empty[s]);   // the stage is in registers: release it

        float x[kVpt][N];
        float vm[kVpt];
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
#pragma unroll
            for (int e = 0; e < N; ++e) x[j][e] = Elem<DT>::get(v[j], e);
            if constexpr (N == 8) {
                vm[j] = max3(max3(x[j][0], x[j][1], x[j][2]), max3(x[j][3], x[j][4], x[j][5]),
                             fmaxf(x[j][6], x[j][7]));
            } else {
                vm[j] = fmaxf(max3(x[j][0], x[j][1], x[j][2]), x[j][3]);
            }
        }
        const float tm = fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3]));
        table_store(tab, t * kThreads + tid, tm);

        if (sums) {
            const float ts = tm * kLog2e;             // the reference exponent bounds every logit seen
            if (ts > c) {
                const float d = c - ts;
                const float sc = ex2_approx(d);
                T = (T + S * d) * sc;
                S = S * sc;
                c = ts;
            }
            // two logits per instruction: a = x * log2(e) - c, S += 2^a, T += 2^a * a
            const unsigned long long nc2 = pack2(-c, -c), l2e2 = pack2(kLog2e, kLog2e);
            unsigned long long S2 = pack2(S, 0.f), T2 = pack2(T, 0.f);
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < N; e += 2) {
                    const unsigned long long a2 = fma2(pack2(x[j][e], x[j][e + 1]), l2e2, nc2);
                    float a0, a1;
                    unpack2(a2, a0, a1);
                    const unsigned long long e2 = pack2(ex2_approx(a0), ex2_approx(a1));
                    S2 = add2(S2, e2);
                    T2 = fma2(e2, a2, T2);
                }
            }
            float s0f, s1f, t0f, t1f;
            unpack2(S2, s0f, s1f);
            unpack2(T2, t0f, t1f);
            S = s0f + s1f;
            T = t0f + t1f;
        }
    }
    if (sums) {
        // this warp's sums against one reference exponent, in double (shuffles only)
        const float cw = warp_max(c);
        const float d = c - cw;
        const float a = ex2_approx(d);
        const double Sd = warp_sum((double)(S * a));
        const double Td = warp_sum((double)((T + S * d) * a));
        if (lane == 0) {
            WarpPartial p;
            p.S = Sd; p.T = Td; p.c = cw; p.pad = 0;
            wpart[warp] = p;
        }
    }
}

// Pass 2: the n = nslices * kWarps warp partials of a row into one (c, S, T), in double and in
// a fixed order.  Partials without finite logits are skipped.  Block-wide (n <= kThreads).
template <typename SY>
__device__ void merge_warp_partials(const WarpPartial *p, int n, ScanSmem &sm, float &c_out, double &S_out,
                                    double &T_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float c = kRefFloor;
    double S = 0.0, T = 0.0;
    if (tid < n) {
        S = __ldcg(&p[tid].S); T = __ldcg(&p[tid].T); c = __ldcg(&p[tid].c);
    }
    const bool live = S > 0.0 || !(S == S);          // NaN sums must stay visible
    float cm = warp_max(live ? c : kRefFloor);
    if (lane == 0) sm.redc[warp] = cm;
    SY::sync();
    cm = sm.redc[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) cm = fmaxf(cm, sm.redc[w]);
    double Sm = 0.0, Tm = 0.0;
    if (S != 0.0) {
        const double d = (double)c - (double)cm;
        const double a = exp2(d);
        Sm = a * S;
        Tm = a * (T + S * d);
    }
    Sm = warp_sum(Sm);
    Tm = warp_sum(Tm);
    if (lane == 0) { sm.redS[warp] = Sm; sm.redT[warp] = Tm; }
    SY::sync();
    Sm = 0.0; Tm = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { Sm += sm.redS[w]; Tm += sm.redT[w]; }
    SY::sync();
    c_out = cm; S_out = Sm; T_out = Tm;
}

// The streaming kernels need more dynamic shared memory than the default limit: raise the limit
// of `kernel` once per device (the attribute is per device).  `rec` is the caller's per-kernel
// record.
struct RingSmemDone {
    bool dev[64] = {};
};
template <typename KernelT>
inline cudaError_t allow_ring_smem(KernelT *kernel, RingSmemDone &rec) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && rec.dev[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) rec.dev[dev] = true;
    return e;
}

// True if rows of this layout can be streamed with bulk copies.
template <typename DT>
inline bool stream_layout_ok(const void *base, int V, long long stride_b, long long stride_l) {
    const size_t es = sizeof(DT);
    return (reinterpret_cast<uintptr_t>(base) & 15) == 0 && ((size_t)V * es) % 16 == 0 &&
           ((size_t)stride_b * es) % 16 == 0 && ((size_t)stride_l * es) % 16 == 0;
}

}  // namespace dsp
