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
// Pass 2 (one warp per row, row_warp.cuh, run by the kernels in lattice.cu / verify.cu) adds up
// the sums and picks the exact top-K from the table.  Results are the same as scan_slice's
// (scan_core.cuh).
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
__device__ __forceinline__ bool mbar_try(uint32_t bar_addr, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity)
        : "memory");
    return ok != 0u;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort) {
    const uint32_t a = smem_addr(bar);
    if (mbar_try(a, parity)) return true;              // the usual case: no clock is read
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try(a, parity)) return true;
        if (*abort || clock64() - t0 > kWaitCycles) return false;
    }
}
// Bulk copy global -> this CTA's shared memory; both addresses and the size are multiples of 16.
// The logits are read once: their L2 lines are marked "evict first", so that streaming them does
// not push out what pass 1 writes for pass 2 (the table of tile maxima and the sums).
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
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
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
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

// The tiles of a row dealt to its slices as evenly as whole tiles allow: slice s of n covers the
// tiles [s * T / n, (s + 1) * T / n) of the row's T tiles (n <= T, so no slice is empty).
template <typename DT>
__device__ __forceinline__ void slice_range(int slice, int nslices, int ntiles_row, int V, int &s0, int &s1) {
    constexpr int TE = tile_elems<DT>();
    s0 = (int)((long long)slice * ntiles_row / nslices) * TE;
    s1 = min(V, (int)((long long)(slice + 1) * ntiles_row / nslices) * TE);
}

// Issue the bulk copy of tile t of the slice at `src` into its ring stage s = t % kStages (one thread).
__device__ __forceinline__ void issue_tile(const char *src, int nbytes, int t, int s, unsigned char *ring,
                                           StreamBars &bars) {
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

// Log-sum-exp terms of one warp of one slice, as pass 1 leaves them.
struct WarpPartial {
    double S, T;
    float c;
    int pad;
};

// Pass 1 over [s0, s1) of `row` (all kThreads threads of the CTA).  Writes the slice's part of
// the row's table of per-thread tile maxima (`tab` points at the slice's first tile: entry
// [t][thread]), every thread's largest logit of the whole slice (smax[thread]) and, with `sums`
// (block-uniform), this warp's sums relative to its own reference exponent into wpart[warp]
// (c = kRefFloor, S = 0 if the warp saw no finite logit).
template <typename DT>
__device__ void stream_slice(const DT *__restrict__ row, int s0, int s1, bool sums, StreamBars &bars,
                             unsigned char *ring, DT *__restrict__ tab, DT *__restrict__ smax, WarpPartial *wpart) {
    constexpr int N = Elem<DT>::N;
    constexpr int VT = kTileBytes / 16;
    static_assert(VT == kThreads * kVpt && tile_elems<DT>() * (int)sizeof(DT) == kTileBytes, "tile geometry");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nbytes = (s1 - s0) * (int)sizeof(DT);
    const int ntiles = (nbytes + kTileBytes - 1) / kTileBytes;
    volatile int *abort = &bars.timed_out;

    float c = kRefFloor, S = 0.f, T = 0.f;
    float rm = -CUDART_INF_F;                        // this thread's largest logit so far

    // Thread 0 also issues the copies, kStages - 1 tiles ahead of the tile being scanned.
    const char *src = reinterpret_cast<const char *>(row + s0);
    if (tid == 0) {
        for (int tt = 0; tt < min(kStages, ntiles); ++tt) issue_tile(src, nbytes, tt, tt, ring, bars);
    }
    int s = 0;                                       // stage of tile t: t % kStages
    uint32_t ph = 0u;                                // phase parity of tile t in its stage: (t / kStages) & 1
    DT *tp = tab + tid;                              // this thread's table entry of tile t
    // the sums of this thread's even and odd logits (register pairs), against the reference exponent c
    unsigned long long S2 = pack2(0.f, 0.f), T2 = pack2(0.f, 0.f);
    for (int t = 0; t < ntiles; ++t, tp += kThreads) {
        if (tid == 0 && t >= 1 && t + kStages - 1 < ntiles) {
            // tile t + kStages - 1 goes to the stage that held tile t - 1, once every warp has released it
            const int es = s == 0 ? kStages - 1 : s - 1;
            if (!mbar_wait(&bars.empty[es], s == 0 ? ph ^ 1u : ph, abort)) bars.timed_out = 1;
            issue_tile(src, nbytes, t + kStages - 1, es, ring, bars);
        }
        if (!mbar_wait(&bars.full[s], ph, abort)) bars.timed_out = 1;
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
        const float tm = fmaxf(fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3])), fmaxf(vm[4], vm[5]));
        table_store(tp, 0, tm);
        rm = fmaxf(rm, tm);

        if (sums) {
            const float ts = tm * kLog2e;             // the reference exponent bounds every logit seen
            if (ts > c) {                              // both halves move to the new reference exponent
                const float d = c - ts;
                const float sc = ex2_approx(d);
                const unsigned long long sc2 = pack2(sc, sc);
                T2 = mul2(fma2(S2, pack2(d, d), T2), sc2);
                S2 = mul2(S2, sc2);
                c = ts;
            }
            // two logits per instruction: a = x * log2(e) - c, S += 2^a, T += 2^a * a
            const unsigned long long nc2 = pack2(-c, -c), l2e2 = pack2(kLog2e, kLog2e);
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
        }
        if (++s == kStages) { s = 0; ph ^= 1u; }
    }
    {
        float s0f, s1f, t0f, t1f;
        unpack2(S2, s0f, s1f);
        unpack2(T2, t0f, t1f);
        S = s0f + s1f;
        T = t0f + t1f;
    }
    table_store(smax, tid, rm);
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
