// Streaming pass over row slices whose start, strides and length are multiples of 16 bytes.
//
// stream_slice (one CTA per row slice): the slice streams through a ring of shared-memory stages
// by bulk asynchronous copies (cp.async.bulk, completion counted on an mbarrier per stage, no
// multicast) that one thread issues ahead; all kThreads threads read each stage with one 128-bit
// shared load per vector and do the arithmetic from registers.  The loop has no block-wide
// barrier and stores nothing to global memory.  Every thread owns one "column" of the slice (its
// kVpt vectors of every tile) and keeps of it: the largest logit, the tile that holds it, the
// largest logit of all its other tiles, and (with SUMS) the log-sum-exp terms against its own
// reference exponent.  The exact top-K of the row is selected from these records afterwards
// (row_engine.cuh): only columns whose largest logit reaches a threshold can hold a top-K logit,
// and of such a column only the one recorded tile, unless its second value reaches it too.
#pragma once

#include "scan_core.cuh"

namespace dsp {

constexpr int kTileBytes = kThreads * kVpt * 16;     // one ring stage = one tile of either dtype
constexpr int kMinStages = 3;                        // ring depth when the grid fills every SM several times over
constexpr int kMaxStages = 9;                        // ring depth of a CTA that has its SM to itself
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
// not push out what the kernels of a step hand to one another (measured: faster than no hint).
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
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
struct WarpPartial {             // log-sum-exp terms of one warp of one slice
    double S, T;
    float c;
    int pad;
};
struct StreamBars {
    uint64_t full[kMaxStages];   // stage filled by its bulk copy
    uint64_t empty[kMaxStages];  // stage released by all warps
    WarpPartial wp[kWarps];      // the slice's sums, one entry per warp, written when the warp is through
    int timed_out;               // non-zero once a bounded wait gave up
};

// Called by every thread before the scan starts (ends with a CTA-wide barrier).
__device__ __forceinline__ void stream_begin(StreamBars &bars, int nstages) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
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
__host__ __device__ __forceinline__ int slice_first_tile(int slice, int nslices, int ntiles_row) {
    return (int)((long long)slice * ntiles_row / nslices);
}
template <typename DT>
__device__ __forceinline__ void slice_range(int slice, int nslices, int ntiles_row, int V, int &s0, int &s1) {
    constexpr int TE = tile_elems<DT>();
    s0 = slice_first_tile(slice, nslices, ntiles_row) * TE;
    s1 = min(V, slice_first_tile(slice + 1, nslices, ntiles_row) * TE);
}

// Issue the bulk copy of tile t of the slice at `src` into ring stage s (one thread).
__device__ __forceinline__ void issue_tile(const char *src, int nbytes, int t, int s, unsigned char *ring,
                                           StreamBars &bars) {
    const uint32_t bytes = (uint32_t)min(kTileBytes, nbytes - t * kTileBytes);
    mbar_expect_tx(&bars.full[s], bytes);
    bulk_load(ring + (size_t)s * kTileBytes, src + (size_t)t * kTileBytes, bytes, &bars.full[s]);
}

// Largest of three, NaN if any is NaN (so that one NaN logit shows in a tile's maximum).
__device__ __forceinline__ float max3_nan(float a, float b, float c) {
    float d;
    asm("max.NaN.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float max2_nan(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// What a thread keeps of its column of a slice.
struct ColTop {
    float rm1;      // largest logit of the column (-inf: none finite)
    float rm2;      // largest logit of the column's other tiles (tiles other than t1)
    int t1;         // tile of the slice (0-based) that holds rm1
    float seen;     // NaN-keeping maximum of everything the thread saw: NaN or +inf flags the row
};
struct ColSums {    // S = sum 2^(x*kLog2e - c), T = sum 2^(x*kLog2e - c) * (x*kLog2e - c)
    float c, S, T;
};

// One tile from shared memory into the thread's running values.  nvec: 16-byte vectors of the
// tile that exist (RAGGED: fewer than a whole tile; the missing ones take no part in anything).
template <typename DT, bool SUMS, bool RAGGED>
__device__ __forceinline__ void scan_tile(const uint4 *__restrict__ sp, int nvec, int t, int tid, ColTop &top,
                                          float &c, unsigned long long &S2, unsigned long long &T2) {
    constexpr int N = Elem<DT>::N;
    uint4 v[kVpt];
    if constexpr (!RAGGED) {
#pragma unroll
        for (int j = 0; j < kVpt; ++j) v[j] = sp[j * kThreads + tid];
    } else {
        const uint32_t nw = Elem<DT>::kNegInfWord;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            const int vi = j * kThreads + tid;
            v[j] = vi < nvec ? sp[vi] : make_uint4(nw, nw, nw, nw);
        }
    }
    float x[kVpt][N];
    float vm[kVpt];
#pragma unroll
    for (int j = 0; j < kVpt; ++j) {
#pragma unroll
        for (int e = 0; e < N; ++e) x[j][e] = Elem<DT>::get(v[j], e);
        if constexpr (N == 8) {
            vm[j] = max3_nan(max3_nan(x[j][0], x[j][1], x[j][2]), max3_nan(x[j][3], x[j][4], x[j][5]),
                             max2_nan(x[j][6], x[j][7]));
        } else {
            vm[j] = max2_nan(max3_nan(x[j][0], x[j][1], x[j][2]), x[j][3]);
        }
    }
    float tm = vm[0];
    if constexpr (kVpt == 6) {
        tm = max2_nan(max3_nan(vm[0], vm[1], vm[2]), max3_nan(vm[3], vm[4], vm[5]));
    } else {
#pragma unroll
        for (int j = 1; j < kVpt; ++j) tm = max2_nan(tm, vm[j]);
    }
    // the column's best tile and the best of the others (a NaN maximum changes neither)
    const bool gt = tm > top.rm1;
    top.rm2 = gt ? top.rm1 : fmaxf(top.rm2, tm);
    top.t1 = gt ? t : top.t1;
    top.rm1 = gt ? tm : top.rm1;
    top.seen = max2_nan(top.seen, tm);

    if constexpr (SUMS) {
        const float ts = tm * kLog2e;                 // the reference exponent bounds every logit seen
        if (ts > c) {                                  // both halves move to the new reference exponent
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
            if (RAGGED && j * kThreads + tid >= nvec) continue;
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
}

// The sums of this thread's column of [s0, s1) once more, straight from global memory, against
// the known reference exponent c with the exponent clamped: used when masked (-inf) logits
// poisoned T only (0 * -inf) in the streaming loop.
template <typename DT>
__device__ void redo_column_sums(const DT *__restrict__ row, int s0, int s1, int tid, ColSums &cs) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    const float nc = -cs.c;
    float S = 0.f, T = 0.f;
    for (int base = s0; base < s1; base += TE) {
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            const int e0 = base + (j * kThreads + tid) * N;
            if (e0 < s1) {                                         // vectors are whole: the slice ends on a multiple of N
                const uint4 vv = ldg_stream(row + e0);
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float a = fmaxf(fmaf(Elem<DT>::get(vv, e), kLog2e, nc), -1000.f);
                    const float ex = ex2_approx(a);
                    S += ex;
                    T = fmaf(ex, a, T);
                }
            }
        }
    }
    cs.S = S;
    cs.T = T;
}

// Streams [s0, s1) of `row` through the ring (all kThreads threads of the CTA; `nstages` stages of
// kTileBytes in `ring`).  On return `top` holds the thread's column record and, with SUMS, `cs`
// its sums (c = kRefFloor, S = 0 if the thread saw no finite logit).
template <typename DT, bool SUMS>
__device__ void stream_slice(const DT *__restrict__ row, int s0, int s1, int nstages, StreamBars &bars,
                             unsigned char *ring, ColTop &top, ColSums &cs) {
    constexpr int VT = kTileBytes / 16;
    static_assert(VT == kThreads * kVpt && tile_elems<DT>() * (int)sizeof(DT) == kTileBytes, "tile geometry");
    const int tid = threadIdx.x, lane = tid & 31;
    const int nbytes = (s1 - s0) * (int)sizeof(DT);
    const int ntiles = (nbytes + kTileBytes - 1) / kTileBytes;
    volatile int *abort = &bars.timed_out;

    top.rm1 = -CUDART_INF_F; top.rm2 = -CUDART_INF_F; top.t1 = 0; top.seen = -CUDART_INF_F;
    float c = kRefFloor;
    // the sums of this thread's even and odd logits (register pairs), against the reference exponent c
    unsigned long long S2 = pack2(0.f, 0.f), T2 = pack2(0.f, 0.f);

    // Thread 0 also issues the copies, nstages - 1 tiles ahead of the tile being scanned.
    const char *src = reinterpret_cast<const char *>(row + s0);
    if (tid == 0) {
        for (int tt = 0; tt < min(nstages, ntiles); ++tt) issue_tile(src, nbytes, tt, tt, ring, bars);
    }
    int s = 0;                                       // stage of tile t: t % nstages
    uint32_t ph = 0u;                                // phase parity of tile t in its stage: (t / nstages) & 1
    for (int t = 0; t < ntiles; ++t) {
        if (tid == 0 && t >= 1 && t + nstages - 1 < ntiles) {
            // tile t + nstages - 1 goes to the stage that held tile t - 1, once every warp has released it
            const int es = s == 0 ? nstages - 1 : s - 1;
            if (!mbar_wait(&bars.empty[es], s == 0 ? ph ^ 1u : ph, abort)) bars.timed_out = 1;
            issue_tile(src, nbytes, t + nstages - 1, es, ring, bars);
        }
        if (!mbar_wait(&bars.full[s], ph, abort)) bars.timed_out = 1;
        const int nvec = min(kTileBytes, nbytes - t * kTileBytes) >> 4;
        const uint4 *sp = reinterpret_cast<const uint4 *>(ring + (size_t)s * kTileBytes);
        if (nvec == VT) scan_tile<DT, SUMS, false>(sp, nvec, t, tid, top, c, S2, T2);
        else            scan_tile<DT, SUMS, true>(sp, nvec, t, tid, top, c, S2, T2);
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.empty[s]);   // the stage has been read: release it
        if (++s == nstages) { s = 0; ph ^= 1u; }
    }
    float s0f, s1f, t0f, t1f;
    unpack2(S2, s0f, s1f);
    unpack2(T2, t0f, t1f);
    cs.c = c;
    cs.S = s0f + s1f;
    cs.T = t0f + t1f;
}

// The sums of the threads of a warp against one reference exponent, in double (shuffles only);
// lane 0 gets the result.
__device__ __forceinline__ WarpPartial warp_partial(const ColSums &cs) {
    const float cw = warp_max(cs.c);
    const float d = cs.c - cw;
    const float a = ex2_approx(d);
    // a thread so far below the warp's reference that its weight is zero adds nothing (its S * d
    // may overflow), unless its own sum is NaN or infinite (NaN / +inf logits), which must stay
    // visible; so must a NaN weight (+inf logits of another thread)
    const bool nothing = a == 0.f && cs.S < CUDART_INF_F;
    WarpPartial p;
    p.c = cw; p.pad = 0;
    p.S = warp_sum(nothing ? 0.0 : (double)(cs.S * a));
    p.T = warp_sum(nothing ? 0.0 : (double)((cs.T + cs.S * d) * a));
    return p;
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
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxStages * kTileBytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) rec.dev[dev] = true;
    return e;
}

// Number of SMs of the current device (asked once per device).
inline int device_sm_count() {
    static int sms[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!sms[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        sms[dev] = n;
    }
    return sms[dev];
}

// Rows are cut into slices until about this many CTAs exist.
constexpr int kSliceCtasPerSm = 1;
inline int slice_target_ctas() { return device_sm_count() * kSliceCtasPerSm; }

// Ring depth of a streaming launch of `nblocks` CTAs.  A CTA that shares its SM with two others
// needs no more than three stages (the SM then has six tiles in flight); with fewer CTAs than SM
// slots each CTA takes a deeper ring, because one CTA's copies in flight are what bounds its
// speed: at most two CTAs per SM -> four stages, one CTA per SM -> the whole shared memory.
inline int ring_stages(long long nblocks) {
    const int sms = device_sm_count();
    if (nblocks <= sms) return kMaxStages;
    if (nblocks <= 2ll * sms) return 4;
    return kMinStages;
}

// True if rows of this layout can be streamed with bulk copies.
template <typename DT>
inline bool stream_layout_ok(const void *base, int V, long long stride_b, long long stride_l) {
    const size_t es = sizeof(DT);
    return (reinterpret_cast<uintptr_t>(base) & 15) == 0 && ((size_t)V * es) % 16 == 0 &&
           ((size_t)stride_b * es) % 16 == 0 && ((size_t)stride_l * es) % 16 == 0;
}

}  // namespace dsp
