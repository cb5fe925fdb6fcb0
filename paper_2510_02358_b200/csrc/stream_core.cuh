// TMA-fed variant of the one-pass slice scan for rows whose start, strides and length are
// multiples of 16 bytes.  The slice streams through a ring of shared-memory stages by bulk
// asynchronous copies (cp.async.bulk, completion counted on an mbarrier per stage, no
// multicast) that one consumer thread issues three tiles ahead; the kThreads consumer threads
// read each stage with one 128-bit shared load per vector and do the arithmetic from registers.
// Logits at or above the current threshold are appended to the candidate list of their tile
// (four lists in rotation).  A ninth warp, the fold warp, folds each tile's list into
// a register-resident sorted top-K and publishes a tighter threshold that the consumers pick
// up at their next tile.  The two sides hand over through mbarriers with time-bounded waits,
// so the consumers meet no block-wide barrier after the first tile's threshold bootstrap.  Results are the same as scan_slice's
// (scan_core.cuh): log-sum-exp terms and the exact top-K.
#pragma once

#include "scan_core.cuh"

namespace dsp {

constexpr int kTileBytes = kThreads * kVpt * 16;     // one ring stage = one tile of either dtype
constexpr int kStages = 4;
constexpr int kStreamThreads = kThreads + 32;        // consumers + the fold warp
constexpr int kRingBytes = kStages * kTileBytes;
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
// Non-blocking test of a phase.
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
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

struct StreamBars {
    uint64_t full[kStages];      // stage filled by its bulk copy
    uint64_t empty[kStages];     // stage released by all consumer warps
    uint64_t listed[4];          // list l, phase n: every consumer warp is past tile 4n + l
    uint64_t folded[4];          // list l, phase n: the fold warp has folded tile 4n + l's candidates
};

// The candidates of tile t go to list t % kLists; the list is folded after the tile and must be
// empty again before tile t + kLists, which leaves the fold warp three tiles of slack.
constexpr int kLists = 4;
constexpr int kListCap = kCandCap / kLists;
static_assert(kLists == 4, "StreamBars holds four barriers of each kind");

// Shared state of one slice scan besides ScanSmem.
struct StreamCtl {
    int cnt[kLists];     // entries appended to each candidate list (may exceed kListCap: overflow)
    int nsel;            // keys the fold warp left in ScanSmem::sel after the last fold
    int timed_out;       // non-zero once a bounded wait gave up
};

// Called by every thread before produce/consume start (ends with a CTA-wide barrier).
__device__ __forceinline__ void stream_begin(ScanSmem &sm, StreamCtl &ctl, StreamBars &bars) {
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars.full[s], 1);
            mbar_init(&bars.empty[s], kWarps);
        }
        for (int l = 0; l < kLists; ++l) {
            mbar_init(&bars.listed[l], kWarps);
            mbar_init(&bars.folded[l], 1);
            ctl.cnt[l] = 0;
        }
        mbar_init_fence();
        sm.cnt = 0; sm.thrkey = 0ull; sm.thr_v = -CUDART_INF_F; sm.overflow = 0;
        ctl.nsel = 0; ctl.timed_out = 0;
    }
    __syncthreads();
}

__device__ __forceinline__ unsigned long long umax64(unsigned long long a, unsigned long long b) { return a > b ? a : b; }
__device__ __forceinline__ unsigned long long umin64(unsigned long long a, unsigned long long b) { return a < b ? a : b; }

// Sort 32 keys, one per lane, descending over the lanes (bitonic network).
__device__ __forceinline__ unsigned long long sort32_desc(unsigned long long v, int lane) {
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
            const bool up = (lane & k) == 0;
            const bool lower = (lane & j) == 0;
            v = (lower == up) ? umax64(v, o) : umin64(v, o);
        }
    }
    return v;
}

// Best 32 of two descending 32-key lists (one key per lane each), descending: the lane-wise
// maximum of one list and the other reversed is bitonic and holds the best 32; five
// compare-exchange stages sort it.
__device__ __forceinline__ unsigned long long merge_top32(unsigned long long a, unsigned long long b, int lane) {
    unsigned long long v = umax64(a, __shfl_sync(0xFFFFFFFFu, b, 31 - lane));
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
        v = (lane & j) == 0 ? umax64(v, o) : umin64(v, o);
    }
    return v;
}

// Fold candidate list `which` into the warp's sorted top-32 (one key per lane in `mykey`,
// descending, 0 = empty slot below every real key).  A batch of 32 keys is read at once and
// those that do not beat the K-th key are dropped by one ballot; a few survivors are inserted
// one by one (ballot, shuffle-up, select), many are sorted and merged in.  Empties the list and
// publishes the K-th key's value as the new threshold.  Whole warp.
__device__ __forceinline__ void fold_list(ScanSmem &sm, StreamCtl &ctl, int which, int K,
                                          unsigned long long &mykey) {
    const int lane = threadIdx.x & 31;
    const unsigned long long *list = sm.cand + which * kListCap;
    const int total = ctl.cnt[which];
    const int n = min(total, kListCap);
    unsigned long long kth = __shfl_sync(0xFFFFFFFFu, mykey, K - 1);
    for (int base = 0; base < n; base += 32) {
        unsigned long long key = base + lane < n ? list[base + lane] : 0ull;
        if (!(key > kth)) key = 0ull;
        unsigned pending = __ballot_sync(0xFFFFFFFFu, key != 0ull);
        if (__popc(pending) > 3) {
            mykey = merge_top32(mykey, sort32_desc(key, lane), lane);
        } else {
            while (pending) {
                const int from = __ffs(pending) - 1;
                pending &= pending - 1;
                const unsigned long long nk = __shfl_sync(0xFFFFFFFFu, key, from);
                const int p = __popc(__ballot_sync(0xFFFFFFFFu, mykey > nk));   // keys ahead of nk
                const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, mykey, 1);
                if (lane == p) mykey = nk;
                else if (lane > p) mykey = up;
            }
        }
        kth = __shfl_sync(0xFFFFFFFFu, mykey, K - 1);
    }
    if (lane == 0) {
        if (total > kListCap) sm.overflow = 1;
        ctl.cnt[which] = 0;
        if (kth != 0ull) *reinterpret_cast<volatile float *>(&sm.thr_v) = key_value(kth);
    }
}

// First threshold of a slice from the thread maxima of its first tile, for the consumers of a
// streaming kernel: with r = ceil(K / #warps), the smallest over the warps of each warp's r-th
// largest thread maximum has K distinct logits at or above it.  One barrier; every thread
// derives the value itself and thread 0 also stores it in sm.thr_v.  If some warp has fewer
// than r finite maxima (masked rows) the general rule of bootstrap_threshold applies.
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
    if (t > -CUDART_INF_F) {
        if (tid == 0) sm.thr_v = t;
        return t;
    }
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

// Issue the bulk copy of tile t of the slice at `src` into its ring stage (one thread).
__device__ __forceinline__ void issue_tile(const char *src, int nbytes, int t, unsigned char *ring,
                                           StreamBars &bars) {
    const int s = t % kStages;
    const uint32_t bytes = (uint32_t)min(kTileBytes, nbytes - t * kTileBytes);
    mbar_expect_tx(&bars.full[s], bytes);
    bulk_load(ring + (size_t)s * kTileBytes, src + (size_t)t * kTileBytes, bytes, &bars.full[s]);
}

// The fold warp of a slice scan (32 threads, all of them call this; it takes part in no barrier
// of the CTA after stream_begin and exits when it returns).  For every tile i in order it waits
// until every consumer warp is past the tile (bars.listed), folds list i % kLists into its
// sorted top-32, publishes the threshold and completes the list's bars.folded phase.  After the
// last fold the best min(K, #keys) keys are in sm.sel[0 .. ctl.nsel), sorted.  If a wait gives
// up, the work goes on all the same so that every other wait still ends.
__device__ __forceinline__ void stream_service(int nbytes, int K, ScanSmem &sm, StreamCtl &ctl,
                                               StreamBars &bars) {
    const int lane = threadIdx.x & 31;
    volatile int *abort = &ctl.timed_out;
    const int ntiles = (nbytes + kTileBytes - 1) / kTileBytes;
    unsigned long long mykey = 0ull;
    for (int fold = 0; fold < ntiles; ++fold) {
        const int l = fold % kLists;
        if (!mbar_wait(&bars.listed[l], (fold / kLists) & 1, abort)) ctl.timed_out = 1;
        fold_list(sm, ctl, l, K, mykey);
        if (fold == ntiles - 1) {
            const unsigned have = __ballot_sync(0xFFFFFFFFu, mykey != 0ull && lane < K);
            if (lane < DSP_MAX_K) sm.sel[lane] = mykey;
            if (lane == 0) ctl.nsel = __popc(have);
        }
        __syncwarp();
        if (lane == 0) {
            __threadfence_block();
            mbar_arrive(&bars.folded[l]);
        }
    }
}

// Padding for the vectors past the end of a ragged last tile: -2^124, below every finite
// logit the interface allows, finite when scaled by log2(e), never a candidate (its index is
// past the row).
template <typename DT> struct Pad;
template <> struct Pad<__nv_bfloat16> { static constexpr uint32_t kWord = 0xFD80FD80u; };
template <> struct Pad<float> { static constexpr uint32_t kWord = 0xFD800000u; };

// Consumer side of the scan of [s0, s1) of `row` (kThreads threads, barriers via SyncConsumers;
// the fold warp runs stream_service meanwhile).  Same contract as scan_slice.
template <typename DT, bool SUMS>
__device__ void scan_slice_stream(const DT *__restrict__ row, int s0, int s1, int K, ScanSmem &sm,
                                  StreamCtl &ctl, unsigned char *ring, StreamBars &bars,
                                  float &c_out, double &S_out, double &T_out) {
    using SY = SyncConsumers;
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    constexpr int VT = kTileBytes / 16;
    static_assert(VT == kThreads * kVpt && TE * (int)sizeof(DT) == kTileBytes, "tile geometry");
    const int tid = threadIdx.x, lane = tid & 31;
    const int nbytes = (s1 - s0) * (int)sizeof(DT);
    const int ntiles = (nbytes + kTileBytes - 1) / kTileBytes;

    float c = kRefFloor, S = 0.f, T = 0.f;
    float thr = -CUDART_INF_F;
    volatile int *abort = &ctl.timed_out;

    // the reference exponent must bound every logit below the threshold (those skip the test)
    auto raise_ref = [&](float ts) {
        if (ts > c) {
            const float d = c - ts;
            const float sc = ex2_approx(d);
            T = (T + S * d) * sc;
            S = S * sc;
            c = ts;
        }
    };

    // Thread 0 also issues the copies, kStages - 1 tiles ahead of the tile being scanned.
    const char *src = reinterpret_cast<const char *>(row + s0);
    if (tid == 0) {
        for (int tt = 0; tt < min(kStages, ntiles); ++tt) issue_tile(src, nbytes, tt, ring, bars);
    }
    for (int t = 0; t < ntiles; ++t) {
        if (tid == 0 && t >= 1 && t + kStages - 1 < ntiles) {
            const int tt = t + kStages - 1;           // its stage held tile t - 1
            if (!mbar_wait(&bars.empty[tt % kStages], ((tt / kStages) - 1) & 1, abort)) ctl.timed_out = 1;
            issue_tile(src, nbytes, tt, ring, bars);
        }
        const int s = t % kStages;
        if (!mbar_wait(&bars.full[s], (t / kStages) & 1, abort)) ctl.timed_out = 1;
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

        float thr_now;
        if (t == 0) {
            thr_now = bootstrap_threshold_fast<SY>(sm, tm, K);   // consumers only; no candidate exists yet
        } else {
            thr_now = *reinterpret_cast<volatile float *>(&sm.thr_v);
        }
        if (thr_now > thr) {
            thr = thr_now;
            if constexpr (SUMS) raise_ref(thr * kLog2e);
        }
        // Vectors holding a logit at or above the threshold are few: the warp takes them one at a
        // time and its first N lanes test one logit each, read back from the ring stage.
        if (__ballot_sync(0xFFFFFFFFu, tm >= thr)) {
            if constexpr (SUMS) { if (tm >= thr) raise_ref(tm * kLog2e); }
            const DT *tile = reinterpret_cast<const DT *>(sp);
            const int l = t % kLists;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                unsigned hitters = __ballot_sync(0xFFFFFFFFu, vm[j] >= thr);
                while (hitters) {
                    const int from = __ffs(hitters) - 1;
                    hitters &= hitters - 1;
                    if (lane < N) {
                        const int pos_in_tile = (j * kThreads + (tid - lane) + from) * N + lane;
                        const int idx = s0 + t * TE + pos_in_tile;
                        const float xv = Elem<DT>::load1(tile + pos_in_tile);
                        if (xv >= thr && xv > -CUDART_INF_F && idx < s1) {
                            const int pos = atomicAdd(&ctl.cnt[l], 1);
                            if (pos < kListCap) sm.cand[l * kListCap + pos] = make_key(xv, idx);
                        }
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.empty[s]);   // done with the stage: release it
        if constexpr (SUMS) {
            const float nc = -c;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float a = fmaf(x[j][e], kLog2e, nc);
                    const float ex = ex2_approx(a);
                    S += ex;
                    T = fmaf(ex, a, T);
                }
            }
        }
        // this warp's candidates of tile t are complete; the list of the next tile must have
        // been folded (emptied) since it was last used, kLists tiles earlier
        if (t + 1 < ntiles && t + 1 >= kLists &&
            !mbar_wait(&bars.folded[(t + 1) % kLists], ((t + 1 - kLists) / kLists) & 1, abort))
            ctl.timed_out = 1;
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.listed[t % kLists]);
    }
    // the last fold leaves the slice's best keys, sorted, in sm.sel
    if (!mbar_wait(&bars.folded[(ntiles - 1) % kLists], ((ntiles - 1) / kLists) & 1, abort)) ctl.timed_out = 1;
    const int nsel = min(ctl.nsel, K);
    if (tid < nsel) sm.cand[tid] = sm.sel[tid];
    if (tid == 0) sm.cnt = nsel;
    SY::sync();
    if (sm.overflow) topk_careful<DT, SY>(row, s0, s1, K, sm);

    if constexpr (SUMS) {
        reduce_sums<DT, SY>(row, s0, s1, sm, c, S, T, c_out, S_out, T_out);
    } else {
        c_out = kRefFloor; S_out = 0.0; T_out = 0.0;
    }
}

// The ring needs more dynamic shared memory than the default limit: raise the limit of `kernel`
// once per device (the attribute is per device).  `rec` is the caller's per-kernel record.
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
inline bool stream_layout_ok(const void *base, size_t elem_bytes, int V, long long stride_b,
                             long long stride_l) {
    return (reinterpret_cast<uintptr_t>(base) & 15) == 0 && ((size_t)V * elem_bytes) % 16 == 0 &&
           ((size_t)stride_b * elem_bytes) % 16 == 0 && ((size_t)stride_l * elem_bytes) % 16 == 0;
}

}  // namespace dsp
