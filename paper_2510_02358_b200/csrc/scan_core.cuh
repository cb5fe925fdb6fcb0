// One-pass streaming scan of a slice of a vocabulary row: running log-sum-exp terms and the
// exact top-K under (logit desc, id asc).  Used by the lattice kernel (K = K_max, sums on)
// and by the target-row kernel of verification (K = 1, sums only for stochastic rows).
#pragma once

#include "dsp_common.cuh"

namespace dsp {

struct ScanSmem {
    unsigned long long cand[kCandCap];   // candidate keys appended by the streaming loop
    unsigned long long sel[DSP_MAX_K];   // output of a prune: the best keys, sorted
    unsigned long long thrkey;           // K-th best key so far (0 = none yet)
    float wsorted[kWarps][32];           // per-warp sorted thread maxima (threshold bootstrap)
    double redS[kWarps], redT[kWarps];
    float redc[kWarps];
    double pk[DSP_MAX_K + 1];            // finaliser scratch
    double fin[4];
    float thr_v;                         // value of the K-th best key so far (-inf = none yet)
    int cnt;                             // entries in cand (may exceed kCandCap: overflow)
    int overflow;
    int flag;
};

// Block-wide barrier policy of the helpers below: every thread of the CTA.
struct SyncAll {
    static __device__ __forceinline__ void sync() { __syncthreads(); }
};

template <typename DT>
__device__ __forceinline__ uint4 load_vec(const DT *__restrict__ row, int e0, int end, bool aligned) {
    constexpr int N = Elem<DT>::N;
    if (aligned && e0 + N <= end) return ldg_stream(row + e0);
    const uint32_t ninf = Elem<DT>::kNegInfWord;
    uint4 v = make_uint4(ninf, ninf, ninf, ninf);
    if (e0 < end) {
        uint32_t w[4] = {ninf, ninf, ninf, ninf};
        if constexpr (N == 8) {
            const unsigned short *p = reinterpret_cast<const unsigned short *>(row);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (e0 + e < end) {
                    uint32_t h = p[e0 + e];
                    w[e >> 1] = (e & 1) ? ((w[e >> 1] & 0x0000FFFFu) | (h << 16))
                                        : ((w[e >> 1] & 0xFFFF0000u) | h);
                }
            }
        } else {
            const uint32_t *p = reinterpret_cast<const uint32_t *>(row);
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (e0 + e < end) w[e] = p[e0 + e];
        }
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    return v;
}

// Keep the best min(K, n) of the n = min(cnt, cap) buffered keys, sorted, at the front of
// cand; refresh the thresholds.  Every key is unique, so ranks are unique.  Block-wide.
template <typename SY = SyncAll>
__device__ __forceinline__ void prune(ScanSmem &sm, int K) {
    SY::sync();
    const int tid = threadIdx.x;
    const int n = min(sm.cnt, kCandCap);
    if (tid == 0 && sm.cnt > kCandCap) sm.overflow = 1;
    for (int i = tid; i < n; i += kThreads) {
        const unsigned long long key = sm.cand[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += sm.cand[j] > key;
        if (rank < K) sm.sel[rank] = key;
    }
    SY::sync();
    const int nk = min(n, K);
    if (tid < nk) sm.cand[tid] = sm.sel[tid];
    if (tid == 0) {
        sm.cnt = nk;
        if (nk == K) {
            sm.thrkey = sm.sel[K - 1];
            sm.thr_v = key_value(sm.sel[K - 1]);
        }
    }
    SY::sync();
}

__device__ __forceinline__ float bitonic_desc(float v, int lane) {
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            const float o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
            const bool up = (lane & k) == 0;
            const bool lower = (lane & j) == 0;
            v = (lower == up) ? fmaxf(v, o) : fminf(v, o);
        }
    }
    return v;
}

// First threshold of a slice from the 256 thread maxima of its first tile: the smallest r
// such that r * (#warps whose r-th largest thread maximum is finite) >= K gives K distinct
// elements >= min over those warps of that r-th largest.  -inf if there is no such r.
template <typename SY = SyncAll>
__device__ __forceinline__ void bootstrap_threshold(ScanSmem &sm, float tm, int K) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float s = bitonic_desc(tm == tm ? tm : -CUDART_INF_F, lane);
    sm.wsorted[warp][lane] = s;
    SY::sync();
    if (tid == 0) {
        float t = -CUDART_INF_F;
        for (int r = 1; r <= 32; ++r) {
            int nw = 0;
            float lo = CUDART_INF_F;
            for (int w = 0; w < kWarps; ++w) {
                const float x = sm.wsorted[w][r - 1];
                if (x > -CUDART_INF_F) { ++nw; lo = fminf(lo, x); }
            }
            if (nw == 0) break;
            if (r * nw >= K) { t = lo; break; }
        }
        sm.thr_v = t;
    }
    SY::sync();
}

// Exact top-K of a slice when the fast path overflowed its buffer (heavily tied or
// adversarially ordered rows): one element per thread per round, exact key test, prune
// whenever another round could overflow.  Slow, bounded, always correct.
template <typename DT, typename SY = SyncAll>
__device__ void topk_careful(const DT *__restrict__ row, int s0, int s1, int K, ScanSmem &sm) {
    const int tid = threadIdx.x;
    SY::sync();
    if (tid == 0) { sm.cnt = 0; sm.thrkey = 0ull; sm.thr_v = -CUDART_INF_F; sm.overflow = 0; }
    SY::sync();
    for (int base = s0; base < s1; base += kThreads) {
        const int idx = base + tid;
        if (idx < s1) {
            const float x = Elem<DT>::load1(row + idx);
            if (x > -CUDART_INF_F) {
                const unsigned long long key = make_key(x, idx);
                if (key > sm.thrkey) {
                    const int pos = atomicAdd(&sm.cnt, 1);
                    sm.cand[pos] = key;
                }
            }
        }
        SY::sync();
        const int n = sm.cnt;          // read between two barriers: the same value in every thread
        SY::sync();
        if (n > kCandCap - kThreads) prune<SY>(sm, K);
    }
    prune<SY>(sm, K);
}

// Sums of [s0, s1) of `row` against the known reference exponent cb with the exponent clamped:
// used when masked (-inf) logits poisoned T only (0 * -inf) in the streaming pass.  Block-wide.
template <typename DT, typename SY>
__device__ void redo_sums(const DT *__restrict__ row, int s0, int s1, ScanSmem &sm, float cb,
                          double &Sd, double &Td) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool aligned = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
    const int ntiles = (s1 - s0 + TE - 1) / TE;
    const float nc = -cb;
    float S2 = 0.f, T2 = 0.f;
    for (int t = 0; t < ntiles; ++t) {
        const int base = s0 + t * TE;
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            const uint4 vv = load_vec<DT>(row, base + (j * kThreads + tid) * N, s1, aligned);
#pragma unroll
            for (int e = 0; e < N; ++e) {
                const float x = Elem<DT>::get(vv, e);
                const float a2 = fmaxf(fmaf(x, kLog2e, nc), -1000.f);
                const float ex = ex2_approx(a2);
                S2 += ex;
                T2 = fmaf(ex, a2, T2);
            }
        }
    }
    double S2d = warp_sum((double)S2), T2d = warp_sum((double)T2);
    if (lane == 0) { sm.redS[warp] = S2d; sm.redT[warp] = T2d; }
    SY::sync();
    Sd = 0.0; Td = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { Sd += sm.redS[w]; Td += sm.redT[w]; }
    SY::sync();
}

// Block reduction of the per-thread sums (c, S, T) of a slice to one reference exponent, in
// double.  If masked (-inf) logits poisoned T only (0 * -inf), the slice's sums are redone from
// global memory against the now known reference with the exponent clamped.
template <typename DT, typename SY>
__device__ void reduce_sums(const DT *__restrict__ row, int s0, int s1, ScanSmem &sm, float c, float S,
                            float T, float &c_out, double &S_out, double &T_out) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float cb = warp_max(c);
    if (lane == 0) sm.redc[warp] = cb;
    SY::sync();
    cb = sm.redc[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) cb = fmaxf(cb, sm.redc[w]);
    const float d = c - cb;
    const float a = ex2_approx(d);
    double Sd = warp_sum((double)(S * a));
    double Td = warp_sum((double)((T + S * d) * a));
    if (lane == 0) { sm.redS[warp] = Sd; sm.redT[warp] = Td; }
    SY::sync();
    Sd = 0.0; Td = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { Sd += sm.redS[w]; Td += sm.redT[w]; }
    SY::sync();

    if (Td != Td && Sd == Sd && Sd < CUDART_INF) redo_sums<DT, SY>(row, s0, s1, sm, cb, Sd, Td);
    c_out = cb; S_out = Sd; T_out = Td;
}

// Scan [s0, s1) of `row`.  On return (after a block barrier) sm.cand[0 .. sm.cnt) holds the
// slice's best min(K, #finite) keys, sorted; with SUMS the slice's
//   S = sum 2^(x*kLog2e - c),  T = sum 2^(x*kLog2e - c) * (x*kLog2e - c)
// are returned relative to the reference exponent c (kRefFloor if the slice has no finite
// logit).  -inf logits contribute nothing; NaN / +inf logits leave S non-finite.
template <typename DT, bool SUMS>
__device__ void scan_slice(const DT *__restrict__ row, int s0, int s1, int K, ScanSmem &sm,
                           float &c_out, double &S_out, double &T_out) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool aligned = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
    const int ntiles = (s1 - s0 + TE - 1) / TE;

    if (tid == 0) { sm.cnt = 0; sm.thrkey = 0ull; sm.thr_v = -CUDART_INF_F; sm.overflow = 0; }
    __syncthreads();

    float c = kRefFloor, S = 0.f, T = 0.f;
    float thr = -CUDART_INF_F;

    for (int t = 0; t < ntiles; ++t) {
        const int base = s0 + t * TE;
        uint4 v[kVpt];
#pragma unroll
        for (int j = 0; j < kVpt; ++j)
            v[j] = load_vec<DT>(row, base + (j * kThreads + tid) * N, s1, aligned);
        float vm[kVpt];
#pragma unroll
        for (int j = 0; j < kVpt; ++j) vm[j] = Elem<DT>::vmax(v[j]);
        const float tm = fmaxf(fmaxf(fmaxf(vm[0], vm[1]), fmaxf(vm[2], vm[3])), fmaxf(vm[4], vm[5]));

        if constexpr (SUMS) {
            const float cn = fmaxf(c, tm * kLog2e);
            const float d = c - cn;
            const float sc = ex2_approx(d);
            T = (T + S * d) * sc;
            S = S * sc;
            c = cn;
            const float nc = -c;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float x = Elem<DT>::get(v[j], e);
                    const float a = fmaf(x, kLog2e, nc);
                    const float ex = ex2_approx(a);
                    S += ex;
                    T = fmaf(ex, a, T);
                }
            }
        }

        if (t == 0) {
            bootstrap_threshold(sm, tm, K);
            thr = sm.thr_v;
        }
        // vectors holding a logit at or above the threshold are tested element-wise by the warp
#pragma unroll
        for (int j = 0; j < kVpt; ++j) {
            const bool hit = vm[j] >= thr && vm[j] > -CUDART_INF_F;
            unsigned bal = __ballot_sync(0xFFFFFFFFu, hit);
            while (bal) {
                const int src = __ffs(bal) - 1;
                bal &= bal - 1;
                uint4 w;
                w.x = __shfl_sync(0xFFFFFFFFu, v[j].x, src);
                w.y = __shfl_sync(0xFFFFFFFFu, v[j].y, src);
                w.z = __shfl_sync(0xFFFFFFFFu, v[j].z, src);
                w.w = __shfl_sync(0xFFFFFFFFu, v[j].w, src);
                if (lane < N) {
                    const float x = Elem<DT>::get(w, lane);
                    const int idx = base + (j * kThreads + warp * 32 + src) * N + lane;
                    if (x >= thr && x > -CUDART_INF_F && idx < s1) {
                        const int pos = atomicAdd(&sm.cnt, 1);
                        if (pos < kCandCap) sm.cand[pos] = make_key(x, idx);
                    }
                }
            }
        }
        if (t == 0 || ((t + 1) & t) == 0 || t == ntiles - 1) {
            prune(sm, K);
            thr = sm.thr_v;
        }
    }
    if (ntiles == 0) __syncthreads();
    if (sm.overflow) topk_careful<DT>(row, s0, s1, K, sm);

    if constexpr (SUMS) {
        reduce_sums<DT, SyncAll>(row, s0, s1, sm, c, S, T, c_out, S_out, T_out);
    } else {
        c_out = kRefFloor; S_out = 0.0; T_out = 0.0;
    }
}

// Per-slice record in the workspace when a row is split over several CTAs.
struct SlicePartial {
    double S, T;
    float c;
    int nkeys;
};

// Merge per-slice sums (fixed slice order, double).  Slices without finite logits are skipped.
__device__ __forceinline__ void merge_partials(const SlicePartial *p, int n, float &c, double &S, double &T) {
    float cm = kRefFloor;
    for (int s = 0; s < n; ++s) {
        const float cs = __ldcg(&p[s].c);
        if (__ldcg(&p[s].S) > 0.0 || !(__ldcg(&p[s].S) == __ldcg(&p[s].S))) cm = fmaxf(cm, cs);
    }
    double Sm = 0.0, Tm = 0.0;
    for (int s = 0; s < n; ++s) {
        const double Ss = __ldcg(&p[s].S), Ts = __ldcg(&p[s].T);
        const float cs = __ldcg(&p[s].c);
        if (Ss == 0.0) continue;
        const double d = (double)cs - (double)cm;
        const double a = exp2(d);
        Sm += a * Ss;
        Tm += a * (Ts + Ss * d);
    }
    c = cm; S = Sm; T = Tm;
}

// Natural-log statistics of a row from its merged sums: log-sum-exp, mean logit under the
// softmax, with the kLog2e tilt removed to first order.  Returns false if the row is not finite.
__device__ __forceinline__ bool row_log_stats(float c, double S, double T, double &lse, double &mean_x) {
    if (!(S > 0.0) || !(S < CUDART_INF) || !(T == T) || !(c > kRefFloor) || !(c < CUDART_INF_F)) {
        lse = CUDART_NAN; mean_x = CUDART_NAN;
        return false;
    }
    mean_x = (T / S + (double)c) / (double)kLog2e;
    lse = kLn2 * ((double)c + log2(S)) + kTilt * mean_x;
    return true;
}

// How a row is cut into slices: `tiles_per_slice` whole tiles each (the last may be shorter).
struct SlicePlan {
    int nslices;
    int slice_elems;
};
template <typename DT>
inline SlicePlan plan_slices(int64_t nrows, int V, int target_ctas) {
    const int TE = tile_elems<DT>();
    const int ntiles = (V + TE - 1) / TE;
    int want = (int)((target_ctas + nrows - 1) / (nrows > 0 ? nrows : 1));   // slices per row wanted
    if (want < 1) want = 1;
    int tps = (ntiles + want - 1) / want;            // tiles per slice
    if (tps > 32) tps = 32;                          // bounds the time one CTA holds its SM slot
    const int min_tps = (ntiles + kMaxSlices - 1) / kMaxSlices;
    if (tps < min_tps) tps = min_tps;
    if (tps < 1) tps = 1;
    SlicePlan p;
    p.nslices = (ntiles + tps - 1) / tps;
    if (p.nslices < 1) p.nslices = 1;
    p.slice_elems = tps * TE;
    return p;
}

}  // namespace dsp
