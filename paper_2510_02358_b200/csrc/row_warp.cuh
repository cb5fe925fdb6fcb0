// Warp-level pieces of the row finish: sorting networks on 64-bit keys, the merge of the per-warp
// log-sum-exp terms of a row, and a slow but bounded exact top-K for rows with very many equal
// top values.
#pragma once

#include "stream_core.cuh"

namespace dsp {

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

// The n warp partials of a row into one (c, S, T), in double and in a fixed order (each lane
// its strided share in order, then a shuffle tree).  Partials without finite logits are skipped.
// `at(i)` returns partial i (from shared or global memory).
template <typename At>
__device__ __forceinline__ void warp_merge_partials(At at, int n, int lane, float &c_out, double &S_out,
                                                    double &T_out) {
    float cm = kRefFloor;
    for (int i = lane; i < n; i += 32) {
        const WarpPartial p = at(i);
        if (p.S > 0.0 || !(p.S == p.S)) cm = fmaxf(cm, p.c);           // NaN sums must stay visible
    }
    cm = warp_max(cm);
    double Sm = 0.0, Tm = 0.0;
    for (int i = lane; i < n; i += 32) {
        const WarpPartial p = at(i);
        if (p.S != 0.0) {
            const double d = (double)p.c - (double)cm;
            const double a = exp2(d);
            Sm += a * p.S;
            Tm += a * (p.T + p.S * d);
        }
    }
    c_out = cm;
    S_out = warp_sum(Sm);
    T_out = warp_sum(Tm);
}

// Exact top-K of a 16-byte aligned row by one warp, every logit in turn, the
// best 32 keys kept sorted over the lanes.  Slow (the whole row again), bounded, always correct:
// the fallback for rows with very many equal top values.
template <typename DT>
__device__ unsigned long long warp_topk_careful(const DT *__restrict__ row, int V, int K, int lane) {
    constexpr int N = Elem<DT>::N;
    unsigned long long best = 0ull, kth = 0ull;
    for (int base = 0; base < V; base += 32 * N) {
        const int e0 = base + lane * N;
        const bool valid = e0 < V;
        const uint4 vv = valid ? ldg_stream(row + e0) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int e = 0; e < N; ++e) {
            const float x = Elem<DT>::get(vv, e);
            unsigned long long key = valid && x > -CUDART_INF_F ? make_key(x, e0 + e) : 0ull;
            if (!(key > kth)) key = 0ull;
            if (__ballot_sync(0xFFFFFFFFu, key != 0ull)) {
                best = merge_top32(best, sort32_desc(key, lane), lane);
                kth = __shfl_sync(0xFFFFFFFFu, best, K - 1);
            }
        }
    }
    return best;
}

}  // namespace dsp
