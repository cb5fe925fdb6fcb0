// Pass 2 of the streaming path at warp level: one warp finishes one row from what pass 1 left in
// the workspace (stream_core.cuh) with shuffles and a little shared memory of its own, so the
// rows of a CTA never wait for one another.
#pragma once

#include "stream_core.cuh"

namespace dsp {

constexpr int kRowWarps = kWarps;             // rows per CTA of a pass-2 kernel, one warp each
constexpr int kWarpKeyCap = 256;              // element keys a warp can list before it falls back
constexpr int kWarpShareCap = 128;            // (tile, thread) shares a warp can list before it falls back

struct WarpScratch {
    unsigned long long keys[kWarpKeyCap];
    uint32_t shares[kWarpShareCap];
    int nkeys, nshares;
};

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
__device__ __forceinline__ void warp_merge_partials(const WarpPartial *p, int n, int lane, float &c_out,
                                                    double &S_out, double &T_out) {
    float cm = kRefFloor;
    for (int i = lane; i < n; i += 32) {
        const double S = __ldcg(&p[i].S);
        if (S > 0.0 || !(S == S)) cm = fmaxf(cm, __ldcg(&p[i].c));   // NaN sums must stay visible
    }
    cm = warp_max(cm);
    double Sm = 0.0, Tm = 0.0;
    for (int i = lane; i < n; i += 32) {
        const double S = __ldcg(&p[i].S), T = __ldcg(&p[i].T);
        if (S != 0.0) {
            const double d = (double)__ldcg(&p[i].c) - (double)cm;
            const double a = exp2(d);
            Sm += a * S;
            Tm += a * (T + S * d);
        }
    }
    c_out = cm;
    S_out = warp_sum(Sm);
    T_out = warp_sum(Tm);
}

// Sums of a whole 16-byte aligned row against the known reference exponent cb with the exponent
// clamped: used when masked (-inf) logits poisoned T only (0 * -inf) in pass 1.  One warp.
template <typename DT>
__device__ void warp_redo_sums(const DT *__restrict__ row, int V, int lane, float cb, double &Sd, double &Td) {
    constexpr int N = Elem<DT>::N;
    const float nc = -cb;
    double S = 0.0, T = 0.0;
    for (int base = 0; base < V; base += 32 * N * 16) {           // fp32 partial sums of 16 vectors
        float S2 = 0.f, T2 = 0.f;
        for (int q = 0; q < 16; ++q) {
            const int e0 = base + (q * 32 + lane) * N;
            if (e0 < V) {                                          // vectors are whole: V is a multiple of N
                const uint4 vv = ldg_stream(row + e0);
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float a2 = fmaxf(fmaf(Elem<DT>::get(vv, e), kLog2e, nc), -1000.f);
                    const float ex = ex2_approx(a2);
                    S2 += ex;
                    T2 = fmaf(ex, a2, T2);
                }
            }
        }
        S += (double)S2;
        T += (double)T2;
    }
    Sd = warp_sum(S);
    Td = warp_sum(T);
}

// Exact top-K of a 16-byte aligned row by one warp without the table: every logit in turn, the
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

// Exact top-K of a row from its table of per-thread tile maxima (`tab`, ntiles x kThreads, entry
// [t][thread], in global memory) by one warp.  Returns the best 32 keys, one per lane,
// descending (0 = none): the first min(K, #finite) are the row's top K.
//  1. every lane takes 8 table columns; the K-th largest of the lanes' maxima (from the slices'
//     per-thread maxima that pass 1 left after the table's ntiles rows) has at least K logits at
//     or above it (-inf if fewer than K lanes saw a finite logit);
//  2. the (tile, thread) shares whose maximum reaches it are listed, then looked at again, one
//     share per lane (from global memory: L2 hits), and their logits that reach it are listed;
//  3. the list holds the whole top K: it is sorted 32 keys at a time and merged.
// A list that overflows (very many equal top values) sends the row to warp_topk_careful.
template <typename DT>
__device__ unsigned long long warp_select_topk(const DT *__restrict__ row, int V, int K, const DT *tab, int ntiles,
                                               int nslices, WarpScratch &ws, int lane) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    constexpr int VPL = 8 / N;                   // 16-byte vectors holding a lane's 8 table columns
    if (lane == 0) { ws.nkeys = 0; ws.nshares = 0; }
    float rm = -CUDART_INF_F;                    // over the slices' per-thread maxima (the table's last rows)
    for (int sl = 0; sl < nslices; ++sl) {
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(tab + (ntiles + sl) * kThreads + lane * 8 + q * N));
#pragma unroll
            for (int e = 0; e < N; ++e) rm = fmaxf(rm, Elem<DT>::get(v, e));
        }
    }
    const float t0 = __shfl_sync(0xFFFFFFFFu, bitonic_desc(rm, lane), K - 1);
    __syncwarp();
    constexpr int kBatch = 8;                    // tiles whose table vectors are in flight together
    for (int tb = 0; tb < ntiles; tb += kBatch) {
        uint4 v[kBatch][VPL];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
#pragma unroll
            for (int q = 0; q < VPL; ++q) {
                if (tb + u < ntiles)
                    v[u][q] = __ldcg(reinterpret_cast<const uint4 *>(tab + (tb + u) * kThreads + lane * 8 + q * N));
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            if (tb + u < ntiles) {
#pragma unroll
                for (int q = 0; q < VPL; ++q) {
#pragma unroll
                    for (int e = 0; e < N; ++e) {
                        const float m = Elem<DT>::get(v[u][q], e);
                        if (m >= t0 && m > -CUDART_INF_F) {
                            const int pos = atomicAdd(&ws.nshares, 1);
                            if (pos < kWarpShareCap)
                                ws.shares[pos] = (uint32_t)((tb + u) * kThreads + lane * 8 + q * N + e);
                        }
                    }
                }
            }
        }
    }
    __syncwarp();
    const int nshares = ws.nshares;
    if (nshares > kWarpShareCap) return warp_topk_careful<DT>(row, V, K, lane);
    for (int base = 0; base < nshares; base += 32) {
        if (base + lane < nshares) {
            const uint32_t id = ws.shares[base + lane];
            const int e00 = (int)(id / kThreads) * TE + (int)(id % kThreads) * N;
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
                const int e0 = e00 + j * kThreads * N;
                if (e0 < V) {                        // vectors are whole: the row length is a multiple of N
                    const uint4 v = ldg_stream(row + e0);
#pragma unroll
                    for (int e = 0; e < N; ++e) {
                        const float x = Elem<DT>::get(v, e);
                        if (x >= t0 && x > -CUDART_INF_F) {
                            const int pos = atomicAdd(&ws.nkeys, 1);
                            if (pos < kWarpKeyCap) ws.keys[pos] = make_key(x, e0 + e);
                        }
                    }
                }
            }
        }
    }
    __syncwarp();
    const int nkeys = ws.nkeys;
    if (nkeys > kWarpKeyCap) return warp_topk_careful<DT>(row, V, K, lane);
    unsigned long long best = 0ull;
    for (int base = 0; base < nkeys; base += 32) {
        const unsigned long long key = base + lane < nkeys ? ws.keys[base + lane] : 0ull;
        const unsigned long long sorted = sort32_desc(key, lane);
        best = base == 0 ? sorted : merge_top32(best, sorted, lane);
    }
    return best;
}

}  // namespace dsp
