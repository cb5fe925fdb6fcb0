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
    __align__(16) unsigned long long keys[kWarpKeyCap + 2];
    unsigned long long order[32];               // the best 32 keys in order
    uint32_t shares[kWarpShareCap];
    unsigned short cols[kThreads];              // thread columns that can hold a top-K logit
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
    // the lane's first partial stays in registers (with n <= 32 nothing is read twice)
    double S0 = 0.0, T0 = 0.0;
    float c0 = kRefFloor;
    if (lane < n) { S0 = __ldcg(&p[lane].S); T0 = __ldcg(&p[lane].T); c0 = __ldcg(&p[lane].c); }
    float cm = kRefFloor;
    if (S0 > 0.0 || !(S0 == S0)) cm = c0;                             // NaN sums must stay visible
    for (int i = lane + 32; i < n; i += 32) {
        const double S = __ldcg(&p[i].S);
        if (S > 0.0 || !(S == S)) cm = fmaxf(cm, __ldcg(&p[i].c));
    }
    cm = warp_max(cm);
    double Sm = 0.0, Tm = 0.0;
    for (int i = lane; i < n; i += 32) {
        const double S = i == lane ? S0 : __ldcg(&p[i].S), T = i == lane ? T0 : __ldcg(&p[i].T);
        if (S != 0.0) {
            const double d = (double)(i == lane ? c0 : __ldcg(&p[i].c)) - (double)cm;
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

// One table entry (written by an earlier kernel), past the L1.
__device__ __forceinline__ float table_load(const __nv_bfloat16 *p) {
    return __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short *>(p)) << 16);
}
__device__ __forceinline__ float table_load(const float *p) { return __ldcg(p); }

// The K-th largest (K = 1 .. 32) of the lanes' values: every lane counts the lanes that come
// before it (larger value, or equal value and lower lane); the lane with K - 1 before it has it.
__device__ __forceinline__ float warp_kth_largest(float v, int K, int lane) {
    int before = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const float o = __shfl_sync(0xFFFFFFFFu, v, j);
        before += (o > v || (o == v && j < lane)) ? 1 : 0;
    }
    const unsigned who = __ballot_sync(0xFFFFFFFFu, before == K - 1);
    return __shfl_sync(0xFFFFFFFFu, v, __ffs(who) - 1);
}

// Exact top-K of a row from its table of per-thread tile maxima (`tab`, ntiles x kThreads, entry
// [t][thread], in global memory, then one more row per slice with every thread's maximum over
// the slice) by one warp.  Returns the best 32 keys, one per lane, descending (0 = none): the
// first min(K, #finite) are the row's top K.
//  1. every lane takes 8 thread columns and their maxima over the row; the K-th largest of the
//     lanes' maxima has at least K logits at or above it (-inf if fewer than K lanes saw a finite
//     logit) and serves as threshold;
//  2. only columns whose maximum reaches the threshold can hold a top-K logit: their table
//     entries are fetched (all loads of a round in flight together) and the (tile, thread) shares
//     that reach it are listed;
//  3. the shares are looked at again, one per lane (from global memory), and their logits that
//     reach the threshold are listed;
//  4. the list holds the whole top K: every key counts the keys above it, which is its place.
// A list that overflows (very many equal top values) sends the row to warp_topk_careful.
template <typename DT>
__device__ unsigned long long warp_select_topk(const DT *__restrict__ row, int V, int K, const DT *tab, int ntiles,
                                               int nslices, WarpScratch &ws, int lane) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    constexpr int VPL = 8 / N;                   // 16-byte vectors holding a lane's 8 table columns
    constexpr int kPairBatch = 16;               // table entries a lane has in flight
    if (lane == 0) { ws.nkeys = 0; ws.nshares = 0; }
    float cm[8];                                 // the lane's columns: maxima over the row
#pragma unroll
    for (int j = 0; j < 8; ++j) cm[j] = -CUDART_INF_F;
    for (int sl = 0; sl < nslices; ++sl) {
#pragma unroll
        for (int q = 0; q < VPL; ++q) {
            const uint4 v = __ldcg(reinterpret_cast<const uint4 *>(tab + (ntiles + sl) * kThreads + lane * 8 + q * N));
#pragma unroll
            for (int e = 0; e < N; ++e) cm[q * N + e] = fmaxf(cm[q * N + e], Elem<DT>::get(v, e));
        }
    }
    float rm = cm[0];
#pragma unroll
    for (int j = 1; j < 8; ++j) rm = fmaxf(rm, cm[j]);
    const float t0 = K == 1 ? warp_max(rm) : warp_kth_largest(rm, K, lane);
    int ncols = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const bool in = cm[j] >= t0 && cm[j] > -CUDART_INF_F;
        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, in);
        if (in) ws.cols[ncols + __popc(ballot & ((1u << lane) - 1u))] = (unsigned short)(lane * 8 + j);
        ncols += __popc(ballot);
    }
    __syncwarp();
    const int npairs = ncols * ntiles;
    for (int p0 = 0; p0 < npairs; p0 += 32 * kPairBatch) {
        float mv[kPairBatch];
        int at[kPairBatch];
#pragma unroll
        for (int u = 0; u < kPairBatch; ++u) {
            const int p = p0 + u * 32 + lane;
            mv[u] = -CUDART_INF_F;
            at[u] = 0;
            if (p < npairs) {
                const int ci = p / ntiles, t = p - ci * ntiles;
                at[u] = t * kThreads + ws.cols[ci];
                mv[u] = table_load(tab + at[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kPairBatch; ++u) {
            if (mv[u] >= t0 && mv[u] > -CUDART_INF_F) {
                const int pos = atomicAdd(&ws.nshares, 1);
                if (pos < kWarpShareCap) ws.shares[pos] = (uint32_t)at[u];
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
            uint4 v[kVpt];
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {     // the share's vectors leave together
                const int e0 = e00 + j * kThreads * N;
                v[j] = e0 < V ? ldg_stream(row + e0)      // vectors are whole: the row length is a multiple of N
                              : make_uint4(Elem<DT>::kNegInfWord, Elem<DT>::kNegInfWord, Elem<DT>::kNegInfWord,
                                           Elem<DT>::kNegInfWord);
            }
#pragma unroll
            for (int j = 0; j < kVpt; ++j) {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float x = Elem<DT>::get(v[j], e);
                    if (x >= t0 && x > -CUDART_INF_F) {
                        const int pos = atomicAdd(&ws.nkeys, 1);
                        if (pos < kWarpKeyCap) ws.keys[pos] = make_key(x, e00 + j * kThreads * N + e);
                    }
                }
            }
        }
    }
    __syncwarp();
    const int nkeys = ws.nkeys;
    if (nkeys > kWarpKeyCap) return warp_topk_careful<DT>(row, V, K, lane);
    // every key's place = the keys above it (the keys are unique); the first 32 places are kept
    if (lane == 0 && (nkeys & 1)) ws.keys[nkeys] = 0ull;           // pad to a whole pair (room: kWarpKeyCap + 2)
    ws.order[lane] = 0ull;
    __syncwarp();
    const ulonglong2 *kp = reinterpret_cast<const ulonglong2 *>(ws.keys);
    for (int base = 0; base < nkeys; base += 32) {
        if (base + lane < nkeys) {
            const unsigned long long q = ws.keys[base + lane];
            int place = 0;
            for (int j = 0; j < ((nkeys + 1) >> 1); ++j) {
                const ulonglong2 o = kp[j];
                place += (o.x > q ? 1 : 0) + (o.y > q ? 1 : 0);
            }
            if (place < 32) ws.order[place] = q;
        }
    }
    __syncwarp();
    return ws.order[lane];
}

}  // namespace dsp
