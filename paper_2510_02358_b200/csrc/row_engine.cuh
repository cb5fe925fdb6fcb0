// One vocabulary row from HBM to its statistics in one kernel: the CTAs of a row stream their
// slices (stream_core.cuh) and the CTA that is through last finishes the row on the spot, from
// registers and shared memory (a row of one slice) or from the other slices' small records in
// global memory: sums added up, exact top-K selected.  No CTA waits for another (atomic ticket).
//
// Selection of the exact top-K under (logit desc, id asc), by all threads of the finishing CTA:
//  1. every thread takes one column (all slices) and its largest logit; the columns form 32 groups
//     of 8, and the K-th largest of the groups' maxima has at least K logits at or above it (-inf
//     if fewer exist): the threshold;
//  2. only a column whose largest logit reaches the threshold can hold a top-K logit, and only in
//     the tile recorded for it, unless the largest logit of its other tiles reaches the threshold
//     too (then every tile of that column and slice is looked at): these (tile, column) shares are
//     listed;
//  3. the shares' vectors are read again from global memory, one vector per thread so that all of
//     them are in flight together, and the logits that reach the threshold are listed as keys;
//  4. the list holds the whole top K: every key counts the keys above it (they are unique), which
//     is its place.
// A list that overflows (very many equal top values) sends the row to warp_topk_careful.
#pragma once

#include "row_warp.cuh"
#include "scan_core.cuh"

namespace dsp {

constexpr int kKeyCap = 256;                  // element keys listed before the row falls back
constexpr int kShareCap = 256;                // (tile, column) shares listed before the row falls back

// A thread's column of one slice as it is handed to the finishing CTA (8 bytes).
//   x: largest logit (fp32 bits, exact)
//   y: bits 0-15 the largest logit of the column's other tiles, rounded up to bf16 (only ever
//      compared against the threshold: rounding up can add work, never lose a logit);
//      bits 16-30 the tile of the slice that holds the largest logit; bit 31: NaN or +inf seen.
__device__ __forceinline__ uint32_t bf16_ceil_bits(float v) {
    const uint32_t b = __float_as_uint(v);
    uint32_t h = b >> 16;
    if ((b & 0xFFFFu) != 0u && !(b & 0x80000000u) && (b & 0x7F800000u) != 0x7F800000u) h += 1u;   // positive, inexact: up
    return h;                                                     // negative: dropping bits rounds toward +inf
}
__device__ __forceinline__ uint2 pack_col(const ColTop &t) {
    const bool bad = !(t.seen < CUDART_INF_F);                   // NaN or +inf
    return make_uint2(__float_as_uint(t.rm1), bf16_ceil_bits(t.rm2) | ((uint32_t)t.t1 << 16) | (bad ? 0x80000000u : 0u));
}
__device__ __forceinline__ float col_rm1(uint2 r) { return __uint_as_float(r.x); }
__device__ __forceinline__ float col_rm2(uint2 r) { return __uint_as_float(r.y << 16); }
__device__ __forceinline__ int col_t1(uint2 r) { return (int)((r.y >> 16) & 0x7FFFu); }
__device__ __forceinline__ bool col_bad(uint2 r) { return (r.y & 0x80000000u) != 0u; }
constexpr int kMaxTilesPerSlice = 1 << 15;    // the record's tile field

// Scratch of the finishing CTA; it lies over the ring once the stream is through.
struct FinishSmem {
    __align__(16) unsigned long long keys[kKeyCap + 2];
    unsigned long long order[32];             // the best 32 keys in order
    uint32_t shares[kShareCap];
    __align__(16) uint32_t gmax[4 * kWarps];   // largest logit of every group of 8 columns (order-preserving bits)
    double S, T, lse, mean_x;                 // the row's sums and what follows from them (written by the last warp)
    float c;
    int stats_ok;
    float t0;
    int nkeys, nshares, flag;
};
constexpr int kFinishBytes = (int)((sizeof(FinishSmem) + 255) / 256 * 256);
constexpr int kStashSlices = (kMinStages * kTileBytes - kFinishBytes) / (kThreads * 8);   // column records kept behind it
static_assert(kStashSlices >= kMaxSlices, "the ring must hold the column records of every slice of a row");

// Global scratch of the rows that are cut into several slices.
struct RowScratch {
    unsigned *row_ticket;     // [nrows]                       zeroed per call
    uint2 *cols;              // [nrows, nslices, kThreads]
    WarpPartial *wpart;       // [nrows, nslices, kWarps]
};

// What the finishing CTA's warp 0 gets.
struct RowResult {
    unsigned long long key;   // lane l: the row's l-th best key (0 = none); the first min(K, #finite) count
    float c;                  // sums of the whole row (with `sums`)
    double S, T;
    double lse, mean_x;       // natural-log statistics from the sums (NaN if the row is not finite)
    bool stats_ok;            // the sums describe a finite row
    bool nonfinite;           // a NaN or +inf logit was seen
};

// Barrier 1 of the CTA for its first `nthreads` threads (whole warps): the selecting warps of a
// row finish meet here while the last warp works on its own.
__device__ __forceinline__ void select_barrier(int nthreads) {
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// Inclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ int warp_scan_incl(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += up;
    }
    return v;
}

// The finish of a row by all threads of a CTA.  On entry stash[s * kThreads + tid] holds the column
// records of every slice (behind the FinishSmem in `smem`), the row's warp sums are in wp_own
// (a row of one slice, shared memory) or in ws.wpart (global memory), and a block-wide barrier
// lies between this call and the last use of `smem` for anything else.  Returns true in warp 0.
template <typename DT>
__device__ bool row_finish(const DT *__restrict__ rowp, int V, int K, bool sums, long long row, int nslices,
                           int ntiles_row, const RowScratch &ws, const WarpPartial *wp_own, unsigned char *smem,
                           RowResult &res) {
    constexpr int N = Elem<DT>::N;
    constexpr int TE = tile_elems<DT>();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    FinishSmem &fs = *reinterpret_cast<FinishSmem *>(smem);
    const uint2 *stash = reinterpret_cast<const uint2 *>(smem + kFinishBytes);

    // ---- 1. threshold: the K-th largest of the maxima of 32 groups of 8 neighbouring columns ----
    uint32_t cmax_ord = ord_bits(-CUDART_INF_F);
    bool bad = false;
    for (int s = 0; s < nslices; ++s) {
        const uint2 r = stash[s * kThreads + tid];
        cmax_ord = max(cmax_ord, ord_bits(col_rm1(r)));
        bad |= col_bad(r);
    }
    {
        // each group holds a logit at or above its maximum: K distinct logits reach the K-th largest
        // maximum.  The low five bits of a maximum give way to the group's number (keys are then
        // unique, and lowering a value by less than 32 ulp keeps the threshold valid).
        const uint32_t g = __reduce_max_sync(0xFFu << (lane & 24), cmax_ord);
        if ((lane & 7) == 0) fs.gmax[tid >> 3] = (g & ~31u) | (uint32_t)(31 - (tid >> 3));
    }
    if (tid == 0) { fs.nkeys = 0; fs.nshares = 0; }
    if (tid < 32) fs.order[tid] = 0ull;
    const bool any_bad = __syncthreads_or(bad) != 0;
    // With sums the last warp leaves the others here: it adds up the row's sums and what follows
    // from them (double precision, a long dependent chain) while they select, and meets them again
    // at the last barrier; the others take over its columns.
    const int nsel = sums ? kThreads - 32 : kThreads;  // selecting threads: they meet at barrier 1
    if (sums && warp == kWarps - 1) {
        float c;
        double S, T;
        if (wp_own) {
            warp_merge_partials([&](int i) { return wp_own[i]; }, kWarps, lane, c, S, T);
        } else {
            const WarpPartial *wp = ws.wpart + row * nslices * kWarps;
            warp_merge_partials([&](int i) {
                WarpPartial p;
                p.S = __ldcg(&wp[i].S); p.T = __ldcg(&wp[i].T); p.c = __ldcg(&wp[i].c); p.pad = 0;
                return p;
            }, nslices * kWarps, lane, c, S, T);
        }
        double lse, mean_x;
        const bool ok = row_log_stats(c, S, T, lse, mean_x);
        if (lane == 0) {
            fs.c = c; fs.S = S; fs.T = T; fs.lse = lse; fs.mean_x = mean_x; fs.stats_ok = ok ? 1 : 0;
        }
    } else {
        float t0;
        {
            // every warp ranks the 32 group maxima itself (lane i: value i, by counting the larger ones)
            const uint4 *gp = reinterpret_cast<const uint4 *>(fs.gmax);
            const uint32_t mine = fs.gmax[lane];
            int b0 = 0, b1 = 0, b2 = 0, b3 = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint4 v = gp[q];
                b0 += v.x > mine ? 1 : 0;
                b1 += v.y > mine ? 1 : 0;
                b2 += v.z > mine ? 1 : 0;
                b3 += v.w > mine ? 1 : 0;
            }
            const unsigned who = __ballot_sync(0xFFFFFFFFu, (b0 + b1) + (b2 + b3) == K - 1);
            const uint32_t kb = __shfl_sync(0xFFFFFFFFu, mine, __ffs(who) - 1) & ~31u;
            t0 = kb <= ord_bits(-CUDART_INF_F) ? -CUDART_INF_F : ord_value(kb);    // fewer than K finite maxima: everything finite
        }
        // ---- 2. shares ----
        for (int col0 = warp * 32; col0 < kThreads; col0 += nsel) {
            const int col = col0 + lane;
            for (int s = 0; s < nslices; ++s) {
                const uint2 r = stash[s * kThreads + col];
                const float rm1 = col_rm1(r);
                const bool in = rm1 >= t0 && rm1 > -CUDART_INF_F;
                const bool whole = in && col_rm2(r) >= t0;     // more than one tile of this column may hold a top-K logit
                const int tb = slice_first_tile(s, nslices, ntiles_row);
                const unsigned m = __ballot_sync(0xFFFFFFFFu, in && !whole);
                if (m) {                                       // one tile each: one counter update per warp
                    int base = 0;
                    if (lane == 0) base = atomicAdd(&fs.nshares, __popc(m));
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    const int pos = base + __popc(m & ((1u << lane) - 1u));
                    if (in && !whole && pos < kShareCap) fs.shares[pos] = ((uint32_t)(tb + col_t1(r)) << 8) | (uint32_t)col;
                }
                if (whole) {
                    const int te = slice_first_tile(s + 1, nslices, ntiles_row);
                    const int pos = atomicAdd(&fs.nshares, te - tb);
                    for (int t = tb; t < te; ++t)
                        if (pos + (t - tb) < kShareCap) fs.shares[pos + (t - tb)] = ((uint32_t)t << 8) | (uint32_t)col;
                }
            }
        }
        select_barrier(nsel);
        const int nshares = fs.nshares;

        // ---- 3. keys ----
        if (nshares <= kShareCap) {
            const int items = nshares * kVpt;
            for (int it0 = warp * 32; it0 < items; it0 += nsel) {
                const int it = it0 + lane;
                int e0 = 0;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                unsigned hits = 0u;                    // bit e: element e of this lane's vector reaches the threshold
                if (it < items) {
                    const int sh = it / kVpt, j = it - sh * kVpt;
                    const uint32_t id = fs.shares[sh];
                    e0 = (int)(id >> 8) * TE + (j * kThreads + (int)(id & 255u)) * N;
                    if (e0 < V) {                      // vectors are whole: the row length is a multiple of N
                        v = ldg_stream(rowp + e0);
#pragma unroll
                        for (int e = 0; e < N; ++e) {
                            const float x = Elem<DT>::get(v, e);
                            if (x >= t0 && x > -CUDART_INF_F) hits |= 1u << e;
                        }
                    }
                }
                const int h = __popc(hits);
                const int incl = warp_scan_incl(h, lane);
                const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
                if (total) {                           // one counter update per warp
                    int base = 0;
                    if (lane == 31) base = atomicAdd(&fs.nkeys, total);
                    base = __shfl_sync(0xFFFFFFFFu, base, 31);
                    int pos = base + incl - h;
#pragma unroll
                    for (int e = 0; e < N; ++e) {
                        if (hits & (1u << e)) {
                            if (pos < kKeyCap) fs.keys[pos] = make_key(Elem<DT>::get(v, e), e0 + e);
                            ++pos;
                        }
                    }
                }
            }
            select_barrier(nsel);
            const int nkeys = fs.nkeys;
            // ---- 4. places ----
            if (nkeys <= kKeyCap) {
                if (tid == 0 && (nkeys & 1)) fs.keys[nkeys] = 0ull;    // pad to a whole pair (room: kKeyCap + 2)
                select_barrier(nsel);
                const ulonglong2 *kp = reinterpret_cast<const ulonglong2 *>(fs.keys);
                for (int i = tid; i < nkeys; i += nsel) {
                    const unsigned long long q = fs.keys[i];
                    int place = 0;
                    for (int j = 0; j < ((nkeys + 1) >> 1); ++j) {
                        const ulonglong2 o = kp[j];
                        place += (o.x > q ? 1 : 0) + (o.y > q ? 1 : 0);
                    }
                    if (place < 32) fs.order[place] = q;
                }
            }
        }
    }
    __syncthreads();
    if (warp != 0) return false;

    const bool careful = fs.nshares > kShareCap || fs.nkeys > kKeyCap;    // a list overflowed: the slow, bounded way
    res.key = careful ? warp_topk_careful<DT>(rowp, V, K, lane) : fs.order[lane];
    res.nonfinite = any_bad;
    res.c = kRefFloor; res.S = 0.0; res.T = 0.0;
    res.lse = CUDART_NAN; res.mean_x = CUDART_NAN; res.stats_ok = false;
    if (sums) {
        res.c = fs.c; res.S = fs.S; res.T = fs.T;
        res.lse = fs.lse; res.mean_x = fs.mean_x; res.stats_ok = fs.stats_ok != 0;
    }
    return true;
}

// Streams slice `slice` of `nslices` of the row at `rowp` and, in the CTA that is through last,
// finishes the row.  Returns true in warp 0 of that CTA (with `res` filled in), false in every
// other warp and CTA.  All kThreads threads call it, after stream_begin.  K = 1 .. 32.  A wait of
// the stream that ran out sets DSP_ROW_TIMEOUT in *status_word (before the row can be finished).
// Whatever an earlier kernel of the launch chain prepared (zeroed tickets and status words, see
// launch_prepare) is first touched after the stream: the kernel may start before that kernel
// has ended (programmatic launch) and waits for it here.
template <typename DT>
__device__ bool row_engine(const DT *__restrict__ rowp, int V, int K, bool sums, long long row, int slice,
                           int nslices, int ntiles_row, int nstages, const RowScratch &ws, unsigned *status_word,
                           StreamBars &bars, unsigned char *ring, RowResult &res) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int s0, s1;
    slice_range<DT>(slice, nslices, ntiles_row, V, s0, s1);

    ColTop top;
    ColSums cs;
    cs.c = kRefFloor; cs.S = 0.f; cs.T = 0.f;
    if (sums) stream_slice<DT, true>(rowp, s0, s1, nstages, bars, ring, top, cs);
    else      stream_slice<DT, false>(rowp, s0, s1, nstages, bars, ring, top, cs);

    // masked (-inf) logits leave 0 * -inf in T only: such columns are summed once more, clamped
    const bool poisoned = sums && cs.T != cs.T && cs.S == cs.S && cs.S < CUDART_INF_F;
    if (__syncthreads_or(poisoned)) {                  // also: every warp is through with the ring
        if (poisoned) redo_column_sums<DT>(rowp, s0, s1, tid, cs);
    }
    grid_dependency_wait();
    if (tid == 0 && bars.timed_out) atomicOr(status_word, (unsigned)DSP_ROW_TIMEOUT);
    if (sums) {
        const WarpPartial p = warp_partial(cs);
        if (lane == 0) bars.wp[warp] = p;
    }

    FinishSmem &fs = *reinterpret_cast<FinishSmem *>(ring);
    uint2 *stash = reinterpret_cast<uint2 *>(ring + kFinishBytes);      // [nslices][kThreads]
    const uint2 mine = pack_col(top);
    if (nslices > 1) {
        ws.cols[(row * nslices + slice) * kThreads + tid] = mine;
        if (sums && lane == 0) ws.wpart[(row * nslices + slice) * kWarps + warp] = bars.wp[warp];
        __threadfence();
        __syncthreads();
        if (tid == 0) fs.flag = (int)atomicAdd(&ws.row_ticket[row], 1u);
        __syncthreads();
        if (fs.flag != nslices - 1) return false;
        __threadfence();
        for (int s = 0; s < nslices; ++s)
            stash[s * kThreads + tid] = s == slice ? mine : __ldcg(&ws.cols[(row * nslices + s) * kThreads + tid]);
    } else {
        stash[tid] = mine;
    }
    return row_finish<DT>(rowp, V, K, sums, row, nslices, ntiles_row, ws, nslices > 1 ? nullptr : bars.wp, ring, res);
}

// Global scratch of a launch over `nrows` rows cut into `nslices` slices each.
struct RowScratchLayout {
    size_t off_cols, off_wpart, end;
};
inline RowScratchLayout row_scratch_layout(size_t start, long long nrows, int nslices) {
    RowScratchLayout w;
    size_t o = align_up(start, 256);
    const size_t n = nslices > 1 ? (size_t)nrows * nslices : 0;         // rows of one slice keep everything on chip
    w.off_cols = o;  o += align_up(n * kThreads * sizeof(uint2), 256);
    w.off_wpart = o; o += align_up(n * kWarps * sizeof(WarpPartial), 256);
    w.end = o;
    return w;
}

// ---- what a launch chain prepares before its streaming kernel ----
// One small kernel instead of memset nodes: zeroes up to two word ranges (tickets and status words
// of the workspace, status words of the outputs) and fills one int32 range (gen_len = L).  The
// streaming kernel that follows may be launched as its programmatic dependent: it touches none of
// this before its rows are streamed.
struct PrepareArgs {
    uint32_t *zero_a; long long n_a;
    uint32_t *zero_b; long long n_b;
    int32_t *fill; long long n_fill; int32_t fill_value;
};
static __global__ void __launch_bounds__(kThreads) prepare_kernel(const PrepareArgs a) {
    grid_launch_dependents();
    const long long i0 = (long long)blockIdx.x * kThreads + threadIdx.x, step = (long long)gridDim.x * kThreads;
    for (long long i = i0; i < a.n_a; i += step) a.zero_a[i] = 0u;
    for (long long i = i0; i < a.n_b; i += step) a.zero_b[i] = 0u;
    for (long long i = i0; i < a.n_fill; i += step) a.fill[i] = a.fill_value;
}
inline cudaError_t launch_prepare(const PrepareArgs &a, cudaStream_t st) {
    long long n = a.n_a > a.n_b ? a.n_a : a.n_b;
    if (a.n_fill > n) n = a.n_fill;
    long long blocks = (n + kThreads - 1) / kThreads;
    if (blocks < 1) blocks = 1;
    if (blocks > 1024) blocks = 1024;
    prepare_kernel<<<(unsigned)blocks, kThreads, 0, st>>>(a);
    return cudaGetLastError();
}

}  // namespace dsp
