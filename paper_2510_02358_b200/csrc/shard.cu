// dsp_lattice_shard / dsp_lattice_merge: the lattice of a vocabulary-sharded drafter head.
//
// With a tensor-parallel output layer every GPU holds the logits of one slice of the vocabulary.
// Each GPU reduces its slice of every row to a small record (dsp_lattice_shard: the slice's sums
// for the log-sum-exp and the entropy, its best K_max keys with global token ids, the EOS logit
// if the slice holds it); the records of all slices are gathered into one buffer (one small
// all-gather: (24 + 8 K_max) bytes per row and slice, copied into local memory first) and
// dsp_lattice_merge finishes the rows exactly as dsp_lattice_build does on the whole row:
// top-K by merging the sorted key lists (integer compares: the same K tokens as unsharded), the
// sums added up against a common reference exponent, then Eq. 7, the EOS slot, Eq. 9.
#include "dsp_internal.h"
#include "lattice_rows.cuh"

namespace dsp {

static_assert(sizeof(dsp_shard_sums) == 24, "record layout is part of the ABI");

struct ShardArgs {
    const void *logits;
    int B, L, V;              // V: the slice's length
    long long stride_b, stride_l;
    int vocab_offset, K, K_max, eos_id;
    const int32_t *path, *path_len;   // target side: the row's probe token is its path token (else eos_id)
    int Lp;                           // row length of `path`
    dsp_shard_sums *sums;     // [B,L]
    unsigned long long *keys; // [B,L,K_max]
    uint32_t *shard_status;   // [B]
    int nslices, slice_elems, ntiles_row, nstages;
    RowScratch rs;            // records of rows cut into several slices (streaming path)
};

struct ShardWs {
    size_t off_row_ticket, zero_bytes;
    RowScratchLayout rs;
    size_t total;
};
static ShardWs shard_ws_layout(int64_t B, int64_t L, int nslices) {
    ShardWs w;
    size_t o = 0;
    w.off_row_ticket = o; o += align_up((size_t)(B * L) * 4, 256);
    w.zero_bytes = o;
    w.rs = row_scratch_layout(o, B * L, nslices);
    w.total = w.rs.end;
    return w;
}

// The record of one row of the slice, written by one warp from the row's best keys and sums.
// (shard_status is prepared as 0 before the kernel; a wait that ran out is OR-ed into it.)
template <typename DT>
__device__ __forceinline__ void shard_write_row(const ShardArgs &a, long long row, int b, int l, const DT *rowp,
                                                unsigned long long key, float c, double S, double T, int lane) {
    // keys carry global token ids
    if (lane < a.K_max) {
        unsigned long long out = 0ull;
        if (lane < a.K && key != 0ull) out = make_key(key_value(key), key_id(key) + a.vocab_offset);
        a.keys[row * a.K_max + lane] = out;
    }
    if (lane == 0) {
        dsp_shard_sums r;
        r.S = S; r.T = T; r.c = c;
        int probe = a.eos_id;                  // the one token whose logit the record carries
        if (a.path) probe = (l < a.Lp && l < __ldg(&a.path_len[b])) ? __ldg(&a.path[(long long)b * a.Lp + l]) : -1;
        const int e = probe - a.vocab_offset;
        r.eos_logit = (probe >= 0 && e >= 0 && e < a.V) ? Elem<DT>::load1(rowp + e) : CUDART_NAN_F;
        a.sums[row] = r;
    }
}

// Streaming path: one CTA per row slice; the CTA that is through with a row last writes its record.
template <typename DT>
__global__ void __launch_bounds__(kThreads, 3) shard_scan_kernel(const ShardArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ StreamBars bars;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    stream_begin(bars, a.nstages);
    RowResult r;
    if (!row_engine<DT>(rowp, a.V, a.K, true, row, slice, a.nslices, a.ntiles_row, a.nstages, a.rs, &a.shard_status[b],
                        bars, ring, r))
        return;
    // a NaN or +inf logit must show in the record's sums, whichever unit took its exponential
    shard_write_row<DT>(a, row, b, l, rowp, r.key, r.c, r.nonfinite ? CUDART_NAN : r.S, r.T, threadIdx.x & 31);
}

// Sums and exact top-K of a row that cannot be streamed, element by element, by one warp.
template <typename DT>
__device__ unsigned long long warp_row_elementwise(const DT *__restrict__ row, int V, int K, int lane, float &c_out,
                                                   double &S_out, double &T_out) {
    float m = -CUDART_INF_F;
    unsigned long long best = 0ull, kth = 0ull;
    for (int v0 = 0; v0 < V; v0 += 32) {
        const int v = v0 + lane;
        const float x = v < V ? Elem<DT>::load1(row + v) : -CUDART_INF_F;
        if (x == x && x < CUDART_INF_F) m = fmaxf(m, x);
        unsigned long long key = (v < V && x > -CUDART_INF_F) ? make_key(x, v) : 0ull;   // NaN: no key
        if (!(key > kth)) key = 0ull;
        if (__ballot_sync(0xFFFFFFFFu, key != 0ull)) {
            best = merge_top32(best, sort32_desc(key, lane), lane);
            kth = __shfl_sync(0xFFFFFFFFu, best, K - 1);
        }
    }
    m = warp_max(m);
    const float c = m > -CUDART_INF_F ? m * kLog2e : kRefFloor;
    double S = 0.0, T = 0.0;
    for (int v0 = lane; v0 < V; v0 += 32 * 64) {         // fp32 partial sums of 64 terms, added up in double
        float s = 0.f, t = 0.f;
        for (int q = 0; q < 64; ++q) {
            const int v = v0 + q * 32;
            if (v < V) {
                const float x = Elem<DT>::load1(row + v);
                if (x > -CUDART_INF_F || x != x) {       // -inf adds nothing; NaN / +inf must show in the sums
                    const float a2 = fmaf(x, kLog2e, -c);
                    const float ex = ex2_approx(a2);
                    s += ex;
                    t = fmaf(ex, a2, t);
                }
            }
        }
        S += (double)s;
        T += (double)t;
    }
    c_out = c;
    S_out = warp_sum(S);
    T_out = warp_sum(T);
    return best;
}

// Layouts that cannot be streamed: one warp per row, element by element.
template <typename DT>
__global__ void __launch_bounds__(kThreads) shard_rows_kernel(const ShardArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long row = (long long)blockIdx.x * kWarps + warp;
    if (row >= (long long)a.B * a.L) return;
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    float c;
    double S, T;
    const unsigned long long key = warp_row_elementwise<DT>(rowp, a.V, a.K, lane, c, S, T);
    shard_write_row<DT>(a, row, b, l, rowp, key, c, S, T, lane);
}

struct MergeArgs {
    int G;
    const dsp_shard_sums *sums;        // [G,B,L]
    const unsigned long long *keys;    // [G,B,L,K_max]
    const uint32_t *shard_status;      // [G,B]
    LatticeArgs lat;                   // sizes, parameters, outputs, tickets
};

// One warp per row: merge the slices' records and finish the row.
__global__ void __launch_bounds__(kThreads) shard_merge_kernel(const MergeArgs m) {
    const LatticeArgs &a = m.lat;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long nrows = (long long)a.B * a.L;
    const long long row = (long long)blockIdx.x * kWarps + warp;
    if (row >= nrows) return;
    const int b = (int)(row / a.L);
    // sums against the largest reference exponent, in slice order per lane, then a shuffle tree
    float cm = kRefFloor, eos_x = CUDART_NAN_F;
    for (int g = lane; g < m.G; g += 32) {
        const dsp_shard_sums r = m.sums[g * nrows + row];
        if (r.S > 0.0 || !(r.S == r.S)) cm = fmaxf(cm, r.c);          // NaN sums must stay visible
        if (r.eos_logit == r.eos_logit) eos_x = r.eos_logit;
    }
    cm = warp_max(cm);
    double S = 0.0, T = 0.0;
    for (int g = lane; g < m.G; g += 32) {
        const dsp_shard_sums r = m.sums[g * nrows + row];
        if (r.S != 0.0) {
            const double d = (double)r.c - (double)cm;
            const double w = exp2(d);
            S += w * r.S;
            T += w * (r.T + r.S * d);
        }
    }
    S = warp_sum(S);
    T = warp_sum(T);
    {   // the slice that holds EOS reported its logit (NaN everywhere else): bring it to every lane
        const unsigned has = __ballot_sync(0xFFFFFFFFu, eos_x == eos_x);
        eos_x = has ? __shfl_sync(0xFFFFFFFFu, eos_x, __ffs(has) - 1) : -CUDART_INF_F;
    }
    // best K of all slices: the sorted lists are merged one after the other (integer compares)
    unsigned long long best = 0ull;
    for (int g = 0; g < m.G; ++g) {
        const unsigned long long k = lane < a.K_max ? m.keys[(g * nrows + row) * a.K_max + lane] : 0ull;
        best = g == 0 ? k : merge_top32(best, k, lane);
    }
    unsigned st = 0;                                   // the slices' flags of this batch row (time-outs)
    for (int g = lane; g < m.G; g += 32) st |= m.shard_status[(long long)g * a.B + b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st |= __shfl_xor_sync(0xFFFFFFFFu, st, o);
    double lse, mean_x;
    const bool ok = row_log_stats(cm, S, T, lse, mean_x);
    warp_finalise_row(a, row, b, (int)(row - (long long)b * a.L), best, ok, lse, mean_x, st, lane, [&]() { return eos_x; });
}

template <typename DT>
static int32_t launch_shard(ShardArgs &a, void *workspace, size_t workspace_bytes, cudaStream_t st) {
    const long long nrows = (long long)a.B * a.L;
    const SlicePlan plan = plan_slices<DT>(nrows, a.V, slice_target_ctas());
    a.nslices = plan.nslices;
    a.slice_elems = plan.slice_elems;
    a.ntiles_row = (a.V + tile_elems<DT>() - 1) / tile_elems<DT>();
    const ShardWs w = shard_ws_layout(a.B, a.L, a.nslices);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    a.rs.row_ticket = reinterpret_cast<unsigned *>(ws + w.off_row_ticket);
    a.rs.cols = reinterpret_cast<uint2 *>(ws + w.rs.off_cols);
    a.rs.wpart = reinterpret_cast<WarpPartial *>(ws + w.rs.off_wpart);
    PrepareArgs prep = PrepareArgs();                    // row tickets and shard_status start at zero
    prep.zero_a = reinterpret_cast<uint32_t *>(ws); prep.n_a = (long long)(w.zero_bytes / 4);
    prep.zero_b = a.shard_status; prep.n_b = a.B;
    DSP_CUDA_TRY(launch_prepare(prep, st));
    const long long nblocks = nrows * a.nslices;
    if (nblocks > 0x7FFFFFFFLL) return DSP_ERR_UNSUPPORTED;
    if (a.nslices <= kMaxSlices && stream_layout_ok<DT>(a.logits, a.V, a.stride_b, a.stride_l)) {
        static RingSmemDone smem_done;                   // one per element type
        DSP_CUDA_TRY(allow_ring_smem(shard_scan_kernel<DT>, smem_done));
        a.nstages = ring_stages(nblocks);
        DSP_CUDA_TRY(launch_dependent(shard_scan_kernel<DT>, (unsigned)nblocks, kThreads, (size_t)a.nstages * kTileBytes, st, a,
                                      true));
    } else {
        shard_rows_kernel<DT><<<(unsigned)((nrows + kWarps - 1) / kWarps), kThreads, 0, st>>>(a);
    }
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

template <typename DT>
static size_t shard_ws_bytes(int B, int L, int V) {
    const SlicePlan plan = plan_slices<DT>((long long)B * L, V, slice_target_ctas());
    return shard_ws_layout(B, L, plan.nslices).total;
}

}  // namespace dsp

using namespace dsp;

static int32_t check_shard_shape(int32_t B, int32_t L, int32_t V, int32_t dtype, int32_t K_max) {
    if (B < 0 || L < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (K_max < 1 || K_max > DSP_MAX_K || L > DSP_MAX_L || V > (1 << 30)) return DSP_ERR_UNSUPPORTED;
    return DSP_OK;
}

extern "C" int32_t dsp_shard_workspace_bytes(int32_t B, int32_t L, int32_t V, int32_t dtype, int32_t K_max,
                                             size_t *bytes) {
    if (!bytes) return DSP_ERR_INVALID_ARG;
    const int32_t rc = check_shard_shape(B, L, V, dtype, K_max);
    if (rc != DSP_OK) return rc;
    const int Bq = B > 0 ? B : 1;
    *bytes = dtype == DSP_BF16 ? shard_ws_bytes<__nv_bfloat16>(Bq, L, V) : shard_ws_bytes<float>(Bq, L, V);
    return DSP_OK;
}

static int32_t shard_impl(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                          int64_t stride_b, int64_t stride_l, int32_t vocab_offset,
                          int32_t K_max, int32_t eos_id, const int32_t *path, const int32_t *path_len, int32_t Lp,
                          dsp_shard_sums *sums, uint64_t *keys, uint32_t *shard_status,
                          void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    const int32_t rc = check_shard_shape(B, L, V, dtype, K_max);
    if (rc != DSP_OK) return rc;
    if (vocab_offset < 0 || (int64_t)vocab_offset + V > (int64_t)1 << 30) return DSP_ERR_INVALID_ARG;
    if (B == 0) return DSP_OK;
    if (!logits || !sums || !keys || !shard_status || !workspace) return DSP_ERR_INVALID_ARG;
    if (stride_l < V || stride_b < 0 || (B > 1 && stride_b < (int64_t)(L - 1) * stride_l + V))
        return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(logits) & (es - 1)) != 0) return DSP_ERR_INVALID_ARG;
    ShardArgs a;
    a.logits = logits;
    a.B = B; a.L = L; a.V = V;
    a.stride_b = stride_b; a.stride_l = stride_l;
    a.vocab_offset = vocab_offset;
    a.K_max = K_max;
    a.K = K_max < V ? K_max : V;
    a.eos_id = eos_id;
    a.path = path; a.path_len = path_len; a.Lp = Lp;
    a.sums = sums;
    a.keys = reinterpret_cast<unsigned long long *>(keys);
    a.shard_status = shard_status;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    return dtype == DSP_BF16 ? launch_shard<__nv_bfloat16>(a, workspace, workspace_bytes, st)
                             : launch_shard<float>(a, workspace, workspace_bytes, st);
}

extern "C" int32_t dsp_lattice_shard(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                                     int64_t stride_b, int64_t stride_l, int32_t vocab_offset,
                                     int32_t K_max, int32_t eos_id,
                                     dsp_shard_sums *sums, uint64_t *keys, uint32_t *shard_status,
                                     void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    return shard_impl(logits, dtype, B, L, V, stride_b, stride_l, vocab_offset, K_max, eos_id, nullptr, nullptr, 0,
                      sums, keys, shard_status, workspace, workspace_bytes, stream);
}

// The target side: one key (the slice's argmax) and, as the record's probe logit, the logit of
// the row's path token if the slice holds it.
extern "C" int32_t dsp_target_shard(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t Lt, int32_t V,
                                    int64_t stride_b, int64_t stride_l, int32_t vocab_offset,
                                    const int32_t *path, const int32_t *path_len,
                                    dsp_shard_sums *sums, uint64_t *keys, uint32_t *shard_status,
                                    void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (L < 1 || Lt < L || Lt > L + 1) return DSP_ERR_INVALID_ARG;
    if (B > 0 && (!path || !path_len)) return DSP_ERR_INVALID_ARG;
    return shard_impl(logits, dtype, B, Lt, V, stride_b, stride_l, vocab_offset, 1, -1, path, path_len, L,
                      sums, keys, shard_status, workspace, workspace_bytes, stream);
}

extern "C" int32_t dsp_merge_workspace_bytes(int32_t B, size_t *bytes) {
    if (!bytes || B < 0) return DSP_ERR_INVALID_ARG;
    *bytes = 2 * align_up((size_t)(B > 0 ? B : 1) * 4, 256);
    return DSP_OK;
}

extern "C" int32_t dsp_lattice_merge(int32_t G, const dsp_shard_sums *sums, const uint64_t *keys,
                                     const uint32_t *shard_status,
                                     int32_t B, int32_t L, int32_t V, int32_t K_max, float tau, int32_t eos_id,
                                     int32_t *cand_id, float *cand_logit, float *cand_logp,
                                     int32_t *cand_count, float *lse, double *lse64, float *entropy,
                                     int32_t *gen_len, uint32_t *row_status,
                                     void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (G < 1 || B < 0 || L < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (K_max < 1 || K_max > DSP_MAX_K || L > DSP_MAX_L || V > (1 << 30) || G > 1024) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!sums || !keys || !shard_status || !cand_id || !cand_logit || !cand_logp || !cand_count || !lse64 ||
        !gen_len || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (tau != tau) return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    size_t need = 0;
    dsp_merge_workspace_bytes(B, &need);
    if (workspace_bytes < need) return DSP_ERR_WORKSPACE;
    MergeArgs m;
    m.G = G;
    m.sums = sums;
    m.keys = reinterpret_cast<const unsigned long long *>(keys);
    m.shard_status = shard_status;
    LatticeArgs &a = m.lat;
    a = LatticeArgs();
    a.B = B; a.L = L; a.V = V;
    a.K = K_max < V ? K_max : V;
    a.K_max = K_max;
    a.KC = K_max + (eos_id >= 0 ? 1 : 0);
    a.tau = tau;
    a.eos_id = eos_id;
    a.cand_id = cand_id; a.cand_logit = cand_logit; a.cand_logp = cand_logp;
    a.cand_count = cand_count; a.lse = lse; a.lse64 = lse64; a.entropy = entropy;
    a.gen_len = gen_len; a.row_status = row_status;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    PrepareArgs prep = PrepareArgs();                    // every row adds its part to row_status and gen_len
    prep.zero_a = row_status; prep.n_a = B;
    prep.fill = gen_len; prep.n_fill = B; prep.fill_value = L;
    DSP_CUDA_TRY(launch_prepare(prep, st));
    const long long nrows = (long long)B * L;
    shard_merge_kernel<<<(unsigned)((nrows + kWarps - 1) / kWarps), kThreads, 0, st>>>(m);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
