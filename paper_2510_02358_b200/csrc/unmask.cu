// dsp_unmask_step: one refinement step of the diffusion drafter on its logits (Sec. 3.1, Eq. 5,
// with the update set "top-K by confidence").
//
// For every position that is still masked the step needs the row's argmax and its probability:
// the same whole-vocabulary statistics as the lattice and the verification, with K = 1.  Rows
// whose layout is 16-byte aligned are streamed by unmask_scan_kernel (stream_core.cuh; CTAs of
// revealed rows leave at once, so a later refinement step reads only what is still masked) and
// finished by the CTA that is through with the row last (row_engine.cuh).  Any other layout is
// read element-wise by one warp per row (slower, same results).  The warp that finishes the last
// row of a batch row ranks the masked positions by confidence (counting; equal confidence: the
// lower position first), reveals the best n_update and writes what is left.
#include "dsp_internal.h"
#include "row_engine.cuh"

namespace dsp {

struct UnmaskArgs {
    const void *logits;
    int B, L, V;
    long long stride_b, stride_l;
    int n_update;
    int32_t *tokens;
    uint8_t *masked;
    int32_t *argmax;
    float *confidence;
    double *lse64;            // [B*L] or null: the rows' log-sum-exp (NaN: not computed or not finite)
    int32_t *n_left;
    uint32_t *row_status;
    int nslices, slice_elems, ntiles_row, nstages;
    // workspace
    unsigned *b_ticket;       // [B]  zeroed per call
    unsigned *b_status;       // [B]  zeroed per call
    RowScratch rs;            // records of rows cut into several slices (streaming path)
};

struct UnmaskWs {
    size_t off_b_ticket, off_b_status, off_row_ticket, zero_bytes;
    RowScratchLayout rs;
    size_t total;
};
static UnmaskWs unmask_ws_layout(int64_t B, int64_t L, int nslices) {
    UnmaskWs w;
    size_t o = 0;
    w.off_b_ticket = o;   o += align_up((size_t)B * 4, 256);
    w.off_b_status = o;   o += align_up((size_t)B * 4, 256);
    w.off_row_ticket = o; o += align_up((size_t)(B * L) * 4, 256);
    w.zero_bytes = o;
    w.rs = row_scratch_layout(o, B * L, nslices);
    w.total = w.rs.end;
    return w;
}

// Argmax (lowest id on ties), its logit and the row's log-sum-exp by one warp, element by
// element: for rows that cannot be streamed.  Returns false for NaN / +inf or no finite logit.
template <typename DT>
__device__ bool warp_row_stats_elementwise(const DT *__restrict__ row, int V, int lane, int &am, float &xmax,
                                           double &lse) {
    float m = -CUDART_INF_F;
    int id = 0x7FFFFFFF;
    bool bad = false;
    for (int v = lane; v < V; v += 32) {
        const float x = Elem<DT>::load1(row + v);
        bad |= x != x || x == CUDART_INF_F;
        if (x > m) { m = x; id = v; }                    // ascending ids: the first of equals stays
    }
    bad = __any_sync(0xFFFFFFFFu, bad);
    const float mm = warp_max(m);
    int cand = m == mm ? id : 0x7FFFFFFF;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cand = min(cand, __shfl_xor_sync(0xFFFFFFFFu, cand, o));
    am = cand == 0x7FFFFFFF ? 0 : cand;
    xmax = mm;
    if (bad || !(mm > -CUDART_INF_F)) { lse = CUDART_NAN; return false; }
    double S = 0.0;
    for (int v0 = lane; v0 < V; v0 += 32 * 64) {         // fp32 partial sums of 64 terms, added up in double
        float s = 0.f;
        for (int q = 0; q < 64; ++q) {
            const int v = v0 + q * 32;
            if (v < V) s += ex2_approx((Elem<DT>::load1(row + v) - mm) * kLog2e);
        }
        S += (double)s;
    }
    S = warp_sum(S);
    lse = (double)mm + kLn2 * log2(S);
    return true;
}

// One row is done (am / conf: its argmax and confidence, -1 / -inf for a row that was not masked);
// the warp arriving last for a batch row reveals the best n_update masked positions.  One warp.
__device__ void unmask_row_done(const UnmaskArgs &a, long long row, int b, int am, float conf, double lse, int lane) {
    if (lane == 0) {
        a.argmax[row] = am;
        a.confidence[row] = conf;
        if (a.lse64) a.lse64[row] = lse;
    }
    // ---- last row of this batch row: rank the masked positions and reveal the best ----
    __threadfence();
    __syncwarp();
    unsigned ticket = 0;
    if (lane == 0) ticket = atomicAdd(&a.b_ticket[b], 1u);
    ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
    if (ticket != (unsigned)a.L - 1) return;
    __threadfence();
    static_assert(DSP_MAX_L <= 32 * 32, "one reveal bit per position and lane");
    const long long r0 = (long long)b * a.L;
    int nmask = 0;
    for (int i0 = 0; i0 < a.L; i0 += 32) {
        const int i = i0 + lane;
        nmask += __popc(__ballot_sync(0xFFFFFFFFu, i < a.L && a.masked[r0 + i] != 0));
    }
    const int take = min(a.n_update, nmask);
    unsigned reveal = 0u;                                // bit q: this lane's q-th position is revealed
    for (int i = lane, q = 0; i < a.L; i += 32, ++q) {
        if (!a.masked[r0 + i]) continue;
        const float ci = __ldcg(&a.confidence[r0 + i]);
        int before = 0;                                  // masked positions that come first
        for (int j = 0; j < a.L; ++j) {
            const float cj = __ldcg(&a.confidence[r0 + j]);
            before += (a.masked[r0 + j] && (cj > ci || (cj == ci && j < i))) ? 1 : 0;
        }
        if (before < take) reveal |= 1u << q;
    }
    __syncwarp();                                        // every lane has read the mask: now it may change
    for (int i = lane, q = 0; i < a.L; i += 32, ++q) {
        if (reveal & (1u << q)) {
            a.tokens[r0 + i] = __ldcg(&a.argmax[r0 + i]);
            a.masked[r0 + i] = 0;
        }
    }
    if (lane == 0) {
        a.n_left[b] = nmask - take;
        a.row_status[b] = atomicOr(&a.b_status[b], 0u);
    }
}

// Streaming path: one CTA per row slice of the rows that are still masked; the CTA that is
// through with a row last takes its argmax and confidence.  A row revealed earlier is reported
// by its first CTA alone, without reading it.  (The mask changes only after every row of the
// batch row has been reported, so every CTA of a row sees the same mask.)
template <typename DT>
__global__ void __launch_bounds__(kThreads, 3) unmask_scan_kernel(const UnmaskArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ StreamBars bars;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const int lane = threadIdx.x & 31;
    if (!a.masked[row]) {                                // whole CTA alike
        grid_dependency_wait();                          // the tickets are prepared by the kernel before
        if (slice == 0 && threadIdx.x < 32) unmask_row_done(a, row, b, -1, -CUDART_INF_F, CUDART_NAN, lane);
        return;
    }
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    stream_begin(bars, a.nstages);
    RowResult r;
    if (!row_engine<DT>(rowp, a.V, 1, true, row, slice, a.nslices, a.ntiles_row, a.nstages, a.rs, &a.b_status[b], bars,
                        ring, r))
        return;
    const unsigned long long best = __shfl_sync(0xFFFFFFFFu, r.key, 0);
    const double lse = r.lse;
    const bool ok = r.stats_ok && !r.nonfinite && best != 0ull;
    const int am = best ? key_id(best) : 0;
    float conf = -CUDART_INF_F;
    if (ok) conf = (float)((double)key_value(best) - lse);
    else if (lane == 0) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    unmask_row_done(a, row, b, am, conf, ok ? lse : CUDART_NAN, lane);
}

// Layouts that cannot be streamed: one warp per row, element by element.
template <typename DT>
__global__ void __launch_bounds__(kThreads) unmask_rows_kernel(const UnmaskArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long row = (long long)blockIdx.x * kWarps + warp;
    if (row >= (long long)a.B * a.L) return;
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    int am = -1;
    float conf = -CUDART_INF_F;
    double lse_out = CUDART_NAN;
    if (a.masked[row]) {                                 // read before anyone's update: updates follow the last ticket
        float xmax = 0.f;
        double lse = 0.0;
        if (warp_row_stats_elementwise<DT>(rowp, a.V, lane, am, xmax, lse)) {
            conf = (float)((double)xmax - lse);
            lse_out = lse;
        } else if (lane == 0) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    }
    unmask_row_done(a, row, b, am, conf, lse_out, lane);
}

template <typename DT>
static int32_t launch_unmask(UnmaskArgs &a, void *workspace, size_t workspace_bytes, cudaStream_t st) {
    const long long nrows = (long long)a.B * a.L;
    const SlicePlan plan = plan_slices<DT>(nrows, a.V, slice_target_ctas());
    a.nslices = plan.nslices;
    a.slice_elems = plan.slice_elems;
    a.ntiles_row = (a.V + tile_elems<DT>() - 1) / tile_elems<DT>();
    const UnmaskWs w = unmask_ws_layout(a.B, a.L, a.nslices);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    a.b_ticket = reinterpret_cast<unsigned *>(ws + w.off_b_ticket);
    a.b_status = reinterpret_cast<unsigned *>(ws + w.off_b_status);
    a.rs.row_ticket = reinterpret_cast<unsigned *>(ws + w.off_row_ticket);
    a.rs.cols = reinterpret_cast<uint2 *>(ws + w.rs.off_cols);
    a.rs.wpart = reinterpret_cast<WarpPartial *>(ws + w.rs.off_wpart);
    PrepareArgs prep = PrepareArgs();                    // tickets and status words start at zero
    prep.zero_a = reinterpret_cast<uint32_t *>(ws); prep.n_a = (long long)(w.zero_bytes / 4);
    DSP_CUDA_TRY(launch_prepare(prep, st));
    const long long nblocks = nrows * a.nslices;
    if (nblocks > 0x7FFFFFFFLL) return DSP_ERR_UNSUPPORTED;
    if (a.nslices <= kMaxSlices && stream_layout_ok<DT>(a.logits, a.V, a.stride_b, a.stride_l)) {
        static RingSmemDone smem_done;                   // one per element type
        DSP_CUDA_TRY(allow_ring_smem(unmask_scan_kernel<DT>, smem_done));
        a.nstages = ring_stages(nblocks);
        DSP_CUDA_TRY(launch_dependent(unmask_scan_kernel<DT>, (unsigned)nblocks, kThreads, (size_t)a.nstages * kTileBytes, st, a,
                                      true));
    } else {
        unmask_rows_kernel<DT><<<(unsigned)((nrows + kWarps - 1) / kWarps), kThreads, 0, st>>>(a);
    }
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

template <typename DT>
static size_t unmask_ws_bytes(int B, int L, int V) {
    const SlicePlan plan = plan_slices<DT>((long long)B * L, V, slice_target_ctas());
    return unmask_ws_layout(B, L, plan.nslices).total;
}

}  // namespace dsp

using namespace dsp;

static int32_t check_unmask_shape(int32_t B, int32_t L, int32_t V, int32_t dtype) {
    if (B < 0 || L < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (L > DSP_MAX_L || V > (1 << 30)) return DSP_ERR_UNSUPPORTED;
    return DSP_OK;
}

extern "C" int32_t dsp_unmask_workspace_bytes(int32_t B, int32_t L, int32_t V, int32_t dtype, size_t *bytes) {
    if (!bytes) return DSP_ERR_INVALID_ARG;
    const int32_t rc = check_unmask_shape(B, L, V, dtype);
    if (rc != DSP_OK) return rc;
    const int Bq = B > 0 ? B : 1;
    *bytes = dtype == DSP_BF16 ? unmask_ws_bytes<__nv_bfloat16>(Bq, L, V) : unmask_ws_bytes<float>(Bq, L, V);
    return DSP_OK;
}

int32_t dsp::unmask_impl(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                         int64_t stride_b, int64_t stride_l, int32_t n_update,
                         int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence, double *lse64,
                         int32_t *n_left, uint32_t *row_status,
                         void *workspace, size_t workspace_bytes, cudaStream_t st) {
    const int32_t rc = check_unmask_shape(B, L, V, dtype);
    if (rc != DSP_OK) return rc;
    if (n_update < 0) return DSP_ERR_INVALID_ARG;
    if (B == 0) return DSP_OK;
    if (!logits || !tokens || !masked || !argmax || !confidence || !n_left || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (stride_l < V || stride_b < 0 || (B > 1 && stride_b < (int64_t)(L - 1) * stride_l + V))
        return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(logits) & (es - 1)) != 0) return DSP_ERR_INVALID_ARG;
    UnmaskArgs a;
    a.logits = logits;
    a.B = B; a.L = L; a.V = V;
    a.stride_b = stride_b; a.stride_l = stride_l;
    a.n_update = n_update;
    a.tokens = tokens; a.masked = masked; a.argmax = argmax; a.confidence = confidence; a.lse64 = lse64;
    a.n_left = n_left; a.row_status = row_status;
    return dtype == DSP_BF16 ? launch_unmask<__nv_bfloat16>(a, workspace, workspace_bytes, st)
                             : launch_unmask<float>(a, workspace, workspace_bytes, st);
}

extern "C" int32_t dsp_unmask_step(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                                   int64_t stride_b, int64_t stride_l, int32_t n_update,
                                   int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence,
                                   int32_t *n_left, uint32_t *row_status,
                                   void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (n_update < 1) return DSP_ERR_INVALID_ARG;
    return unmask_impl(logits, dtype, B, L, V, stride_b, stride_l, n_update, tokens, masked, argmax, confidence, nullptr,
                       n_left, row_status, workspace, workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}
