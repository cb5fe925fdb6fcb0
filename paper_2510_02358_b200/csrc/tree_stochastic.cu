// dsp_verify_tree_stochastic: stochastic verification of a token tree (Sec. 2: Eq. 1 and residual
// resampling, in the multi-branch form that tree-based verification takes: the siblings of a node
// are tried one after the other, every rejection replaces the target distribution by the
// normalised residual before the next sibling is tried).
//
// Everything that is the same for all walks runs first, in parallel over the rows, on the streaming
// kernels of the refinement step: argmax, NaN / +inf check and log-sum-exp of every existing target
// row, log-sum-exp of the draft rows.  The walk itself is sequential per batch row: one CTA of 1024
// threads per batch row follows it.  An acceptance test is a few double-precision operations on two
// logits; only a rejection costs a pass over the two rows (the mass R of the residual [f - q]_+,
// 16-byte loads, fp32 terms, sums in double in a fixed order).  After j rejections at a node the
// current distribution is
//   f_j(v) = max(0, f_{j-1}(v) - q(v)) / R_j,   f_0 = softmax(target row),  q = softmax(draft row).
// Each pass leaves the sums of its chunks (one warp-wide vector load each) in the workspace; the
// unnormalised terms of the last pass are the current distribution times R, so the emitted token
// is found from those sums (prefix over the chunks, then one chunk read again) without another
// pass, unless nothing was rejected at the last node (one pass over the target row then).
#include "dsp_common.cuh"
#include "dsp_internal.h"
#include "scan_core.cuh"

namespace dsp {

constexpr int kTreeThreads = 1024;
constexpr int kTreeWarps = kTreeThreads / 32;

struct TreeStochArgs {
    const void *target, *draft;
    int B, N, L, V;
    long long tstride_b, tstride_l, dstride_b, dstride_l;
    const int32_t *node_token, *node_parent, *n_nodes;
    const int32_t *argmax;                // [B, 1+N] of the existing rows
    const double *tlse, *dlse;            // [B, 1+N]: target rows; [B, Ld]: draft rows (NaN: unusable)
    int Ld;
    double *chunks;                       // [B, nchunks]
    int nchunks;
    const float *u;                       // [B, N+1]
    int32_t *accepted_len, *accepted_node, *next_token;
    uint32_t *row_status;
};

struct TreeStochSmem {
    double red[kTreeWarps];
    double scan[kTreeThreads];
    double R[DSP_MAX_W + 1];              // residual masses of the rejections at the current node
    float invR[DSP_MAX_W + 1];
    int child, found;
};

// Sum of one double per thread over the CTA, in a fixed order; every thread gets it.
__device__ double tree_block_sum(double v, TreeStochSmem &sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    v = __shfl_sync(0xFFFFFFFFu, v, 0);
    __syncthreads();                                    // the scratch may still be read from the last call
    if (lane == 0) sm.red[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kTreeWarps; ++w) t += sm.red[w];
    return t;
}

// The current distribution at one token after `nrej` rejections, in double (the acceptance test).
__device__ __forceinline__ double dist_after(float xt, float xd, double lse_t, double lse_d, const double *R, int nrej) {
    double f = exp((double)xt - lse_t);
    if (nrej > 0) {
        const double q = exp((double)xd - lse_d);
        for (int j = 0; j < nrej; ++j) {
            f -= q;
            f = f > 0.0 ? f / R[j] : 0.0;
        }
    }
    return f;
}
// The same in fp32 for the passes over whole rows: the term whose sum is the next residual mass
// (`last`: stop before the division, i.e. [f_{nrej-1} - q]_+ for nrej > 0, f_0 for nrej = 0).
__device__ __forceinline__ float term_after(float xt, float xd, const RowProb &pt, const RowProb &pd, const float *invR,
                                            int nrej) {
    float f = prob(xt, pt);
    if (nrej > 0) {
        const float q = prob(xd, pd);
        for (int j = 0; j + 1 < nrej; ++j) {
            f = __fsub_rn(f, q);
            f = f > 0.f ? __fmul_rn(f, invR[j]) : 0.f;
        }
        f = __fsub_rn(f, q);
        f = f > 0.f ? f : 0.f;                          // NaN -> 0
    }
    return f;
}

// One pass: the chunk sums of the terms after `nrej` rejections (nrej = 0: of the target row's own
// distribution) into `sums`, their total to every thread.
template <typename DT>
__device__ double tree_pass(const DT *__restrict__ trow, const DT *__restrict__ drow, int V, int nchunks, bool aligned,
                            const RowProb &pt, const RowProb &pd, int nrej, double *sums, TreeStochSmem &sm) {
    constexpr int N = Elem<DT>::N;
    constexpr int CE = 32 * N;
    constexpr int kBatch = 2;                           // chunks whose loads a warp has in flight together
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double mine = 0.0;                                  // lane 0: the sums of this warp's chunks
    for (int ch0 = warp; ch0 < nchunks; ch0 += kTreeWarps * kBatch) {
        uint4 vt[kBatch], vd[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int ch = ch0 + b * kTreeWarps;
            if (ch < nchunks) {
                vt[b] = load_vec<DT>(trow, ch * CE + lane * N, V, aligned);
                vd[b] = nrej > 0 ? load_vec<DT>(drow, ch * CE + lane * N, V, aligned) : vt[b];
            }
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
            const int ch = ch0 + b * kTreeWarps;
            if (ch < nchunks) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < N; ++e)
                    s = __fadd_rn(s, term_after(Elem<DT>::get(vt[b], e), Elem<DT>::get(vd[b], e), pt, pd, sm.invR, nrej));
                const double cs = warp_sum((double)s);
                if (lane == 0) { sums[ch] = cs; mine += cs; }
            }
        }
    }
    return tree_block_sum(lane == 0 ? mine : 0.0, sm);
}

// One CTA per batch row.
template <typename DT>
__global__ void __launch_bounds__(kTreeThreads, 1) tree_stochastic_kernel(const TreeStochArgs a) {
    constexpr int NE = Elem<DT>::N;
    constexpr int CE = 32 * NE;
    __shared__ TreeStochSmem sm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const int N = a.N, L = a.L, V = a.V;
    const int nn = max(0, min(a.n_nodes[b], N));
    const int32_t *tok = a.node_token + (long long)b * N, *par = a.node_parent + (long long)b * N;
    const DT *tbase = reinterpret_cast<const DT *>(a.target) + (long long)b * a.tstride_b;
    const DT *dbase = reinterpret_cast<const DT *>(a.draft) + (long long)b * a.dstride_b;
    double *sums = a.chunks + (long long)b * a.nchunks;
    unsigned status = 0u;
    int ctx = -1, acc = 0, token = -1;
    for (int i = tid; i < L; i += kTreeThreads) a.accepted_node[(long long)b * L + i] = -1;

    for (;;) {                                          // one round per node the walk stands on
        const DT *trow = tbase + (long long)(1 + ctx) * a.tstride_l;
        const double lse_t = a.tlse[(long long)b * (1 + N) + 1 + ctx];     // NaN: the batch row is flagged already
        const DT *drow = trow;
        double lse_d = 0.0;
        bool have_q = false;
        int nrej = 0, after = -1;
        bool moved = false, dead = false;
        RowProb pt = row_prob(lse_t), pd = pt;
        bool aligned = false;
        while (acc < L && nrej < DSP_MAX_W) {
            // the next child of ctx in node order
            __syncthreads();
            if (tid == 0) sm.child = 0x7FFFFFFF;
            __syncthreads();
            for (int n = after + 1 + tid; n < nn; n += kTreeThreads)
                if (par[n] == ctx) { atomicMin(&sm.child, n); break; }
            __syncthreads();
            const int n = sm.child;
            if (n == 0x7FFFFFFF) break;
            after = n;
            if (!have_q) {
                drow = dbase + (long long)acc * a.dstride_l;
                lse_d = acc < a.Ld ? a.dlse[(long long)b * a.Ld + acc] : CUDART_NAN;
                if (!(lse_d == lse_d)) status |= DSP_ROW_NONFINITE_INPUT;
                pd = row_prob(lse_d);
                aligned = ((reinterpret_cast<uintptr_t>(trow) | reinterpret_cast<uintptr_t>(drow)) & 15) == 0;
                have_q = true;
            }
            const int x = min(max(tok[n], 0), V - 1);
            const float xt = Elem<DT>::load1(trow + x), xd = Elem<DT>::load1(drow + x);
            const double fx = dist_after(xt, xd, lse_t, lse_d, sm.R, nrej);
            const double qx = exp((double)xd - lse_d);
            const bool ok = qx > 0.0 ? (double)a.u[(long long)b * (N + 1) + n] < fx / qx : fx > 0.0;
            if (ok) {
                if (tid == 0) a.accepted_node[(long long)b * L + acc] = n;
                ++acc;
                ctx = n;
                moved = true;
                break;
            }
            // rejected: the mass of the residual [f - q]_+ is the next normaliser
            const double Rn = tree_pass<DT>(trow, drow, V, a.nchunks, aligned, pt, pd, nrej + 1, sums, sm);
            if (!(Rn > 0.0)) { dead = true; break; }
            __syncthreads();
            if (tid == 0) { sm.R[nrej] = Rn; sm.invR[nrej] = (float)(1.0 / Rn); }
            __syncthreads();
            ++nrej;
        }
        if (moved) continue;
        if (dead) {
            token = a.argmax[(long long)b * (1 + N) + 1 + ctx];
            status |= DSP_ROW_ZERO_RESIDUAL;
            break;
        }
        // The emitted token: inverse CDF of the current distribution in token order.  Its terms times
        // the last residual mass are what the last pass summed; with no rejection here, one pass now.
        double total;
        if (nrej > 0) {
            total = sm.R[nrej - 1];
        } else {
            aligned = (reinterpret_cast<uintptr_t>(trow) & 15) == 0;
            total = tree_pass<DT>(trow, trow, V, a.nchunks, aligned, pt, pt, 0, sums, sm);
        }
        if (!(total > 0.0)) {
            token = a.argmax[(long long)b * (1 + N) + 1 + ctx];
            status |= DSP_ROW_ZERO_RESIDUAL;
            break;
        }
        __threadfence_block();
        __syncthreads();                                // the chunk sums are written (by lanes 0 of this CTA)
        const double thr = (double)a.u[(long long)b * (N + 1) + N] * total;
        // exclusive prefix over the chunks: consecutive chunks per thread, then over the threads in a fixed order
        const int per = (a.nchunks + kTreeThreads - 1) / kTreeThreads;
        const int k0 = min(a.nchunks, tid * per), k1 = min(a.nchunks, k0 + per);
        double mine = 0.0;
        for (int k = k0; k < k1; ++k) mine += sums[k];
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sm.red[warp] = incl;
        if (tid == 0) sm.found = 0x7FFFFFFF;
        __syncthreads();
        double wbase = 0.0;
        for (int w = 0; w < warp; ++w) wbase += sm.red[w];
        {
            // the first chunk at which the running sum reaches the threshold; its finder leaves the sum before it
            double run = wbase + (incl - mine);
            for (int k = k0; k < k1; ++k) {
                const double cs = sums[k];
                if (cs > 0.0 && run + cs >= thr) {
                    atomicMin(&sm.found, k);
                    sm.scan[tid] = run;
                    break;
                }
                run += cs;
            }
        }
        __syncthreads();
        int ch = sm.found;
        const bool at_top = ch == 0x7FFFFFFF;
        if (at_top) {                                   // rounding at the very top: last chunk with mass
            __syncthreads();
            if (tid == 0) {
                int last = -1;
                for (int k = a.nchunks - 1; k >= 0; --k)
                    if (sums[k] > 0.0) { last = k; break; }
                sm.found = last;
            }
            __syncthreads();
            ch = sm.found;
        }
        if (ch < 0) {                                   // cannot be (total > 0), kept in bounds all the same
            token = a.argmax[(long long)b * (1 + N) + 1 + ctx];
            break;
        }
        if (warp == 0) {
            const double before = at_top ? -CUDART_INF : sm.scan[min(kTreeThreads - 1, ch / per)];
            const int e0 = ch * CE + lane * NE;
            const uint4 vt = load_vec<DT>(trow, e0, V, aligned);
            const uint4 vd = nrej > 0 ? load_vec<DT>(drow, e0, V, aligned) : vt;
            float r[NE];
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                r[e] = term_after(Elem<DT>::get(vt, e), Elem<DT>::get(vd, e), pt, pd, sm.invR, nrej);
                s = __fadd_rn(s, r[e]);
            }
            double li = (double)s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xFFFFFFFFu, li, o);
                if (lane >= o) li += up;
            }
            double run = before + (li - (double)s);
            int hit = -1, lastpos = -1;
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                run += (double)r[e];
                if (r[e] > 0.f && e0 + e < V) {
                    lastpos = e0 + e;
                    if (hit < 0 && run >= thr) hit = e0 + e;
                }
            }
            const unsigned bal = __ballot_sync(0xFFFFFFFFu, hit >= 0);
            int t;
            if (bal) {
                t = __shfl_sync(0xFFFFFFFFu, hit, __ffs(bal) - 1);
            } else {
                const unsigned bl = __ballot_sync(0xFFFFFFFFu, lastpos >= 0);
                t = bl ? __shfl_sync(0xFFFFFFFFu, lastpos, 31 - __clz(bl)) : a.argmax[(long long)b * (1 + N) + 1 + ctx];
            }
            if (lane == 0) sm.child = t;
        }
        __syncthreads();
        token = sm.child;
        break;
    }
    if (tid == 0) {
        a.accepted_len[b] = acc;
        a.next_token[b] = token;
        if (status) atomicOr(&a.row_status[b], status);
    }
}

}  // namespace dsp

using namespace dsp;

extern "C" int32_t dsp_verify_tree_stochastic(const void *target_logits, const void *draft_logits, int32_t dtype,
                                              int32_t B, int32_t N, int32_t L, int32_t V,
                                              int64_t tstride_b, int64_t tstride_l, int64_t dstride_b, int64_t dstride_l,
                                              const int32_t *node_token, const int32_t *node_parent,
                                              const int32_t *n_nodes, const float *u,
                                              int32_t *accepted_len, int32_t *accepted_node, int32_t *next_token,
                                              int32_t *tgt_argmax, uint32_t *row_status,
                                              void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (B < 0 || N < 1 || V < 1 || L < 1) return DSP_ERR_INVALID_ARG;
    if (N + 1 > DSP_MAX_L || L > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!target_logits || !draft_logits || !node_token || !node_parent || !n_nodes || !u || !accepted_len ||
        !accepted_node || !next_token || !tgt_argmax || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (tstride_l < V || dstride_l < V || tstride_b < 0 || dstride_b < 0) return DSP_ERR_INVALID_ARG;
    if (B > 1 && (tstride_b < (int64_t)N * tstride_l + V || dstride_b < (int64_t)(L - 1) * dstride_l + V))
        return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if (((reinterpret_cast<uintptr_t>(target_logits) | reinterpret_cast<uintptr_t>(draft_logits)) & (es - 1)) != 0)
        return DSP_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int32_t rc = tree_row_stats(target_logits, dtype, B, N, V, tstride_b, tstride_l, n_nodes, tgt_argmax, true, row_status,
                                workspace, workspace_bytes, st);
    if (rc != DSP_OK) return rc;
    const int32_t Ld = L < N + 1 ? L : N + 1;           // the walk stands at depth acc <= number of nodes
    rc = tree_draft_stats(draft_logits, dtype, B, N, Ld, V, dstride_b, dstride_l, workspace, workspace_bytes, st);
    if (rc != DSP_OK) return rc;
    size_t un = 0;
    rc = tree_unmask_bytes(B, N, V, dtype, &un);
    if (rc != DSP_OK) return rc;
    const TreeWs w = tree_ws_layout(B, N + 1, V, dtype, un);
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    TreeStochArgs a;
    a.tlse = reinterpret_cast<const double *>(ws + w.off_tlse);
    a.dlse = reinterpret_cast<const double *>(ws + w.off_dlse);
    a.Ld = Ld;
    a.chunks = reinterpret_cast<double *>(ws + w.off_chunks);
    a.nchunks = w.nchunks;
    a.target = target_logits; a.draft = draft_logits;
    a.B = B; a.N = N; a.L = L; a.V = V;
    a.tstride_b = tstride_b; a.tstride_l = tstride_l; a.dstride_b = dstride_b; a.dstride_l = dstride_l;
    a.node_token = node_token; a.node_parent = node_parent; a.n_nodes = n_nodes;
    a.argmax = tgt_argmax; a.u = u;
    a.accepted_len = accepted_len; a.accepted_node = accepted_node; a.next_token = next_token;
    a.row_status = row_status;
    if (dtype == DSP_BF16) tree_stochastic_kernel<__nv_bfloat16><<<(unsigned)B, kTreeThreads, 0, st>>>(a);
    else                   tree_stochastic_kernel<float><<<(unsigned)B, kTreeThreads, 0, st>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
