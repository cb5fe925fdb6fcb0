// dsp_verify_tree_stochastic: stochastic verification of a token tree (Sec. 2: Eq. 1 and residual
// resampling, in the multi-branch form that tree-based verification takes: the siblings of a node
// are tried one after the other, every rejection replaces the target distribution by the
// normalised residual before the next sibling is tried).
//
// The statistics of all existing target rows (argmax, NaN / +inf check) come from the streaming
// kernels of the refinement step, as in dsp_verify_tree.  The walk is sequential per batch row:
// one CTA per batch row follows it and makes every pass over a row that the walk asks for
// (log-sum-exp of a visited row, the residual mass after a rejection, the inverse CDF of the
// emitted token) with all its threads, in double precision and in a fixed order of summation.
// After j rejections at a node the current distribution is
//   f_j(v) = max(0, f_{j-1}(v) - q(v)) / R_j,   f_0 = softmax(target row),  q = softmax(draft row),
// which every thread evaluates from the two logits and the masses R_1 .. R_j kept so far.
#include "dsp_common.cuh"
#include "dsp_internal.h"

namespace dsp {

struct TreeStochArgs {
    const void *target, *draft;
    int B, N, L, V;
    long long tstride_b, tstride_l, dstride_b, dstride_l;
    const int32_t *node_token, *node_parent, *n_nodes;
    const int32_t *argmax;                // [B, 1+N] of the existing rows
    const float *u;                       // [B, N+1]
    int32_t *accepted_len, *accepted_node, *next_token;
    uint32_t *row_status;
};

struct TreeStochSmem {
    double red[kWarps];
    double R[DSP_MAX_W + 1];              // residual masses of the rejections at the current node
    double bcast;
    float fbcast;
    int ibcast;
    int found, lastpos, child;
    int bad;
};

// Sum of one double per thread over the CTA, in a fixed order; every thread gets it.
__device__ double block_sum(double v, TreeStochSmem &sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();                                    // the scratch may still be read from the last call
    if (lane == 0) sm.red[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += sm.red[w];
    return t;
}

// Log-sum-exp of a row by the CTA (two passes: largest finite logit, then the sum in double);
// `bad` is set for NaN / +inf or a row without a finite logit.
template <typename DT>
__device__ double block_lse(const DT *__restrict__ row, int V, TreeStochSmem &sm, bool &bad) {
    float m = -CUDART_INF_F;
    bool b = false;
    for (int v = threadIdx.x; v < V; v += kThreads) {
        const float x = Elem<DT>::load1(row + v);
        b |= x != x || x == CUDART_INF_F;
        if (x > m && x < CUDART_INF_F) m = x;
    }
    m = warp_max(m);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sm.red[threadIdx.x >> 5] = (double)m;
    if (threadIdx.x == 0) sm.bad = 0;
    __syncthreads();
    if (b) sm.bad = 1;
    double mm = sm.red[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) mm = sm.red[w] > mm ? sm.red[w] : mm;
    double s = 0.0;
    if (mm > -CUDART_INF)
        for (int v = threadIdx.x; v < V; v += kThreads) {
            const float x = Elem<DT>::load1(row + v);
            if (x > -CUDART_INF_F && x < CUDART_INF_F) s += exp((double)x - mm);
        }
    const double S = block_sum(s, sm);                  // its barriers also publish sm.bad
    bad = sm.bad != 0 || !(mm > -CUDART_INF);
    return bad ? CUDART_NAN : mm + log(S);
}

// The current distribution at token v after `nrej` rejections at this node (xt, xd: the two logits).
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

// One CTA per batch row.
template <typename DT>
__global__ void __launch_bounds__(kThreads) tree_stochastic_kernel(const TreeStochArgs a) {
    __shared__ TreeStochSmem sm;
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    const int N = a.N, L = a.L, V = a.V;
    const int nn = max(0, min(a.n_nodes[b], N));
    const int32_t *tok = a.node_token + (long long)b * N, *par = a.node_parent + (long long)b * N;
    const DT *tbase = reinterpret_cast<const DT *>(a.target) + (long long)b * a.tstride_b;
    const DT *dbase = reinterpret_cast<const DT *>(a.draft) + (long long)b * a.dstride_b;
    unsigned status = 0u;
    int ctx = -1, acc = 0, token = -1;
    for (int i = tid; i < L; i += kThreads) a.accepted_node[(long long)b * L + i] = -1;

    for (;;) {                                          // one round per node the walk stands on
        const DT *trow = tbase + (long long)(1 + ctx) * a.tstride_l;
        bool tbad;                                      // the batch row is flagged by the pass over all existing rows
        const double lse_t = block_lse<DT>(trow, V, sm, tbad);
        const DT *drow = dbase;
        double lse_d = 0.0;
        bool have_q = false;
        int nrej = 0, after = -1;
        bool moved = false, dead = false;
        while (acc < L && nrej < DSP_MAX_W) {
            // the next child of ctx in node order
            __syncthreads();
            if (tid == 0) sm.child = 0x7FFFFFFF;
            __syncthreads();
            for (int n = after + 1 + tid; n < nn; n += kThreads)
                if (par[n] == ctx) { atomicMin(&sm.child, n); break; }
            __syncthreads();
            const int n = sm.child;
            if (n == 0x7FFFFFFF) break;
            after = n;
            if (!have_q) {
                drow = dbase + (long long)acc * a.dstride_l;
                bool dbad;
                lse_d = block_lse<DT>(drow, V, sm, dbad);
                if (dbad) status |= DSP_ROW_NONFINITE_INPUT;
                have_q = true;
            }
            const int x = min(max(tok[n], 0), V - 1);
            const double fx = dist_after(Elem<DT>::load1(trow + x), Elem<DT>::load1(drow + x), lse_t, lse_d, sm.R, nrej);
            const double qx = exp((double)Elem<DT>::load1(drow + x) - lse_d);
            const bool ok = qx > 0.0 ? (double)a.u[(long long)b * (N + 1) + n] < fx / qx : fx > 0.0;
            if (ok) {
                if (tid == 0) a.accepted_node[(long long)b * L + acc] = n;
                ++acc;
                ctx = n;
                moved = true;
                break;
            }
            // rejected: the mass of the residual [f - q]_+ is the next normaliser
            double r = 0.0;
            for (int v = tid; v < V; v += kThreads) {
                const float xd = Elem<DT>::load1(drow + v);
                const double d = dist_after(Elem<DT>::load1(trow + v), xd, lse_t, lse_d, sm.R, nrej) - exp((double)xd - lse_d);
                r += d > 0.0 ? d : 0.0;
            }
            const double Rn = block_sum(r, sm);
            if (!(Rn > 0.0)) { dead = true; break; }
            __syncthreads();
            if (tid == 0) sm.R[nrej] = Rn;
            __syncthreads();
            ++nrej;
        }
        if (moved) continue;
        if (dead) {
            token = a.argmax[(long long)b * (1 + N) + 1 + ctx];
            status |= DSP_ROW_ZERO_RESIDUAL;
            break;
        }
        // the emitted token: inverse CDF of the current distribution in token order
        double s = 0.0;
        for (int v = tid; v < V; v += kThreads)
            s += dist_after(Elem<DT>::load1(trow + v), have_q ? Elem<DT>::load1(drow + v) : 0.f, lse_t, lse_d, sm.R, nrej);
        const double total = block_sum(s, sm);
        if (!(total > 0.0)) {
            token = a.argmax[(long long)b * (1 + N) + 1 + ctx];
            status |= DSP_ROW_ZERO_RESIDUAL;
            break;
        }
        const double thr = (double)a.u[(long long)b * (N + 1) + N] * total;
        __syncthreads();
        if (tid == 0) { sm.found = 0x7FFFFFFF; sm.lastpos = -1; }
        __syncthreads();
        constexpr int E = 4;                              // consecutive tokens per thread and round
        double carry = 0.0;                               // mass of everything before this round
        for (int base = 0; base < V; base += kThreads * E) {
            double f[E];
            double mine = 0.0;
            const int v0 = base + tid * E;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const int v = v0 + e;
                f[e] = v < V ? dist_after(Elem<DT>::load1(trow + v), have_q ? Elem<DT>::load1(drow + v) : 0.f, lse_t, lse_d,
                                          sm.R, nrej)
                             : 0.0;
                mine += f[e];
            }
            // exclusive prefix of the threads' masses: inside the warp, then over the warps
            const int lane = tid & 31, warp = tid >> 5;
            double incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += up;
            }
            __syncthreads();
            if (lane == 31) sm.red[warp] = incl;
            __syncthreads();
            double before = carry, round_total = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                if (w < warp) before += sm.red[w];
                round_total += sm.red[w];
            }
            double run = before + (incl - mine);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                run += f[e];
                if (f[e] > 0.0 && v0 + e < V) {
                    atomicMax(&sm.lastpos, v0 + e);
                    if (run >= thr) { atomicMin(&sm.found, v0 + e); break; }
                }
            }
            carry += round_total;
            __syncthreads();
            if (sm.found != 0x7FFFFFFF) break;
        }
        __syncthreads();
        token = sm.found != 0x7FFFFFFF ? sm.found : sm.lastpos;   // rounding at the very top of the CDF
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
    const int32_t rc = tree_row_stats(target_logits, dtype, B, N, V, tstride_b, tstride_l, n_nodes, tgt_argmax, row_status,
                                      workspace, workspace_bytes, st);
    if (rc != DSP_OK) return rc;
    TreeStochArgs a;
    a.target = target_logits; a.draft = draft_logits;
    a.B = B; a.N = N; a.L = L; a.V = V;
    a.tstride_b = tstride_b; a.tstride_l = tstride_l; a.dstride_b = dstride_b; a.dstride_l = dstride_l;
    a.node_token = node_token; a.node_parent = node_parent; a.n_nodes = n_nodes;
    a.argmax = tgt_argmax; a.u = u;
    a.accepted_len = accepted_len; a.accepted_node = accepted_node; a.next_token = next_token;
    a.row_status = row_status;
    if (dtype == DSP_BF16) tree_stochastic_kernel<__nv_bfloat16><<<(unsigned)B, kThreads, 0, st>>>(a);
    else                   tree_stochastic_kernel<float><<<(unsigned)B, kThreads, 0, st>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
