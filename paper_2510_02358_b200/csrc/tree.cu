// dsp_beam_tree / dsp_verify_tree: the surviving beams as one token tree, verified greedily in one
// target pass (Sec. 2 names tree-based parallel verification as verifier-side engineering; the
// paper itself verifies the rank-0 path only).
//
// dsp_beam_tree: beams that share a prefix share its nodes.  One warp per batch row, one lane per
// beam: a beam's new nodes start at the depth where it leaves every earlier beam (the longest
// prefix it has in common with one of them); counting those per beam numbers the nodes in the
// order (beam rank, depth) of their first use, so the rank-0 path is nodes 0 .. m-1.
// dsp_verify_tree: the argmax of every existing row (row 0: after the prefix, row 1+n: after node n)
// by the streaming kernels of the refinement step (rows of unused node slots are not read), then
// one warp per batch row walks from the root: the argmax of the current row picks the child that
// carries that token.
#include "dsp_common.cuh"
#include "dsp_internal.h"
#include "stream_core.cuh"

namespace dsp {

struct TreeArgs {
    const int32_t *beam_ids, *path_len;
    int B, W, L;
    int32_t *node_token, *node_parent, *node_depth, *beam_node, *n_nodes;
};

__global__ void __launch_bounds__(kThreads) beam_tree_kernel(const TreeArgs a) {
    __shared__ int s_base[kWarps][DSP_MAX_W], s_div[kWarps][DSP_MAX_W];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.x * kWarps + warp;
    if (b >= a.B) return;
    const int W = a.W, L = a.L, N = W * L;
    const int m = max(0, min(a.path_len[b], L));
    const int32_t *beams = a.beam_ids + (long long)b * W * L;
    const int32_t *mine = beams + (long long)lane * L;
    const bool live = lane < W && m > 0 && mine[0] >= 0;
    // longest prefix in common with an earlier live beam = the depth where this beam's own nodes start
    int cpl[DSP_MAX_W];
    int div = 0;
#pragma unroll 1
    for (int w = 0; w < DSP_MAX_W; ++w) {
        int c = 0;
        if (live && w < lane && beams[(long long)w * L] >= 0) {
            const int32_t *other = beams + (long long)w * L;
            while (c < m && mine[c] == other[c]) ++c;
        }
        cpl[w] = c;
        div = max(div, c);
    }
    const int fresh = live ? m - div : 0;
    int incl = fresh;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    const int base = incl - fresh;
    const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    s_base[warp][lane] = base;
    s_div[warp][lane] = div;
    __syncwarp();
    if (lane < W) {
        int prev = -1;                                   // node of this beam one depth up
        for (int i = 0; i < L; ++i) {
            int node = -1;
            if (live && i < m) {
                if (i >= div) {
                    node = base + (i - div);
                    a.node_token[(long long)b * N + node] = mine[i];
                    a.node_parent[(long long)b * N + node] = prev;
                    a.node_depth[(long long)b * N + node] = i;
                } else {
                    int w = 0;                           // the earliest beam that shares this prefix owns the node
                    while (w < DSP_MAX_W - 1 && cpl[w] <= i) ++w;
                    node = s_base[warp][w] + (i - s_div[warp][w]);
                }
            }
            a.beam_node[((long long)b * W + lane) * L + i] = node;
            prev = node;
        }
    }
    for (int n = total + lane; n < N; n += 32) {
        a.node_token[(long long)b * N + n] = -1;
        a.node_parent[(long long)b * N + n] = -1;
        a.node_depth[(long long)b * N + n] = -1;
    }
    if (lane == 0) a.n_nodes[b] = total;
}

struct WalkArgs {
    int B, N, L;
    const int32_t *node_token, *node_parent, *n_nodes;
    const int32_t *argmax;                // [B, 1+N]
    int32_t *accepted_len, *accepted_node, *next_token;
};

// Rows that exist: row 0 and the rows of the nodes.
__global__ void tree_rows_kernel(int B, int N, const int32_t *n_nodes, uint8_t *masked) {
    const long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= (long long)B * (1 + N)) return;
    const int b = (int)(x / (1 + N)), r = (int)(x - (long long)b * (1 + N));
    masked[x] = r <= min(max(n_nodes[b], 0), N) ? 1 : 0;
}

__global__ void __launch_bounds__(kThreads) tree_walk_kernel(const WalkArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.x * kWarps + warp;
    if (b >= a.B) return;
    const int N = a.N;
    const int nn = max(0, min(a.n_nodes[b], N));
    const int32_t *tok = a.node_token + (long long)b * N, *par = a.node_parent + (long long)b * N;
    int ctx = -1, acc = 0, am = 0;
    for (;;) {
        am = a.argmax[(long long)b * (1 + N) + 1 + ctx];
        int child = -1;
        for (int n0 = 0; n0 < nn && child < 0; n0 += 32) {
            const int n = n0 + lane;
            const bool hit = n < nn && par[n] == ctx && tok[n] == am;
            const unsigned bal = __ballot_sync(0xFFFFFFFFu, hit);
            if (bal) child = n0 + __ffs(bal) - 1;
        }
        if (child < 0 || acc >= a.L) break;
        if (lane == 0) a.accepted_node[(long long)b * a.L + acc] = child;
        ++acc;
        ctx = child;
    }
    for (int i = acc + lane; i < a.L; i += 32) a.accepted_node[(long long)b * a.L + i] = -1;
    if (lane == 0) {
        a.accepted_len[b] = acc;
        a.next_token[b] = am;
    }
}

TreeWs tree_ws_layout(int64_t B, int64_t rows, int V, int dtype, size_t unmask_bytes) {
    TreeWs w;
    size_t o = 0;
    w.off_masked = o;  o += align_up((size_t)(B * rows), 256);
    w.off_conf = o;    o += align_up((size_t)(B * rows) * 4, 256);
    w.off_left = o;    o += align_up((size_t)B * 4, 256);
    w.off_unmask = o;  o += align_up(unmask_bytes, 256);
    // the stochastic rule only: log-sum-exp of the target and the draft rows, scratch outputs of the
    // pass over the draft rows, chunk sums of each batch row's latest pass
    w.nchunks = (V + tree_chunk_elems(dtype) - 1) / tree_chunk_elems(dtype);
    w.off_tlse = o;    o += align_up((size_t)(B * rows) * 8, 256);
    w.off_dlse = o;    o += align_up((size_t)(B * rows) * 8, 256);
    w.off_dargmax = o; o += align_up((size_t)(B * rows) * 4, 256);
    w.off_dstatus = o; o += align_up((size_t)B * 4, 256);
    w.off_chunks = o;  o += align_up((size_t)B * w.nchunks * 8, 256);
    w.total = o;
    return w;
}

// Scratch of the row-statistics kernels for any number of rows per batch row up to N + 1 (the
// target rows are N + 1, the draft rows fewer, and fewer rows are cut into more slices).
int32_t tree_unmask_bytes(int32_t B, int32_t N, int32_t V, int32_t dtype, size_t *bytes) {
    // From one slice per row on (B * rows at least the number of CTAs wanted) the size grows with the
    // rows: only the counts below that and the largest count need a look.
    size_t most = 0;
    const long long few = slice_target_ctas() / (B > 0 ? B : 1) + 1;
    for (int32_t rows = 1; rows <= N + 1; ++rows) {
        if (rows > few && rows < N + 1) rows = N + 1;
        size_t n = 0;
        const int32_t rc = dsp_unmask_workspace_bytes(B, rows, V, dtype, &n);
        if (rc != DSP_OK) return rc;
        most = n > most ? n : most;
    }
    *bytes = most;
    return DSP_OK;
}

}  // namespace dsp

using namespace dsp;

// Argmax of every existing row of a tree's target logits (row 0 and the rows of the nodes; -1 for
// unused slots) and the batch rows' status (NaN / +inf, time-outs), by the streaming kernels of the
// refinement step: nothing is revealed (n_update = 0), so its `tokens` argument is never written.
int32_t dsp::tree_row_stats(const void *target_logits, int32_t dtype, int32_t B, int32_t N, int32_t V,
                            int64_t stride_b, int64_t stride_l, const int32_t *n_nodes, int32_t *tgt_argmax,
                            bool with_lse, uint32_t *row_status, void *workspace, size_t workspace_bytes,
                            cudaStream_t st) {
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    size_t un = 0;
    const int32_t rc = tree_unmask_bytes(B, N, V, dtype, &un);
    if (rc != DSP_OK) return rc;
    const TreeWs w = tree_ws_layout(B, N + 1, V, dtype, un);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    uint8_t *masked = ws + w.off_masked;
    float *conf = reinterpret_cast<float *>(ws + w.off_conf);
    int32_t *left = reinterpret_cast<int32_t *>(ws + w.off_left);
    const long long cells = (long long)B * (1 + N);
    tree_rows_kernel<<<(unsigned)((cells + 255) / 256), 256, 0, st>>>(B, N, n_nodes, masked);
    DSP_CUDA_TRY(cudaGetLastError());
    return unmask_impl(target_logits, dtype, B, N + 1, V, stride_b, stride_l, 0, tgt_argmax, masked, tgt_argmax, conf,
                       with_lse ? reinterpret_cast<double *>(ws + w.off_tlse) : nullptr, left, row_status,
                       ws + w.off_unmask, un, st);
}

// Log-sum-exp of the first Ld draft rows of every batch row into the workspace (NaN for a row with
// NaN / +inf or no finite logit: the walk flags the batch row if it uses such a row), by the same
// kernels; to be called after tree_row_stats, whose scratch it takes over.
int32_t dsp::tree_draft_stats(const void *draft_logits, int32_t dtype, int32_t B, int32_t N, int32_t Ld, int32_t V,
                              int64_t stride_b, int64_t stride_l, void *workspace, size_t workspace_bytes,
                              cudaStream_t st) {
    size_t un = 0;
    const int32_t rc = tree_unmask_bytes(B, N, V, dtype, &un);
    if (rc != DSP_OK) return rc;
    const TreeWs w = tree_ws_layout(B, N + 1, V, dtype, un);
    if (workspace_bytes < w.total || Ld < 1 || Ld > N + 1) return DSP_ERR_WORKSPACE;
    unsigned char *ws = static_cast<unsigned char *>(workspace);
    uint8_t *masked = ws + w.off_masked;
    DSP_CUDA_TRY(cudaMemsetAsync(masked, 1, (size_t)B * Ld, st));                  // every row is read
    int32_t *dargmax = reinterpret_cast<int32_t *>(ws + w.off_dargmax);
    return unmask_impl(draft_logits, dtype, B, Ld, V, stride_b, stride_l, 0, dargmax, masked, dargmax,
                       reinterpret_cast<float *>(ws + w.off_conf), reinterpret_cast<double *>(ws + w.off_dlse),
                       reinterpret_cast<int32_t *>(ws + w.off_left), reinterpret_cast<uint32_t *>(ws + w.off_dstatus),
                       ws + w.off_unmask, un, st);
}

extern "C" int32_t dsp_beam_tree(const int32_t *beam_ids, const int32_t *path_len, int32_t B, int32_t W, int32_t L,
                                 int32_t *node_token, int32_t *node_parent, int32_t *node_depth,
                                 int32_t *beam_node, int32_t *n_nodes, dsp_stream_t stream) {
    if (B < 0 || W < 1 || L < 1) return DSP_ERR_INVALID_ARG;
    if (W > DSP_MAX_W || L > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!beam_ids || !path_len || !node_token || !node_parent || !node_depth || !beam_node || !n_nodes)
        return DSP_ERR_INVALID_ARG;
    TreeArgs a;
    a.beam_ids = beam_ids; a.path_len = path_len;
    a.B = B; a.W = W; a.L = L;
    a.node_token = node_token; a.node_parent = node_parent; a.node_depth = node_depth;
    a.beam_node = beam_node; a.n_nodes = n_nodes;
    beam_tree_kernel<<<(unsigned)((B + kWarps - 1) / kWarps), kThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

extern "C" int32_t dsp_verify_tree_workspace_bytes(int32_t B, int32_t N, int32_t V, int32_t dtype, size_t *bytes) {
    if (!bytes || B < 0 || N < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (N + 1 > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    size_t un = 0;
    const int32_t rc = tree_unmask_bytes(B, N, V, dtype, &un);
    if (rc != DSP_OK) return rc;
    *bytes = tree_ws_layout(B > 0 ? B : 1, N + 1, V, dtype, un).total;
    return DSP_OK;
}

extern "C" int32_t dsp_verify_tree(const void *target_logits, int32_t dtype, int32_t B, int32_t N, int32_t V,
                                   int64_t stride_b, int64_t stride_l,
                                   const int32_t *node_token, const int32_t *node_parent, const int32_t *n_nodes,
                                   int32_t L, int32_t *accepted_len, int32_t *accepted_node, int32_t *next_token,
                                   int32_t *tgt_argmax, uint32_t *row_status,
                                   void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (B < 0 || N < 1 || V < 1 || L < 1) return DSP_ERR_INVALID_ARG;
    if (N + 1 > DSP_MAX_L || L > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!target_logits || !node_token || !node_parent || !n_nodes || !accepted_len || !accepted_node || !next_token ||
        !tgt_argmax || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int32_t rc = tree_row_stats(target_logits, dtype, B, N, V, stride_b, stride_l, n_nodes, tgt_argmax, false,
                                      row_status, workspace, workspace_bytes, st);
    if (rc != DSP_OK) return rc;
    WalkArgs k;
    k.B = B; k.N = N; k.L = L;
    k.node_token = node_token; k.node_parent = node_parent; k.n_nodes = n_nodes;
    k.argmax = tgt_argmax;
    k.accepted_len = accepted_len; k.accepted_node = accepted_node; k.next_token = next_token;
    tree_walk_kernel<<<(unsigned)((B + kWarps - 1) / kWarps), kThreads, 0, st>>>(k);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
