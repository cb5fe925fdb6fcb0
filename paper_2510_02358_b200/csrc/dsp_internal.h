// Entry points shared between the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "dsp.h"

namespace dsp {

// The two parts of dsp_verify: the target statistics need only the target logits (and mode);
// the decisions also need the chosen path.
constexpr int kVerifyStats = 1;
constexpr int kVerifyDecide = 2;

// dsp_verify with a choice of parts (same arguments, checks and errors).
int32_t verify_impl(const void *target_logits, int32_t dtype, int32_t B, int32_t L, int32_t Lt, int32_t V,
                    int64_t tstride_b, int64_t tstride_l, const void *draft_logits, int64_t dstride_b,
                    int64_t dstride_l, const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                    const float *cand_logit, const double *draft_lse64, int32_t KC, int32_t all_greedy,
                    const uint8_t *mode, const float *u, int32_t eos_id, int32_t *accepted_len,
                    int32_t *next_token, float *ratio, int32_t *tgt_argmax, float *tgt_lse,
                    uint32_t *row_status, void *workspace, size_t workspace_bytes, cudaStream_t st, int phases);

// dsp_lattice_build on a CUDA stream (same arguments, checks and errors).
int32_t lattice_build_impl(const void *draft_logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                           int64_t stride_b, int64_t stride_l, int32_t K_max, float tau, int32_t eos_id,
                           int32_t *cand_id, float *cand_logit, float *cand_logp, int32_t *cand_count,
                           float *lse, double *lse64, float *entropy, int32_t *gen_len, uint32_t *row_status,
                           void *workspace, size_t workspace_bytes, cudaStream_t st);

// dsp_cps_search on a CUDA stream (same arguments, checks and errors).
int32_t cps_search_impl(const int32_t *cand_id, const float *cand_logit, const double *lse64,
                        const int32_t *cand_count, int32_t B, int32_t L, int32_t KC, const int32_t *prev_token,
                        int32_t proxy_kind, const float *proxy_table, int32_t table_log2, uint32_t hash_seed,
                        int32_t V, int32_t W, float lambda, int32_t eos_id, const float *ver_score, float mu,
                        int32_t *path, int32_t *path_slot,
                        int32_t *path_len, float *path_score, int32_t *beam_ids, float *beam_score,
                        float *beam_cum, uint32_t *row_status, cudaStream_t stream);

// dsp_unmask_step that also takes n_update = 0 (row statistics of the masked rows only, nothing
// revealed): the per-row argmax of a chosen set of rows, used by the tree verification; lse64
// (may be null) takes the rows' log-sum-exp in double (NaN: row not read, or not finite).
int32_t unmask_impl(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                    int64_t stride_b, int64_t stride_l, int32_t n_update,
                    int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence, double *lse64,
                    int32_t *n_left, uint32_t *row_status,
                    void *workspace, size_t workspace_bytes, cudaStream_t st);

// First half of the tree verifications: the argmax of every existing target row of the tree and
// the batch rows' status; workspace as dsp_verify_tree_workspace_bytes says.
// (with_lse: also their log-sum-exp, into the workspace at off_tlse).
int32_t tree_row_stats(const void *target_logits, int32_t dtype, int32_t B, int32_t N, int32_t V,
                       int64_t stride_b, int64_t stride_l, const int32_t *n_nodes, int32_t *tgt_argmax,
                       bool with_lse, uint32_t *row_status, void *workspace, size_t workspace_bytes,
                       cudaStream_t st);
int32_t tree_draft_stats(const void *draft_logits, int32_t dtype, int32_t B, int32_t N, int32_t Ld, int32_t V,
                         int64_t stride_b, int64_t stride_l, void *workspace, size_t workspace_bytes,
                         cudaStream_t st);
// Layout of that workspace (rows = N + 1 target rows per batch row).
struct TreeWs {
    size_t off_masked, off_conf, off_left, off_unmask, off_tlse, off_dlse, off_dargmax, off_dstatus, off_chunks, total;
    int nchunks;               // chunks of a row: one warp-wide 16-byte vector load each
};
inline int tree_chunk_elems(int dtype) { return dtype == DSP_BF16 ? 256 : 128; }
TreeWs tree_ws_layout(int64_t B, int64_t rows, int V, int dtype, size_t unmask_bytes);
int32_t tree_unmask_bytes(int32_t B, int32_t N, int32_t V, int32_t dtype, size_t *bytes);

}  // namespace dsp
