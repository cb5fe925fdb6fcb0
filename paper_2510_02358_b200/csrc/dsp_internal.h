// Entry points shared between the translation units of the library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

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
// revealed): the per-row argmax of a chosen set of rows, used by the tree verification.
int32_t unmask_impl(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                    int64_t stride_b, int64_t stride_l, int32_t n_update,
                    int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence,
                    int32_t *n_left, uint32_t *row_status,
                    void *workspace, size_t workspace_bytes, cudaStream_t st);

// First half of the tree verifications: the argmax of every existing target row of the tree and
// the batch rows' status; workspace as dsp_verify_tree_workspace_bytes says.
int32_t tree_row_stats(const void *target_logits, int32_t dtype, int32_t B, int32_t N, int32_t V,
                       int64_t stride_b, int64_t stride_l, const int32_t *n_nodes, int32_t *tgt_argmax,
                       uint32_t *row_status, void *workspace, size_t workspace_bytes, cudaStream_t st);

}  // namespace dsp
