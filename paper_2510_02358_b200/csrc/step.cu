// dsp_draft_verify_step: one whole draft-and-verify step (Alg. 1 stages 1-3 on logits) in one call.
//
// Same kernels and results as dsp_lattice_build, dsp_cps_search and dsp_verify called one after
// the other.  What the single call adds is overlap: the statistics of the target rows (argmax,
// log-sum-exp) need only the target logits, so the pass over the target logits runs beside the
// pass over the draft logits and the path search; the decisions (acceptance scan, residual draw)
// wait for both sides.  The two sides run on the caller's stream and on a stream of the library.
// When the passes are long (their grid is several times what the SMs hold at once) the library's
// stream, which has the highest priority the device offers, takes the build and the search: the
// two passes then run back to back without a gap or a drained last wave between them, and the
// search's few CTAs get the next free places on the SMs instead of queueing behind the target
// pass's grid.
#include <mutex>

#include "stream_core.cuh"
#include "dsp_internal.h"

namespace {

constexpr int kMaxDevices = 64;
// Target logits from which the pass over them counts as long: its grid is then several times
// what the SMs hold at once, and a kernel launched behind it waits for most of the pass.
constexpr long long kLongPassBytes = 400ll << 20;
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};
std::mutex g_side_mutex;
SideStream g_side[kMaxDevices];

// The second stream and its two events, created at the first call on each device.  The caller holds
// g_side_mutex.
int32_t side_stream(SideStream **out) {
    int dev = -1;
    DSP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DSP_ERR_UNSUPPORTED;
    SideStream &s = g_side[dev];
    if (!s.stream) {
        int least = 0, greatest = 0;                     // numerically lower = higher priority
        DSP_CUDA_TRY(cudaDeviceGetStreamPriorityRange(&least, &greatest));
        DSP_CUDA_TRY(cudaStreamCreateWithPriority(&s.stream, cudaStreamNonBlocking, greatest));
        DSP_CUDA_TRY(cudaEventCreateWithFlags(&s.fork, cudaEventDisableTiming));
        DSP_CUDA_TRY(cudaEventCreateWithFlags(&s.join, cudaEventDisableTiming));
    }
    *out = &s;
    return DSP_OK;
}

}  // namespace

extern "C" int32_t dsp_draft_verify_step(
    const void *draft_logits, const void *target_logits, int32_t dtype,
    int32_t B, int32_t L, int32_t Lt, int32_t V,
    int64_t dstride_b, int64_t dstride_l, int64_t tstride_b, int64_t tstride_l,
    int32_t K_max, float tau, int32_t eos_id,
    const int32_t *prev_token, int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
    uint32_t hash_seed, int32_t W, float lambda,
    int32_t all_greedy, const uint8_t *mode, const float *u,
    int32_t *cand_id, float *cand_logit, float *cand_logp, int32_t *cand_count,
    float *lse, double *lse64, float *entropy, int32_t *gen_len,
    int32_t *path, int32_t *path_slot, int32_t *path_len, float *path_score,
    int32_t *beam_ids, float *beam_score, float *beam_cum,
    int32_t *accepted_len, int32_t *next_token, float *ratio, int32_t *tgt_argmax, float *tgt_lse,
    uint32_t *row_status,
    void *lattice_workspace, size_t lattice_workspace_bytes,
    void *verify_workspace, size_t verify_workspace_bytes, dsp_stream_t stream) {
    using namespace dsp;
    if (B == 0) return DSP_OK;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int32_t KC = K_max + (eos_id >= 0 ? 1 : 0);
    // One call at a time enqueues on the second stream and its fork / join events: calls from
    // several host threads (or for several caller streams) then each see their own fork point.
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SideStream *side = nullptr;
    int32_t rc = side_stream(&side);
    if (rc != DSP_OK) return rc;

    const long long target_bytes = (long long)B * Lt * V * (dtype == DSP_BF16 ? 2 : 4);
    const bool long_pass = target_bytes >= kLongPassBytes;
    auto stats = [&](cudaStream_t s) {
        return verify_impl(target_logits, dtype, B, L, Lt, V, tstride_b, tstride_l, draft_logits, dstride_b,
                           dstride_l, path, path_slot, path_len, cand_logit, lse64, KC, all_greedy, mode, u, eos_id,
                           accepted_len, next_token, ratio, tgt_argmax, tgt_lse, row_status, verify_workspace,
                           verify_workspace_bytes, s, kVerifyStats);
    };
    auto search = [&](cudaStream_t s) {
        return cps_search_impl(cand_id, cand_logit, lse64, cand_count, B, L, KC, prev_token, proxy_kind,
                               proxy_table, table_log2, hash_seed, V, W, lambda, eos_id, nullptr, 0.f, path, path_slot,
                               path_len, path_score, beam_ids, beam_score, beam_cum, row_status, s);
    };
    int32_t rc2 = DSP_OK;
    // The two sides start together: the second stream takes up where the caller's stream stands.
    DSP_CUDA_TRY(cudaEventRecord(side->fork, st));
    DSP_CUDA_TRY(cudaStreamWaitEvent(side->stream, side->fork, 0));
    // Long passes: the build and the search go to the second stream, whose priority hands its CTAs
    // out first: the draft logits stream first, the target pass's CTAs fill the places the draft
    // pass's last wave leaves free, and the search gets in ahead of the target pass's grid.
    // Short passes leave SMs free anyway: the build and the search stay on the caller's stream
    // (no event on their way) and the target statistics take the second stream.
    cudaStream_t draft_side = long_pass ? side->stream : st;
    cudaStream_t target_side = long_pass ? st : side->stream;
    rc = lattice_build_impl(draft_logits, dtype, B, L, V, dstride_b, dstride_l, K_max, tau, eos_id, cand_id,
                            cand_logit, cand_logp, cand_count, lse, lse64, entropy, gen_len, row_status,
                            lattice_workspace, lattice_workspace_bytes, draft_side);
    if (rc == DSP_OK) rc = stats(target_side);
    if (rc == DSP_OK) rc2 = search(draft_side);
    // whatever happened, the caller's stream joins the second stream again
    cudaError_t e = cudaEventRecord(side->join, side->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, side->join, 0);
    if (rc != DSP_OK) return rc;
    if (e != cudaSuccess) return cuda_fail(e);
    if (rc2 != DSP_OK) return rc2;
    // stage 3's decisions once both sides are there
    return verify_impl(target_logits, dtype, B, L, Lt, V, tstride_b, tstride_l, draft_logits, dstride_b, dstride_l,
                       path, path_slot, path_len, cand_logit, lse64, KC, all_greedy, mode, u, eos_id, accepted_len,
                       next_token, ratio, tgt_argmax, tgt_lse, row_status, verify_workspace,
                       verify_workspace_bytes, st, kVerifyDecide);
}
