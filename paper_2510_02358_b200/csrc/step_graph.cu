// dsp_step_graph_*: dsp_draft_verify_step recorded once as a CUDA graph and replayed.
//
// A step on a short draft is seven short kernels and two memsets on two streams; replaying them
// as one graph takes the host's launch work (and the event traffic between the two streams) out
// of every step.  The draft length changes from step to step (Sec. 3.3, Eq. 11), but only over a
// few values: the caller records one graph per draft length it uses and replays the one the
// controller asks for.  A graph holds the addresses and sizes it was recorded with; the caller
// refreshes the inputs in place.
#include <new>

#include "dsp_common.cuh"
#include "dsp_internal.h"

struct dsp_step_graph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
};

extern "C" int32_t dsp_step_graph_create(
    dsp_step_graph **out,
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
    void *verify_workspace, size_t verify_workspace_bytes) {
    using namespace dsp;
    if (!out) return DSP_ERR_INVALID_ARG;
    *out = nullptr;
    // events set through dsp_profile_events would be recorded into the graph and lost to the caller
    for (int p = 0; p < 2; ++p)
        if (g_profile[p].start || g_profile[p].stop) return DSP_ERR_UNSUPPORTED;

    cudaStream_t cs = nullptr;
    DSP_CUDA_TRY(cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking));
    cudaError_t e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeRelaxed);
    if (e != cudaSuccess) {
        cudaStreamDestroy(cs);
        return cuda_fail(e);
    }
    const int32_t rc = dsp_draft_verify_step(
        draft_logits, target_logits, dtype, B, L, Lt, V, dstride_b, dstride_l, tstride_b, tstride_l, K_max, tau,
        eos_id, prev_token, proxy_kind, proxy_table, table_log2, hash_seed, W, lambda, all_greedy, mode, u,
        cand_id, cand_logit, cand_logp, cand_count, lse, lse64, entropy, gen_len, path, path_slot, path_len,
        path_score, beam_ids, beam_score, beam_cum, accepted_len, next_token, ratio, tgt_argmax, tgt_lse,
        row_status, lattice_workspace, lattice_workspace_bytes, verify_workspace, verify_workspace_bytes, cs);
    cudaGraph_t graph = nullptr;
    e = cudaStreamEndCapture(cs, &graph);            // always: the stream must leave capture mode
    cudaStreamDestroy(cs);
    if (rc != DSP_OK || e != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        if (rc != DSP_OK) {
            (void)cudaGetLastError();                // an argument error: nothing of CUDA's to report
            return rc;
        }
        return cuda_fail(e);
    }
    cudaGraphExec_t exec = nullptr;
    // the kernels recorded from the step's second stream keep that stream's priority in the replay
    e = cudaGraphInstantiateWithFlags(&exec, graph, cudaGraphInstantiateFlagUseNodePriority);
    if (e != cudaSuccess) {
        cudaGraphDestroy(graph);
        return cuda_fail(e);
    }
    dsp_step_graph *g = new (std::nothrow) dsp_step_graph;
    if (!g) {
        cudaGraphExecDestroy(exec);
        cudaGraphDestroy(graph);
        return DSP_ERR_CUDA;
    }
    g->graph = graph;
    g->exec = exec;
    *out = g;
    return DSP_OK;
}

extern "C" int32_t dsp_step_graph_launch(dsp_step_graph *g, dsp_stream_t stream) {
    using namespace dsp;
    if (!g || !g->exec) return DSP_ERR_INVALID_ARG;
    DSP_CUDA_TRY(cudaGraphLaunch(g->exec, reinterpret_cast<cudaStream_t>(stream)));
    return DSP_OK;
}

extern "C" int32_t dsp_step_graph_destroy(dsp_step_graph *g) {
    using namespace dsp;
    if (!g) return DSP_OK;
    cudaError_t e1 = g->exec ? cudaGraphExecDestroy(g->exec) : cudaSuccess;
    cudaError_t e2 = g->graph ? cudaGraphDestroy(g->graph) : cudaSuccess;
    delete g;
    if (e1 != cudaSuccess) return cuda_fail(e1);
    if (e2 != cudaSuccess) return cuda_fail(e2);
    return DSP_OK;
}
