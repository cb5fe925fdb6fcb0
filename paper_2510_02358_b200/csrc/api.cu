// Host-only entry points: status strings, ABI version, and the adaptive draft-length
// controller (Sec. 3.3, Eq. 9-11; Alg. 1 init and stage 4).
#include <math.h>

#include "dsp_common.cuh"

namespace dsp {
int32_t g_last_cuda_error = 0;
ProfileEvents g_profile[2] = {{nullptr, nullptr}, {nullptr, nullptr}};
}

extern "C" int32_t dsp_profile_events(int32_t point, void *start, void *stop) {
    if (point != DSP_PROFILE_LATTICE_SCAN && point != DSP_PROFILE_TARGET_SCAN) return DSP_ERR_INVALID_ARG;
    if ((start == nullptr) != (stop == nullptr)) return DSP_ERR_INVALID_ARG;
    dsp::g_profile[point].start = reinterpret_cast<cudaEvent_t>(start);
    dsp::g_profile[point].stop = reinterpret_cast<cudaEvent_t>(stop);
    return DSP_OK;
}

// Read-only streaming probe: every thread of a CTA takes four 128-bit vectors of one 16 KB piece
// (coalesced, read-only path, lines not kept in L1) and folds them into one word that is stored
// only if it equals a value the data never produces, so the loads cannot be dropped.
namespace dsp {
constexpr int kProbeVpt = 4;
__global__ void __launch_bounds__(kThreads) read_probe_kernel(const uint4 *p, unsigned long long nvec,
                                                              uint32_t *sink) {
    const unsigned long long base = (unsigned long long)blockIdx.x * (kThreads * kProbeVpt) + threadIdx.x;
    uint4 v[kProbeVpt];
#pragma unroll
    for (int j = 0; j < kProbeVpt; ++j) {
        const unsigned long long i = base + (unsigned long long)j * kThreads;
        v[j] = i < nvec ? ldg_stream(p + i) : make_uint4(0u, 0u, 0u, 0u);
    }
    uint32_t acc = 0u;
#pragma unroll
    for (int j = 0; j < kProbeVpt; ++j) acc += (v[j].x ^ v[j].y) + (v[j].z ^ v[j].w);
    if (acc == 0x9E3779B1u && sink) *sink = acc;
}
}  // namespace dsp

extern "C" int32_t dsp_read_probe(const void *buffer, size_t bytes, uint32_t *sink, dsp_stream_t stream) {
    using namespace dsp;
    if (!buffer || !sink || bytes < 16) return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(buffer) & 15) != 0) return DSP_ERR_INVALID_ARG;
    const unsigned long long nvec = bytes / 16;
    const unsigned long long per_cta = (unsigned long long)kThreads * kProbeVpt;
    const unsigned long long nblocks = (nvec + per_cta - 1) / per_cta;
    if (nblocks > 0x7FFFFFFFull) return DSP_ERR_UNSUPPORTED;
    read_probe_kernel<<<(unsigned)nblocks, kThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4 *>(buffer), nvec, sink);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

extern "C" const char *dsp_strerror(int32_t status) {
    switch (status) {
        case DSP_OK: return "ok";
        case DSP_ERR_INVALID_ARG: return "invalid argument";
        case DSP_ERR_UNSUPPORTED: return "unsupported dtype or size beyond the compiled limits";
        case DSP_ERR_WORKSPACE: return "workspace too small";
        case DSP_ERR_CUDA: return "CUDA runtime error (see dsp_last_cuda_error)";
        case DSP_ERR_STATIC_SCRATCH: return "problem too large for the library's built-in scratch array";
        default: return "unknown status";
    }
}

extern "C" int32_t dsp_last_cuda_error(void) { return dsp::g_last_cuda_error; }

extern "C" int32_t dsp_version(void) { return 1; }

static bool adl_params_ok(const dsp_adl_params *p) {
    return p && p->k_min >= 1 && p->k_min <= p->k_max && p->rho > 0.0 && p->rho <= 1.0 &&
           p->delta >= 0.0 && p->granularity >= 1;
}

extern "C" int32_t dsp_adl_init(dsp_adl_state *state, const dsp_adl_params *params) {
    if (!state || !adl_params_ok(params)) return DSP_ERR_INVALID_ARG;
    state->ema_gen = 0.0;
    state->ema_acc = 0.0;
    state->k = params->k_max;
    state->steps = 0;
    return DSP_OK;
}

extern "C" int32_t dsp_adl_update(dsp_adl_state *state, const dsp_adl_params *params,
                                  const int32_t *accepted_len, const int32_t *gen_len, int32_t B,
                                  int32_t *next_L) {
    if (!state || !adl_params_ok(params) || !accepted_len || !gen_len || B < 1)
        return DSP_ERR_INVALID_ARG;
    long long sum_gen = 0, sum_acc = 0;
    for (int32_t b = 0; b < B; ++b) {
        sum_gen += gen_len[b];
        sum_acc += accepted_len[b];
    }
    const double rho = params->rho;
    state->ema_gen = (1.0 - rho) * state->ema_gen + rho * ((double)sum_gen / (double)B);
    state->ema_acc = (1.0 - rho) * state->ema_acc + rho * ((double)sum_acc / (double)B);
    const double grow = state->ema_acc >= state->ema_gen ? params->delta : 0.0;
    long long k = (long long)ceil(state->ema_gen + grow);
    const long long g = params->granularity;
    if (g > 1) k = (k + g - 1) / g * g;
    if (k < params->k_min) k = params->k_min;
    if (k > params->k_max) k = params->k_max;
    state->k = (int32_t)k;
    state->steps += 1;
    if (next_L) *next_L = state->k;
    return DSP_OK;
}

// ---- breadth controller (host): candidate cap from the drafter's perplexity, beam width from
// the acceptance shortfall, both through moving averages of Eq. 10's form ----
static bool breadth_params_ok(const dsp_breadth_params *p) {
    return p && p->K_min >= 1 && p->K_min <= p->K_max && p->K_max <= DSP_MAX_K && p->W_min >= 1 &&
           p->W_min <= p->W_max && p->W_max <= DSP_MAX_W && p->rho > 0.0 && p->rho <= 1.0;
}

extern "C" int32_t dsp_breadth_init(dsp_breadth_state *state, const dsp_breadth_params *params) {
    if (!state || !breadth_params_ok(params)) return DSP_ERR_INVALID_ARG;
    state->ema_entropy = 0.0;
    state->ema_shortfall = 0.0;
    state->K = params->K_max;
    state->W = params->W_max;
    state->steps = 0;
    return DSP_OK;
}

extern "C" int32_t dsp_breadth_update(dsp_breadth_state *state, const dsp_breadth_params *params,
                                      const float *entropy, const int32_t *accepted_len, const int32_t *gen_len,
                                      int32_t B, int32_t L, int32_t *next_K, int32_t *next_W) {
    if (!state || !breadth_params_ok(params) || !entropy || !accepted_len || !gen_len || B < 1 || L < 1)
        return DSP_ERR_INVALID_ARG;
    double h_sum = 0.0, s_sum = 0.0;
    long long positions = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int32_t g = gen_len[b];
        const int32_t take = g < 1 ? 1 : (g > L ? L : g);           // drafted positions of this row
        const float *row = entropy + (size_t)b * L;
        for (int32_t i = 0; i < take; ++i) h_sum += (double)row[i];
        positions += take;
        const int32_t cut = g > accepted_len[b] ? g - accepted_len[b] : 0;
        s_sum += (double)cut / (double)(g < 1 ? 1 : g);
    }
    const double rho = params->rho;
    state->ema_entropy = (1.0 - rho) * state->ema_entropy + rho * (h_sum / (double)positions);
    state->ema_shortfall = (1.0 - rho) * state->ema_shortfall + rho * (s_sum / (double)B);
    double k = ceil(exp(state->ema_entropy));
    double w = ceil((double)params->W_min + (double)(params->W_max - params->W_min) * state->ema_shortfall);
    k = k < params->K_min ? params->K_min : (k > params->K_max ? params->K_max : k);
    w = w < params->W_min ? params->W_min : (w > params->W_max ? params->W_max : w);
    state->K = (int32_t)k;
    state->W = (int32_t)w;
    state->steps += 1;
    if (next_K) *next_K = state->K;
    if (next_W) *next_W = state->W;
    return DSP_OK;
}
