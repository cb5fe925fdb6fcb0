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
