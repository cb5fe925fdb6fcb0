// What the finish of a lattice row needs, shared by the kernels that finish rows: the lattice
// build's own pass 2 (lattice.cu) and the merge of vocabulary shards (shard.cu).
#pragma once

#include "row_warp.cuh"

namespace dsp {

struct LatticeArgs {
    const void *logits;
    int B, L, V;
    long long stride_b, stride_l;
    int K;          // min(K_max, V)
    int K_max, KC;
    float tau;
    int eos_id;
    int nslices, slice_elems;
    int32_t *cand_id;
    float *cand_logit, *cand_logp;
    int32_t *cand_count;
    float *lse;
    double *lse64;
    float *entropy;
    int32_t *gen_len;
    uint32_t *row_status;
    // workspace
    unsigned *row_ticket;     // [B*L]   zeroed per call
    unsigned *b_ticket;       // [B]     zeroed per call
    unsigned *b_status;       // [B]     zeroed per call
    SlicePartial *partials;   // [B*L, nslices]               (element-wise path)
    unsigned long long *keys; // [B*L, nslices, K]            (element-wise path)
    WarpPartial *wpart;       // [B*L, nslices, kWarps]       (streaming path)
    void *table;              // [B*L, ntiles_row + nslices, kThreads]  (streaming path), element type of the logits
    int ntiles_row;           // tiles of a whole row
};

// Finish one row by one warp from its best keys (`key`: one per lane, descending, 0 = none; the
// first min(K, #finite) count) and its whole-row sums (c, S, T): log-sum-exp, entropy, Eq. 7
// count, EOS slot (`eos_logit()` fetches the row's EOS logit when it is needed), candidate
// outputs; the warp that finishes the last row of a batch row also writes gen_len (Eq. 9) and
// row_status.
template <typename EosLogit>
__device__ __forceinline__ void warp_finalise_row(const LatticeArgs &a, long long row, int b, unsigned long long key,
                                                  float c, double S, double T, int lane, EosLogit eos_logit) {
    const int nk = __popc(__ballot_sync(0xFFFFFFFFu, key != 0ull && lane < a.K));

    double lse, mean_x;
    const bool ok = row_log_stats(c, S, T, lse, mean_x) && nk > 0;
    int count = nk;
    if (a.tau > 0.f && a.tau <= 1.f && ok) {           // Eq. 7 on full-vocabulary probabilities
        const double p = lane < nk ? exp((double)key_value(key) - lse) : 0.0;
        const double tau = (double)a.tau;
        double cum = 0.0;
        bool found = false;
        for (int k = 0; k < nk; ++k) {                 // in rank order, every lane alike
            cum += __shfl_sync(0xFFFFFFFFu, p, k);
            if (!found && cum >= tau) { count = k + 1; found = true; }
        }
    }
    int eos_slot = -1;
    float eos_x = 0.f;
    if (a.eos_id >= 0 && a.eos_id < a.V) {              // always keep EOS
        const bool has = __ballot_sync(0xFFFFFFFFu, lane < count && key_id(key) == a.eos_id) != 0u;
        if (!has) {
            eos_x = eos_logit();
            if (eos_x > -CUDART_INF_F && eos_x < CUDART_INF_F) eos_slot = count;
        }
    }
    if (lane == 0) {
        a.cand_count[row] = count + (eos_slot >= 0 ? 1 : 0);
        if (a.lse) a.lse[row] = (float)lse;
        a.lse64[row] = lse;
        if (a.entropy) a.entropy[row] = (float)(lse - mean_x);
        if (!ok) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    }
    for (int slot = lane; slot < a.KC; slot += 32) {      // slot 32 can only be the EOS slot
        const unsigned long long ks = key;                  // slot == lane whenever slot < count <= 32
        int id = -1;
        float x = -CUDART_INF_F, lp = -CUDART_INF_F;
        if (slot < count) {
            id = key_id(ks);
            x = key_value(ks);
            lp = (float)((double)x - lse);
        } else if (slot == eos_slot) {
            id = a.eos_id;
            x = eos_x;
            lp = (float)((double)x - lse);
        }
        const long long o = row * a.KC + slot;
        a.cand_id[o] = id;
        a.cand_logit[o] = x;
        a.cand_logp[o] = lp;
    }
    // ---- last row of this batch row: generation length (Eq. 9) and status ----
    __threadfence();
    __syncwarp();
    unsigned ticket = 0;
    if (lane == 0) ticket = atomicAdd(&a.b_ticket[b], 1u);
    ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
    if (ticket != (unsigned)a.L - 1) return;
    __threadfence();
    int g = a.L;
    if (a.eos_id >= 0) {
        for (int i0 = 0; i0 < a.L && g == a.L; i0 += 32) {
            const int i = i0 + lane;
            const bool eos = i < a.L && __ldcg(&a.cand_id[((long long)b * a.L + i) * a.KC]) == a.eos_id;
            const unsigned m = __ballot_sync(0xFFFFFFFFu, eos);
            if (m) g = i0 + __ffs(m) - 1;
        }
    }
    if (lane == 0) {
        a.gen_len[b] = g;
        a.row_status[b] = atomicOr(&a.b_status[b], 0u);
    }
}

}  // namespace dsp
