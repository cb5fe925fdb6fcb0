// What the finish of a lattice row needs, shared by the kernels that finish rows: the lattice
// build's streaming kernel (lattice.cu) and the merge of vocabulary shards (shard.cu).
#pragma once

#include "row_engine.cuh"

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
    RowScratch rs;            // records of rows cut into several slices (streaming path)
    int ntiles_row;           // tiles of a whole row
    int nstages;              // ring depth of the streaming kernel
};

// Finish one row by one warp from its best keys (`key`: one per lane, descending, 0 = none; the
// first min(K, #finite) count) and its log-sum-exp and mean logit (`stats_ok` false: the sums do
// not describe a finite row): entropy, Eq. 7 count, EOS slot (`eos_logit()` fetches the row's EOS
// logit when it is needed), candidate outputs.  The batch row's outputs take part of every row:
// status flags (`flags` and DSP_ROW_NONFINITE_INPUT) are OR-ed into row_status[b] and a row whose
// best token is EOS lowers gen_len[b] to its position (Eq. 9); both were prepared before the
// kernel (row_status 0, gen_len L), so no row waits for another.
template <typename EosLogit>
__device__ __forceinline__ void warp_finalise_row(const LatticeArgs &a, long long row, int b, int l,
                                                  unsigned long long key, bool stats_ok, double lse, double mean_x,
                                                  unsigned flags, int lane, EosLogit eos_logit) {
    const int nk = __popc(__ballot_sync(0xFFFFFFFFu, key != 0ull && lane < a.K));
    const bool ok = stats_ok && nk > 0;
    int count = nk;
    if (a.tau > 0.f && a.tau <= 1.f && ok) {           // Eq. 7 on full-vocabulary probabilities
        double cum = lane < nk ? exp((double)key_value(key) - lse) : 0.0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {             // cumulative mass in rank order
            const double up = __shfl_up_sync(0xFFFFFFFFu, cum, o);
            if (lane >= o) cum += up;
        }
        const unsigned reached = __ballot_sync(0xFFFFFFFFu, lane < nk && cum >= (double)a.tau);
        if (reached) count = __ffs(reached);
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
        const unsigned fl = flags | (ok ? 0u : (unsigned)DSP_ROW_NONFINITE_INPUT);
        if (fl) atomicOr(&a.row_status[b], fl);
        if (a.eos_id >= 0 && nk > 0 && key_id(key) == a.eos_id) atomicMin(&a.gen_len[b], l);   // Eq. 9
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
}

}  // namespace dsp
