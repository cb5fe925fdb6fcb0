/*
 * dsp_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, scalar CPU statement of what one draft-and-verify step of
 * DiffuSpec computes on logits: token lattice, causal-consistency path search
 * (CPS), verification, adaptive draft length (ADL).  Every function follows
 * the definition it cites, one loop per definition, double precision unless
 * the step says otherwise.  Nothing here is tuned, blocked or fused.
 *
 * This file shares no code, header, table or constant with the CUDA library.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Parity pins: every function below is pinned by CPU tests against closed
 * forms, library routines, brute force or hand-built cases (see the pin list
 * in the test files named test_oracle_*).  The paper prints no worked numeric
 * example, so no value is pinned to a printed figure; end-to-end accepted
 * length on real models is "parity unpinned" (needs the models).
 *
 * Conventions: positions and ranks are 0-based here (the paper is 1-based).
 * dtype 0 = IEEE fp32 logits, dtype 1 = bfloat16 logits given as raw 16-bit
 * words.  All tensors are dense, row-major, last dimension contiguous.
 * Threads (OpenMP) split batch rows only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_NONFINITE_INPUT 1u
#define ORC_ZERO_RESIDUAL   2u
#define ORC_NO_BONUS_ROW    4u
#define ORC_EOS_ACCEPTED    8u
#define ORC_EOS_STOPPED     16u

/* Exact value of logit number idx as a double. */
static double logit_at(const void *base, int dtype, int64_t idx)
{
    if (dtype == 0)
        return (double)((const float *)base)[idx];
    uint32_t w = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* The total order on (logit, token id): larger logit first, then lower id. */
static int better(double xa, int64_t ia, double xb, int64_t ib)
{
    if (xa > xb) return 1;
    if (xa < xb) return 0;
    return ia < ib;
}

/*
 * Row statistics over a whole vocabulary row (Sec. 3.2: l^dlm = log q, the
 * log-softmax; "entropy-adaptive" names the Shannon entropy, taken in nats).
 *   m = max x,  Z = sum exp(x-m),  lse = m + log Z,
 *   H = lse - (sum x exp(x-m)) / Z, terms with x = -inf contributing 0.
 * Returns 0, or 1 if the row holds NaN / +inf or no finite logit.
 */
static int row_stats(const void *row, int dtype, int64_t V, double *lse, double *H,
                     int64_t *argmax)
{
    double m = -INFINITY;
    int64_t am = 0;
    int bad = 0;
    for (int64_t v = 0; v < V; ++v) {
        double x = logit_at(row, dtype, v);
        if (isnan(x) || x == INFINITY) bad = 1;
        if (x > m) { m = x; am = v; }        /* strict: lowest id wins ties */
    }
    if (argmax) *argmax = am;
    if (bad || m == -INFINITY) {
        if (lse) *lse = NAN;
        if (H) *H = NAN;
        return 1;
    }
    double Z = 0.0, T = 0.0;
    for (int64_t v = 0; v < V; ++v) {
        double x = logit_at(row, dtype, v);
        if (x == -INFINITY) continue;
        double e = exp(x - m);
        Z += e;
        T += x * e;
    }
    if (lse) *lse = m + log(Z);
    if (H) *H = (m + log(Z)) - T / Z;
    return 0;
}

/* Exported for pins: statistics of one row. */
int orc_row_stats(const void *row, int dtype, int64_t V, double *lse, double *entropy,
                  int64_t *argmax)
{
    return row_stats(row, dtype, V, lse, entropy, argmax);
}

/*
 * Token lattice (Sec. 3.2, "Lattice and pruning"; Alg. 1 stage 1-2).
 * Per row (b,l):
 *   - top-K candidates under the order (logit desc, id asc), K = min(K_max, V);
 *     candidates whose logit is -inf are not kept (at least one is);
 *   - cand_logp = x - lse, the full-vocabulary log-probability;
 *   - Eq. 7: count = smallest m <= K whose cumulative full-vocabulary mass
 *     reaches tau; K if none does; pruning is off unless 0 < tau <= 1;
 *   - "always keep EOS": if eos_id >= 0, EOS is not among the kept ones and its
 *     logit is finite, it takes one extra slot after them;
 *   - Eq. 9: gen_len[b] = number of positions before the first whose top-1 is
 *     EOS (L if there is none).
 * Arrays: cand_* are [B,L,KC], KC = K_max + (eos_id >= 0); unused slots hold
 * id -1, logit -inf, logp -inf.
 */
int orc_lattice_build(const void *draft, int dtype, int B, int L, int64_t V,
                      int K_max, double tau, int eos_id,
                      int32_t *cand_id, float *cand_logit, float *cand_logp,
                      int32_t *cand_count, float *lse32, double *lse64, float *entropy,
                      int32_t *gen_len, uint32_t *row_status)
{
    if (B < 0 || L < 1 || V < 1 || K_max < 1) return -1;
    const int KC = K_max + (eos_id >= 0 ? 1 : 0);
    const int K = (int64_t)K_max < V ? K_max : (int)V;

#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        uint32_t status = 0;
        double *kx = (double *)malloc(sizeof(double) * (size_t)K);
        int64_t *ki = (int64_t *)malloc(sizeof(int64_t) * (size_t)K);
        int first_eos = -1;
        for (int l = 0; l < L; ++l) {
            const int64_t r = (int64_t)b * L + l;
            const char *row = (const char *)draft + (size_t)r * (size_t)V * (dtype ? 2 : 4);
            double lse, H;
            int bad = row_stats(row, dtype, V, &lse, &H, NULL);
            if (bad) status |= ORC_NONFINITE_INPUT;
            lse32[r] = (float)lse;
            lse64[r] = lse;
            entropy[r] = (float)H;

            /* top-K by insertion into a list kept sorted under the order */
            int n = 0;
            for (int64_t v = 0; v < V; ++v) {
                double x = logit_at(row, dtype, v);
                if (isnan(x)) continue;
                if (n == K && !better(x, v, kx[K - 1], ki[K - 1])) continue;
                int p = n < K ? n : K - 1;
                while (p > 0 && better(x, v, kx[p - 1], ki[p - 1])) {
                    kx[p] = kx[p - 1];
                    ki[p] = ki[p - 1];
                    --p;
                }
                kx[p] = x;
                ki[p] = v;
                if (n < K) ++n;
            }
            /* drop -inf candidates, keep at least one */
            int kept = 0;
            while (kept < n && kx[kept] > -INFINITY) ++kept;
            if (kept == 0) kept = n > 0 ? 1 : 0;

            /* Eq. 7 on full-vocabulary probabilities, cumulative in rank order */
            int count = kept;
            if (tau > 0.0 && tau <= 1.0 && !bad) {
                double cum = 0.0;
                for (int k = 0; k < kept; ++k) {
                    cum += exp(kx[k] - lse);
                    if (cum >= tau) { count = k + 1; break; }
                }
            }
            int32_t *cid = cand_id + r * KC;
            float *clg = cand_logit + r * KC;
            float *clp = cand_logp + r * KC;
            for (int k = 0; k < KC; ++k) {
                cid[k] = -1;
                clg[k] = -INFINITY;
                clp[k] = -INFINITY;
            }
            int has_eos = 0;
            for (int k = 0; k < count; ++k) {
                cid[k] = (int32_t)ki[k];
                clg[k] = (float)kx[k];
                clp[k] = (float)(kx[k] - lse);
                if (eos_id >= 0 && ki[k] == eos_id) has_eos = 1;
            }
            if (eos_id >= 0 && eos_id < V && !has_eos) {
                double xe = logit_at(row, dtype, eos_id);
                if (xe > -INFINITY && !isnan(xe)) {
                    cid[count] = eos_id;
                    clg[count] = (float)xe;
                    clp[count] = (float)(xe - lse);
                    ++count;
                }
            }
            cand_count[r] = count;
            if (first_eos < 0 && eos_id >= 0 && n > 0 && ki[0] == eos_id) first_eos = l;
        }
        gen_len[b] = first_eos < 0 ? L : first_eos;
        row_status[b] = status;
        free(kx);
        free(ki);
    }
    return 0;
}

/*
 * Causal proxy l^ng(prev, cur) (Sec. 3.2: "a small causal proxy, e.g. an
 * n-gram"); here a bigram table supplied by the caller.
 *   kind 0: hashed table of 2^table_log2 floats.  All arithmetic on uint32
 *           modulo 2^32:  h = prev * 0x9E3779B1;  h ^= cur + seed;
 *           h *= 0x9E3779B1;  h ^= h >> 15;  h *= 0x9E3779B1;  h ^= h >> 13;
 *           index = h >> (32 - table_log2).
 *   kind 1: dense [V,V] table, index = prev * V + cur.
 */
static float proxy_score(int kind, const float *table, int table_log2, uint32_t seed,
                         int64_t V, int32_t prev, int32_t cur)
{
    if (kind == 1)
        return table[(int64_t)prev * V + cur];
    uint32_t h = (uint32_t)prev * 0x9E3779B1u;
    h ^= (uint32_t)cur + seed;
    h *= 0x9E3779B1u;
    h ^= h >> 15;
    h *= 0x9E3779B1u;
    h ^= h >> 13;
    uint32_t idx = table_log2 >= 32 ? h : (table_log2 <= 0 ? 0u : h >> (32 - table_log2));
    return table[idx];
}

float orc_proxy_score(int kind, const float *table, int table_log2, uint32_t seed,
                      int64_t V, int32_t prev, int32_t cur)
{
    return proxy_score(kind, table, table_log2, seed, V, prev, cur);
}

/*
 * Hashed trigram proxy (the paper's causal proxy is a 3-gram model, Sec. 4):
 * l^ng(cur | prev2, prev) = table[mix3(prev2, prev, cur) >> (32 - table_log2)],
 *   g = prev2 * 0xC2B2AE35;  g ^= g >> 16;
 *   h = (prev ^ g) * 0x9E3779B1;  h ^= cur + seed;  h *= 0x9E3779B1;
 *   h ^= h >> 15;  h *= 0x9E3779B1;  h ^= h >> 13          (all in uint32).
 */
static float trigram_score(const float *table, int table_log2, uint32_t seed,
                           int32_t prev2, int32_t prev, int32_t cur)
{
    uint32_t g = (uint32_t)prev2 * 0xC2B2AE35u;
    g ^= g >> 16;
    uint32_t h = ((uint32_t)prev ^ g) * 0x9E3779B1u;
    h ^= (uint32_t)cur + seed;
    h *= 0x9E3779B1u;
    h ^= h >> 15;
    h *= 0x9E3779B1u;
    h ^= h >> 13;
    uint32_t idx = table_log2 >= 32 ? h : (table_log2 <= 0 ? 0u : h >> (32 - table_log2));
    return table[idx];
}

float orc_trigram_score(const float *table, int table_log2, uint32_t seed,
                        int32_t prev2, int32_t prev, int32_t cur)
{
    return trigram_score(table, table_log2, seed, prev2, prev, cur);
}

/*
 * l^ng of candidate slot k at position i of batch row b, for a path whose
 * earlier tokens / slots are ids[0..i) / slots[0..i)  (Eq. 8's causal term):
 *   kind 0, 1: bigram on (previous token, token): hashed table or dense [V,V];
 *              position 0 conditions on prev_token[b];
 *   kind 2   : a tensor [B,L,KC,KC] of scores the caller computed (a small
 *              causal model): entry [b][i][p][k], p = the previous position's
 *              slot (row p = 0 at position 0);
 *   kind 3   : hashed trigram on (token before, previous token, token);
 *              prev_token is [B,2] (oldest first) and supplies what the path
 *              does not have yet.
 */
static float proxy_at(int kind, const float *table, int table_log2, uint32_t seed, int64_t V,
                      const int32_t *prev_token, int b, int L, int KC, int i, int k, int32_t tok,
                      const int32_t *ids, const int32_t *slots)
{
    if (kind == 2) {
        const int p = i == 0 ? 0 : slots[i - 1];
        return table[(((int64_t)b * L + i) * KC + p) * KC + k];
    }
    if (kind == 3) {
        const int32_t prev = i == 0 ? prev_token[2 * b + 1] : ids[i - 1];
        const int32_t prev2 = i == 0 ? prev_token[2 * b] : (i == 1 ? prev_token[2 * b + 1] : ids[i - 2]);
        return trigram_score(table, table_log2, seed, prev2, prev, tok);
    }
    const int32_t prev = i == 0 ? prev_token[b] : ids[i - 1];
    return proxy_score(kind, table, table_log2, seed, V, prev, tok);
}

typedef struct {
    float cum;
    int32_t tok;
    int32_t parent;
    int32_t slot;
} expansion;

/* (cum desc, token id asc, parent rank asc) */
static int exp_before(const expansion *a, const expansion *b)
{
    if (a->cum > b->cum) return 1;
    if (a->cum < b->cum) return 0;
    if (a->tok != b->tok) return a->tok < b->tok;
    return a->parent < b->parent;
}

/*
 * Causal-consistency path search (Sec. 3.2 "Scoring and search", Eq. 8,
 * Alg. 1 stage 2): left-to-right beam of width W over the lattice.
 *
 * Ranking quantity.  All live beams have the same depth, so Eq. 8's term
 * lambda * sum_i (lse_i - x_top1,i) is the same for all of them; beams are
 * ranked on  cum = sum_i [ lambda * (x_i - x_top1,i) + (1-lambda) * l^ng_i ]
 * evaluated in fp32 in this exact order:
 *   g = fp32(x - x_top1);  step = fp32( fp32(lambda*g) + fp32((1-lambda)*n) );
 *   cum = fp32(parent_cum + step),   1-lambda = fp32(1 - lambda).
 * l^ng comes from one of four proxies (see proxy_at above).
 * Survivors: the best min(W, #expansions) under (cum desc, token id asc,
 * parent rank asc).  The search stops after the depth at which the rank-0
 * survivor's new token is EOS (early stop at the first EOS placed).
 *
 * Outputs: path[B,L] (rank-0 tokens, -1 padded), path_slot[B,L] (their
 * candidate slots), path_len[B], path_score[B] = Eq. 8 of the rank-0 path in
 * double from cand_logit - lse64, beam_ids[B,W,L], beam_score[B,W] (Eq. 8 per
 * beam, -inf where no beam), beam_cum[B,W] (the fp32 ranking quantity).
 * beam_* may be NULL.
 *
 * Verifier-aware scoring (Sec. 6, future work ii, names it without a rule; the reading taken):
 * a third term mu * l^ver in Eq. 8, with l^ver a per-candidate log-score from the verifier's
 * side that the caller supplies slot by slot, ver_score[B,L,KC] (NULL or mu = 0: Eq. 8 as it is):
 *   step = fp32( fp32( fp32(lambda*g) + fp32((1-lambda)*n) ) + fp32(mu * v) ).
 */
int orc_cps_search_biased(const int32_t *cand_id, const float *cand_logit, const double *lse64,
                   const int32_t *cand_count, int B, int L, int KC,
                   const int32_t *prev_token, int proxy_kind, const float *table,
                   int table_log2, uint32_t hash_seed, int64_t V,
                   int W, float lambda, int eos_id, const float *ver_score, float mu,
                   int32_t *path, int32_t *path_slot, int32_t *path_len, float *path_score,
                   int32_t *beam_ids, float *beam_score, float *beam_cum,
                   uint32_t *row_status)
{
    if (B < 0 || L < 1 || KC < 1 || W < 1) return -1;
    const float oml = 1.0f - lambda;

#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)W * L);
        int32_t *slots = (int32_t *)malloc(sizeof(int32_t) * (size_t)W * L);
        int32_t *nids = (int32_t *)malloc(sizeof(int32_t) * (size_t)W * L);
        int32_t *nslots = (int32_t *)malloc(sizeof(int32_t) * (size_t)W * L);
        float *cum = (float *)malloc(sizeof(float) * (size_t)W);
        float *ncum = (float *)malloc(sizeof(float) * (size_t)W);
        expansion *ex = (expansion *)malloc(sizeof(expansion) * (size_t)W * KC);
        int live = 1, m = L;
        uint32_t status = 0;
        cum[0] = 0.0f;

        for (int i = 0; i < L; ++i) {
            const int64_t r = (int64_t)b * L + i;
            const int cnt = cand_count[r];
            const float top1 = cand_logit[r * KC];
            int n = 0;
            for (int w = 0; w < live; ++w) {
                for (int k = 0; k < cnt; ++k) {
                    int32_t tok = cand_id[r * KC + k];
                    volatile float g = cand_logit[r * KC + k] - top1;
                    float ng = proxy_at(proxy_kind, table, table_log2, hash_seed, V, prev_token, b, L, KC,
                                        i, k, tok, ids + w * L, slots + w * L);
                    volatile float a = lambda * g;
                    volatile float c = oml * ng;
                    volatile float step = a + c;
                    if (ver_score) {
                        volatile float v = mu * ver_score[r * KC + k];
                        step = step + v;
                    }
                    volatile float s = cum[w] + step;
                    ex[n].cum = s;
                    ex[n].tok = tok;
                    ex[n].parent = w;
                    ex[n].slot = k;
                    ++n;
                }
            }
            if (n == 0) { m = i; break; }          /* an empty position ends the lattice */
            /* plain insertion sort of all expansions under the beam order */
            for (int a = 1; a < n; ++a) {
                expansion e = ex[a];
                int p = a;
                while (p > 0 && exp_before(&e, &ex[p - 1])) { ex[p] = ex[p - 1]; --p; }
                ex[p] = e;
            }
            int keep = n < W ? n : W;
            for (int w = 0; w < keep; ++w) {
                memcpy(nids + w * L, ids + ex[w].parent * L, sizeof(int32_t) * (size_t)i);
                memcpy(nslots + w * L, slots + ex[w].parent * L, sizeof(int32_t) * (size_t)i);
                nids[w * L + i] = ex[w].tok;
                nslots[w * L + i] = ex[w].slot;
                ncum[w] = ex[w].cum;
            }
            int32_t *t;
            float *tf;
            t = ids; ids = nids; nids = t;
            t = slots; slots = nslots; nslots = t;
            tf = cum; cum = ncum; ncum = tf;
            live = keep;
            if (eos_id >= 0 && ids[i] == eos_id) { m = i + 1; status |= ORC_EOS_STOPPED; break; }
        }

        path_len[b] = m;
        for (int i = 0; i < L; ++i) {
            path[(int64_t)b * L + i] = i < m ? ids[i] : -1;
            path_slot[(int64_t)b * L + i] = i < m ? slots[i] : -1;
        }
        for (int w = 0; w < W; ++w) {
            double s = -INFINITY;
            if (w < live) {
                /* Eq. 8 written out on the returned path */
                s = 0.0;
                for (int i = 0; i < m; ++i) {
                    const int64_t r = (int64_t)b * L + i;
                    double ldlm = (double)cand_logit[r * KC + slots[w * L + i]] - lse64[r];
                    double lng = (double)proxy_at(proxy_kind, table, table_log2, hash_seed, V, prev_token,
                                                  b, L, KC, i, slots[w * L + i], ids[w * L + i],
                                                  ids + w * L, slots + w * L);
                    s += (double)lambda * ldlm + (double)oml * lng;
                    if (ver_score) s += (double)mu * (double)ver_score[r * KC + slots[w * L + i]];
                }
            }
            if (w == 0) path_score[b] = (float)s;
            if (beam_score) beam_score[(int64_t)b * W + w] = (float)s;
            if (beam_cum) beam_cum[(int64_t)b * W + w] = w < live ? cum[w] : -INFINITY;
            if (beam_ids)
                for (int i = 0; i < L; ++i)
                    beam_ids[((int64_t)b * W + w) * L + i] = (w < live && i < m) ? ids[w * L + i] : -1;
        }
        if (row_status) row_status[b] = status;
        free(ids); free(slots); free(nids); free(nslots); free(cum); free(ncum); free(ex);
    }
    return 0;
}

/* Eq. 8 as the paper has it: no verifier-side term. */
int orc_cps_search(const int32_t *cand_id, const float *cand_logit, const double *lse64,
                   const int32_t *cand_count, int B, int L, int KC,
                   const int32_t *prev_token, int proxy_kind, const float *table,
                   int table_log2, uint32_t hash_seed, int64_t V,
                   int W, float lambda, int eos_id,
                   int32_t *path, int32_t *path_slot, int32_t *path_len, float *path_score,
                   int32_t *beam_ids, float *beam_score, float *beam_cum,
                   uint32_t *row_status)
{
    return orc_cps_search_biased(cand_id, cand_logit, lse64, cand_count, B, L, KC, prev_token, proxy_kind, table,
                                 table_log2, hash_seed, V, W, lambda, eos_id, NULL, 0.0f, path, path_slot, path_len,
                                 path_score, beam_ids, beam_score, beam_cum, row_status);
}

/*
 * Inverse-CDF draw in token-id order from unnormalised masses
 *   r_v = max(0, p(v) - q(v))      (Sec. 2: residual distribution [p - q]_+)
 * with p = softmax(target row), q = softmax(draft row) (q = 0 if draft row is
 * NULL: a draw from p itself).  token = smallest v with r_v > 0 and
 * sum_{w<=v} r_w >= u * R, R = sum_v r_v.  Returns -1 when R = 0.
 * If probe >= 0 also reports F(probe-1), F(probe) (normalised CDF) and r_probe.
 */
static int64_t residual_draw(const void *trow, const void *drow, int dtype, int64_t V,
                             double lse_t, double lse_d, double u,
                             int64_t probe, double *F_lo, double *F_hi, double *r_probe)
{
    double R = 0.0;
    for (int64_t v = 0; v < V; ++v) {
        double p = exp(logit_at(trow, dtype, v) - lse_t);
        double q = drow ? exp(logit_at(drow, dtype, v) - lse_d) : 0.0;
        double r = p - q;
        if (r > 0.0) R += r;
    }
    if (!(R > 0.0)) return -1;
    const double thr = u * R;
    double cum = 0.0;
    int64_t tok = -1, last_pos = -1;
    for (int64_t v = 0; v < V; ++v) {
        double p = exp(logit_at(trow, dtype, v) - lse_t);
        double q = drow ? exp(logit_at(drow, dtype, v) - lse_d) : 0.0;
        double r = p - q;
        if (!(r > 0.0)) r = 0.0;
        if (v == probe) {
            if (F_lo) *F_lo = cum / R;
            if (F_hi) *F_hi = (cum + r) / R;
            if (r_probe) *r_probe = r;
        }
        cum += r;
        if (r > 0.0) {
            last_pos = v;
            if (tok < 0 && cum >= thr) tok = v;
        }
    }
    return tok >= 0 ? tok : last_pos;   /* rounding at the very top of the CDF */
}

/* Exported for tolerance checks: the oracle's CDF around a given token. */
int64_t orc_residual_probe(const void *trow, const void *drow, int dtype, int64_t V,
                           double u, int64_t probe, double *F_lo, double *F_hi, double *r_probe)
{
    double lse_t, lse_d = 0.0;
    if (row_stats(trow, dtype, V, &lse_t, NULL, NULL)) return -2;
    if (drow && row_stats(drow, dtype, V, &lse_d, NULL, NULL)) return -2;
    return residual_draw(trow, drow, dtype, V, lse_t, lse_d, u, probe, F_lo, F_hi, r_probe);
}

/*
 * Verification of the chosen path (Sec. 2: Eq. 1 acceptance, residual
 * resampling, Eq. 2 accepted length; Sec. 4: greedy = temperature 0;
 * Alg. 1 stage 3; q is the draft row's own softmax, the left-to-right proxy
 * of Eq. 6 under one refinement step).
 *
 * mode[b] = 0 greedy: token i is accepted iff it equals argmax of target row
 *   i (lowest id on ties); the correction at the first rejection is that
 *   argmax.
 * mode[b] = 1 stochastic: ratio_i = p_i(y_i) / q_i(y_i); accept iff
 *   u[b,i] < ratio_i; on the first rejection the replacement is drawn from
 *   the residual with u[b,L].
 * All m tokens accepted: if a target row m exists (m < Lt) the bonus token is
 *   its argmax (greedy) or a draw from p_m with u[b,L]; else next_token = -1
 *   and NO_BONUS_ROW is flagged.
 * accepted_len counts an accepted EOS; EOS_ACCEPTED is flagged then.
 * ratio[B,L]: the ratio at every i < m of a stochastic row, -1 elsewhere.
 * tgt_argmax / tgt_lse [B,Lt] are filled for every target row.
 */
int orc_verify(const void *target, const void *draft, int dtype, int B, int L, int Lt, int64_t V,
               const int32_t *path, const int32_t *path_len,
               const uint8_t *mode, const float *u, int eos_id,
               int32_t *accepted_len, int32_t *next_token, float *ratio,
               int32_t *tgt_argmax, float *tgt_lse, uint32_t *row_status)
{
    if (B < 0 || L < 1 || Lt < L || V < 1) return -1;
    const size_t es = dtype ? 2 : 4;

#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        uint32_t status = 0;
        const int m = path_len[b];
        const int stochastic = mode ? mode[b] != 0 : 0;
        double *lse_t = (double *)malloc(sizeof(double) * (size_t)Lt);
        int64_t *amax = (int64_t *)malloc(sizeof(int64_t) * (size_t)Lt);
        for (int i = 0; i < Lt; ++i) {
            const char *trow = (const char *)target + ((size_t)b * Lt + i) * (size_t)V * es;
            if (row_stats(trow, dtype, V, &lse_t[i], NULL, &amax[i])) status |= ORC_NONFINITE_INPUT;
            if (tgt_argmax) tgt_argmax[(int64_t)b * Lt + i] = (int32_t)amax[i];
            if (tgt_lse) tgt_lse[(int64_t)b * Lt + i] = (float)lse_t[i];
        }
        if (ratio)
            for (int i = 0; i < L; ++i) ratio[(int64_t)b * L + i] = -1.0f;

        int acc = m;       /* Eq. 2: first failure index, or m */
        double lse_d_rej = 0.0;
        for (int i = 0; i < m; ++i) {
            const int32_t y = path[(int64_t)b * L + i];
            int ok;
            if (!stochastic) {
                ok = (int64_t)y == amax[i];
            } else {
                const char *trow = (const char *)target + ((size_t)b * Lt + i) * (size_t)V * es;
                const char *drow = (const char *)draft + ((size_t)b * L + i) * (size_t)V * es;
                double lse_d;
                if (row_stats(drow, dtype, V, &lse_d, NULL, NULL)) status |= ORC_NONFINITE_INPUT;
                double lp = logit_at(trow, dtype, y) - lse_t[i];
                double lq = logit_at(drow, dtype, y) - lse_d;
                double rt = exp(lp - lq);                     /* Eq. 1: p/q */
                if (ratio) ratio[(int64_t)b * L + i] = (float)rt;
                ok = (double)u[(int64_t)b * (L + 1) + i] < rt;
                if (!ok && acc == m) lse_d_rej = lse_d;
            }
            if (!ok && acc == m) {
                acc = i;
                if (!ratio || !stochastic) break;             /* later ratios only feed the output */
            }
        }
        accepted_len[b] = acc;
        for (int i = 0; i < acc; ++i)
            if (eos_id >= 0 && path[(int64_t)b * L + i] == eos_id) status |= ORC_EOS_ACCEPTED;

        int32_t nt = -1;
        if (acc < m) {                                       /* rejected at position acc */
            if (!stochastic) {
                nt = (int32_t)amax[acc];
            } else {
                const char *trow = (const char *)target + ((size_t)b * Lt + acc) * (size_t)V * es;
                const char *drow = (const char *)draft + ((size_t)b * L + acc) * (size_t)V * es;
                int64_t t = residual_draw(trow, drow, dtype, V, lse_t[acc], lse_d_rej,
                                          (double)u[(int64_t)b * (L + 1) + L], -1, NULL, NULL, NULL);
                if (t < 0) { t = amax[acc]; status |= ORC_ZERO_RESIDUAL; }
                nt = (int32_t)t;
            }
        } else if (m < Lt) {                                 /* bonus from target row m */
            if (!stochastic) {
                nt = (int32_t)amax[m];
            } else {
                const char *trow = (const char *)target + ((size_t)b * Lt + m) * (size_t)V * es;
                int64_t t = residual_draw(trow, NULL, dtype, V, lse_t[m], 0.0,
                                          (double)u[(int64_t)b * (L + 1) + L], -1, NULL, NULL, NULL);
                if (t < 0) { t = amax[m]; status |= ORC_ZERO_RESIDUAL; }
                nt = (int32_t)t;
            }
        } else {
            status |= ORC_NO_BONUS_ROW;
        }
        next_token[b] = nt;
        if (row_status) row_status[b] = status;
        free(lse_t);
        free(amax);
    }
    return 0;
}

/*
 * One refinement step of the diffusion drafter, on its logits (Sec. 3.1,
 * Eq. 5, with the update set "top-K by confidence").
 * For every position i of batch row b that is still masked:
 *   a_i    = argmax_v x_{i,v}            (lowest id on ties)
 *   conf_i = log q(a_i) = x_max - lse     (rounded to fp32: the precision in
 *            which positions are compared)
 * U = the min(n_update, |M|) masked positions with the largest conf (equal
 * conf: the lower position first).  For i in U: tokens[i] = a_i and
 * masked[i] = 0; every other entry of tokens / masked stays as it is.
 * argmax / confidence report a_i / conf_i of the positions that were masked
 * on entry and -1 / -inf elsewhere; n_left[b] = |M| on return.
 * A masked row with NaN / +inf or without a finite logit flags the batch row
 * (ORC_NONFINITE_INPUT) and takes conf = -inf.
 */
int orc_unmask_step(const void *logits, int dtype, int B, int L, int64_t V, int n_update,
                    int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence,
                    int32_t *n_left, uint32_t *row_status)
{
    if (B < 0 || L < 1 || V < 1 || n_update < 1) return -1;
    #pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        uint32_t status = 0;
        int nmask = 0;
        for (int i = 0; i < L; ++i) {
            const int64_t r = (int64_t)b * L + i;
            argmax[r] = -1;
            confidence[r] = -INFINITY;
            if (!masked[r]) continue;
            ++nmask;
            const char *row = (const char *)logits + (size_t)r * (size_t)V * (dtype == 0 ? 4 : 2);
            double lse;
            int64_t am;
            if (row_stats(row, dtype, V, &lse, NULL, &am)) {
                status |= ORC_NONFINITE_INPUT;
                argmax[r] = (int32_t)am;
                continue;
            }
            argmax[r] = (int32_t)am;
            confidence[r] = (float)(logit_at(row, dtype, am) - lse);
        }
        const int take = n_update < nmask ? n_update : nmask;
        for (int t = 0; t < take; ++t) {
            int best = -1;
            for (int i = 0; i < L; ++i) {                 /* strict >: the lower position wins ties */
                const int64_t r = (int64_t)b * L + i;
                if (!masked[r]) continue;
                if (best < 0 || confidence[r] > confidence[(int64_t)b * L + best]) best = i;
            }
            const int64_t r = (int64_t)b * L + best;
            tokens[r] = argmax[r];
            masked[r] = 0;
        }
        n_left[b] = nmask - take;
        if (row_status) row_status[b] = status;
    }
    return 0;
}

/*
 * Token tree of the surviving beams, for verifying several paths in one target
 * pass (Sec. 2 names tree-based parallel verification as verifier-side
 * engineering; the paper verifies the rank-0 path only).
 * Beams that share a prefix share its nodes.  Nodes are numbered in the order
 * (beam rank ascending, depth ascending) of their first use, so the rank-0 path
 * is nodes 0 .. m-1.  node_parent is the node before it on its path (-1 at depth
 * 0).  beam_node[b,w,i] = node of beam w at depth i (-1 where the beam has no
 * token).  Unused node slots hold token -1, parent -1, depth -1.
 */
int orc_beam_tree(const int32_t *beam_ids, const int32_t *path_len, int B, int W, int L,
                  int32_t *node_token, int32_t *node_parent, int32_t *node_depth,
                  int32_t *beam_node, int32_t *n_nodes)
{
    if (B < 0 || W < 1 || L < 1) return -1;
    const int N = W * L;
    for (int b = 0; b < B; ++b) {
        int32_t *tok = node_token + (int64_t)b * N, *par = node_parent + (int64_t)b * N;
        int32_t *dep = node_depth + (int64_t)b * N, *bn = beam_node + (int64_t)b * N;
        for (int n = 0; n < N; ++n) { tok[n] = -1; par[n] = -1; dep[n] = -1; bn[n] = -1; }
        const int m = path_len[b] < 0 ? 0 : (path_len[b] > L ? L : path_len[b]);
        int count = 0;
        for (int w = 0; w < W; ++w) {
            const int32_t *ids = beam_ids + ((int64_t)b * W + w) * L;
            int parent = -1;
            for (int i = 0; i < m; ++i) {
                if (ids[i] < 0) break;                  /* this beam does not exist */
                int found = -1;
                for (int n = 0; n < count; ++n)         /* a child of `parent` with this token? */
                    if (dep[n] == i && par[n] == parent && tok[n] == ids[i]) { found = n; break; }
                if (found < 0) {
                    found = count++;
                    tok[found] = ids[i]; par[found] = parent; dep[found] = i;
                }
                bn[w * L + i] = found;
                parent = found;
            }
        }
        n_nodes[b] = count;
    }
    return 0;
}

/*
 * Greedy verification of a token tree (the greedy rule of Sec. 4 applied along
 * the tree): target row 0 is the distribution after the prefix, row 1+n the
 * distribution after node n.  Starting at the root, the argmax (lowest id on
 * ties) of the current row selects the child that carries that token; the walk
 * ends where no child does.  accepted_len = nodes walked, accepted_node[b,i] =
 * the i-th of them (-1 beyond), next_token = the argmax of the row the walk
 * ended at (correction, or bonus after a leaf).
 * target is [B, 1 + N, V] with N = W*L node slots; only rows of existing nodes
 * are read.  An existing row with NaN / +inf or no finite logit flags the batch
 * row.
 */
int orc_verify_tree(const void *target, int dtype, int B, int N, int64_t V,
                    const int32_t *node_token, const int32_t *node_parent, const int32_t *n_nodes,
                    int L, int32_t *accepted_len, int32_t *accepted_node, int32_t *next_token,
                    uint32_t *row_status)
{
    if (B < 0 || N < 1 || V < 1 || L < 1) return -1;
    const size_t es = dtype == 0 ? 4 : 2;
    #pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = node_token + (int64_t)b * N, *par = node_parent + (int64_t)b * N;
        uint32_t status = 0;
        int ctx = -1, acc = 0;                          /* node the walk stands on; -1 = root */
        for (int i = 0; i < L; ++i) accepted_node[(int64_t)b * L + i] = -1;
        int64_t am = 0;
        for (int r = 0; r <= n_nodes[b]; ++r) {         /* every existing row is checked, as in orc_verify */
            const char *row = (const char *)target + ((size_t)b * (size_t)(1 + N) + (size_t)r) * (size_t)V * es;
            if (row_stats(row, dtype, V, NULL, NULL, &am)) status |= ORC_NONFINITE_INPUT;
        }
        for (;;) {
            const char *row = (const char *)target + ((size_t)b * (size_t)(1 + N) + (size_t)(1 + ctx)) * (size_t)V * es;
            row_stats(row, dtype, V, NULL, NULL, &am);
            int child = -1;
            for (int n = 0; n < n_nodes[b]; ++n)
                if (par[n] == ctx && tok[n] == (int32_t)am) { child = n; break; }
            if (child < 0 || acc >= L) break;
            accepted_node[(int64_t)b * L + acc] = child;
            ++acc;
            ctx = child;
        }
        accepted_len[b] = acc;
        next_token[b] = (int32_t)am;
        if (row_status) row_status[b] = status;
    }
    return 0;
}

/*
 * Adaptive draft length (Sec. 3.3, Eq. 9-11; Alg. 1 init and stage 4).
 * state = { ema_gen, ema_acc, k }.  Init: both averages 0, k = k_max.
 * Update with the batch means of gen_len and accepted_len (batch 1 is the
 * paper's case):
 *   ema = (1-rho) * ema + rho * signal                           (Eq. 10)
 *   k'  = clip( ceil( ema_gen + delta * [ema_acc >= ema_gen] ), k_min, k_max )   (Eq. 11)
 * with the ceiling result first rounded up to a multiple of `granularity`
 * (1 = the paper's rule).
 */
typedef struct {
    double ema_gen;
    double ema_acc;
    int32_t k;
    int32_t steps;
} orc_adl_state;

void orc_adl_init(orc_adl_state *st, int k_max)
{
    st->ema_gen = 0.0;
    st->ema_acc = 0.0;
    st->k = k_max;
    st->steps = 0;
}

int orc_adl_update(orc_adl_state *st, const int32_t *accepted_len, const int32_t *gen_len, int B,
                   int k_min, int k_max, double delta, double rho, int granularity)
{
    double sg = 0.0, sa = 0.0;
    for (int b = 0; b < B; ++b) { sg += gen_len[b]; sa += accepted_len[b]; }
    double Lgen = sg / B, Lacc = sa / B;
    st->ema_gen = (1.0 - rho) * st->ema_gen + rho * Lgen;
    st->ema_acc = (1.0 - rho) * st->ema_acc + rho * Lacc;
    double z = ceil(st->ema_gen + (st->ema_acc >= st->ema_gen ? delta : 0.0));
    long k = (long)z;
    if (granularity > 1) k = ((k + granularity - 1) / granularity) * granularity;
    if (k < k_min) k = k_min;
    if (k > k_max) k = k_max;
    st->k = (int32_t)k;
    st->steps += 1;
    return st->k;
}

/*
 * Joint control of the search breadth (Sec. 6, future work iii, names it without a rule; the
 * reading taken, stated in the design doc: the controller of Eq. 10-11 with two more signals).
 * Per step, batch means:
 *   H = mean over batch rows b and positions i < max(1, gen_len[b]) of entropy[b,i]   (nats)
 *   s = mean over b of max(0, gen_len[b] - accepted_len[b]) / max(1, gen_len[b])       (shortfall)
 *   ema = (1-rho) * ema + rho * signal                  (the form of Eq. 10, both start at 0)
 *   K' = clip( ceil( exp(ema_H) ), K_min, K_max )       (the drafter's perplexity: how many
 *                                                        candidates carry its mass)
 *   W' = clip( ceil( W_min + (W_max - W_min) * ema_s ), W_min, W_max )
 *                                                       (wider beams while verification cuts
 *                                                        drafts short)
 * Init: K = K_max, W = W_max (as Alg. 1 starts the draft length at k_max).
 */
typedef struct {
    double ema_entropy;
    double ema_shortfall;
    int32_t K, W;
    int32_t steps;
} orc_breadth_state;

void orc_breadth_init(orc_breadth_state *st, int K_max, int W_max)
{
    st->ema_entropy = 0.0;
    st->ema_shortfall = 0.0;
    st->K = K_max;
    st->W = W_max;
    st->steps = 0;
}

int orc_breadth_update(orc_breadth_state *st, const float *entropy, const int32_t *accepted_len,
                       const int32_t *gen_len, int B, int L, int K_min, int K_max, int W_min, int W_max,
                       double rho)
{
    if (B < 1 || L < 1) return -1;
    double Hsum = 0.0, ssum = 0.0;
    int64_t npos = 0;
    for (int b = 0; b < B; ++b) {
        int g = gen_len[b] < 1 ? 1 : (gen_len[b] > L ? L : gen_len[b]);
        for (int i = 0; i < g; ++i) Hsum += (double)entropy[(int64_t)b * L + i];
        npos += g;
        int short_by = gen_len[b] - accepted_len[b];
        if (short_by < 0) short_by = 0;
        ssum += (double)short_by / (double)(gen_len[b] < 1 ? 1 : gen_len[b]);
    }
    st->ema_entropy = (1.0 - rho) * st->ema_entropy + rho * (Hsum / (double)npos);
    st->ema_shortfall = (1.0 - rho) * st->ema_shortfall + rho * (ssum / (double)B);
    double k = ceil(exp(st->ema_entropy));
    double w = ceil((double)W_min + (double)(W_max - W_min) * st->ema_shortfall);
    if (k < K_min) k = K_min;
    if (k > K_max) k = K_max;
    if (w < W_min) w = W_min;
    if (w > W_max) w = W_max;
    st->K = (int32_t)k;
    st->W = (int32_t)w;
    st->steps += 1;
    return 0;
}

/*
 * Stochastic verification of a token tree (Sec. 2 names tree-based parallel verification and
 * cites it; the rule is the multi-branch form of Eq. 1 with residual resampling: the siblings
 * of a node are tried one after the other, and every rejection replaces the target
 * distribution by the normalised residual before the next sibling is tried).
 *
 * target [B, 1+N, V]: row 0 after the prefix, row 1+n after node n.  draft [B, L, V]: row i is
 * the drafter's distribution q_i of every node at depth i (one refinement step: the left-to-right
 * proxy of Eq. 6 is the draft row itself).  u [B, N+1]: u[b,n] is the draw used if node n is
 * tried, u[b,N] the draw of the emitted token.
 *
 * Walk from the root (depth i = 0, f = softmax(target row 0)):
 *   the children of the current node, in node order: child n with token x is accepted iff
 *   u[b,n] < f(x) / q_i(x) (f(x) > 0 = q_i(x) accepts, f(x) = 0 rejects); accepted: the walk
 *   moves to n, i += 1, f = softmax(target row 1+n).  Rejected: f <- [f - q_i]_+ / R with
 *   R = sum_v [f(v) - q_i(v)]_+, and the next sibling is tried against the new f.
 *   When no child is left (all rejected, a leaf, or i = L): next_token = smallest v with
 *   f(v) > 0 and sum_{w<=v} f(w) >= u[b,N] * sum_w f(w).
 *   R = 0 (not a number either): next_token = argmax of the current node's target row,
 *   ORC_ZERO_RESIDUAL.
 * accepted_len = nodes walked, accepted_node[b,i] = the i-th of them (-1 beyond).
 * An existing target row or a used draft row with NaN / +inf or no finite logit flags the batch row.
 *
 * margin [B] (may be NULL; a diagnostic, no part of the rule): how far the batch row's closest
 * decision was from going the other way: over the acceptance tests |u - f(x)/q(x)| relative to
 * the larger of the two, and for the emitted token the distance of u * sum f from the two ends of
 * that token's step of the cumulative sum, relative to sum f.  A comparison against arithmetic of
 * lower precision can tell a rounding difference from a wrong result with it.
 */
int orc_verify_tree_stochastic(const void *target, const void *draft, int dtype, int B, int N, int L, int64_t V,
                               const int32_t *node_token, const int32_t *node_parent, const int32_t *n_nodes,
                               const float *u, int32_t *accepted_len, int32_t *accepted_node,
                               int32_t *next_token, uint32_t *row_status, double *margin)
{
    if (B < 0 || N < 1 || V < 1 || L < 1) return -1;
    const size_t es = dtype == 0 ? 4 : 2;
    #pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const int32_t *tok = node_token + (int64_t)b * N, *par = node_parent + (int64_t)b * N;
        const int nn = n_nodes[b] < 0 ? 0 : (n_nodes[b] > N ? N : n_nodes[b]);
        uint32_t status = 0;
        double closest = INFINITY;
        double *f = (double *)malloc(sizeof(double) * (size_t)V);
        double *q = (double *)malloc(sizeof(double) * (size_t)V);
        for (int i = 0; i < L; ++i) accepted_node[(int64_t)b * L + i] = -1;
        for (int r = 0; r <= nn; ++r) {                 /* every existing row is checked */
            const char *row = (const char *)target + ((size_t)b * (size_t)(1 + N) + (size_t)r) * (size_t)V * es;
            if (row_stats(row, dtype, V, NULL, NULL, NULL)) status |= ORC_NONFINITE_INPUT;
        }
        int ctx = -1, acc = 0;
        int64_t token = -1;
        for (;;) {
            const char *trow = (const char *)target + ((size_t)b * (size_t)(1 + N) + (size_t)(1 + ctx)) * (size_t)V * es;
            double lse_t;
            int64_t am;
            row_stats(trow, dtype, V, &lse_t, NULL, &am);
            for (int64_t v = 0; v < V; ++v) f[v] = exp(logit_at(trow, dtype, v) - lse_t);
            int moved = 0, dead = 0, have_q = 0;
            for (int n = 0; n < nn && acc < L && !moved && !dead; ++n) {
                if (par[n] != ctx) continue;
                if (!have_q) {
                    const char *drow = (const char *)draft + ((size_t)b * L + (size_t)acc) * (size_t)V * es;
                    double lse_d;
                    if (row_stats(drow, dtype, V, &lse_d, NULL, NULL)) status |= ORC_NONFINITE_INPUT;
                    for (int64_t v = 0; v < V; ++v) q[v] = exp(logit_at(drow, dtype, v) - lse_d);
                    have_q = 1;
                }
                const int32_t x = tok[n];
                const double fx = f[x], qx = q[x];
                int ok;
                if (qx > 0.0) {
                    const double uu = (double)u[(int64_t)b * (N + 1) + n], ratio = fx / qx;
                    ok = uu < ratio;
                    const double big = uu > ratio ? uu : ratio;
                    const double m = big > 0.0 ? fabs(uu - ratio) / big : 0.0;
                    if (m < closest) closest = m;
                } else ok = fx > 0.0;
                if (ok) {
                    accepted_node[(int64_t)b * L + acc] = n;
                    ++acc;
                    ctx = n;
                    moved = 1;
                } else {
                    double R = 0.0;
                    for (int64_t v = 0; v < V; ++v) {
                        double r = f[v] - q[v];
                        f[v] = r > 0.0 ? r : 0.0;
                        R += f[v];
                    }
                    if (!(R > 0.0)) { dead = 1; token = am; status |= ORC_ZERO_RESIDUAL; }
                    else for (int64_t v = 0; v < V; ++v) f[v] /= R;
                }
            }
            if (moved) continue;
            if (!dead) {
                double R = 0.0;
                for (int64_t v = 0; v < V; ++v) R += f[v];
                if (!(R > 0.0)) { token = am; status |= ORC_ZERO_RESIDUAL; }
                else {
                    const double thr = (double)u[(int64_t)b * (N + 1) + N] * R;
                    double cum = 0.0;
                    int64_t last_pos = -1;
                    for (int64_t v = 0; v < V; ++v) {
                        cum += f[v];
                        if (f[v] > 0.0) {
                            last_pos = v;
                            if (cum >= thr) {
                                token = v;
                                const double up = (cum - thr) / R, down = (thr - (cum - f[v])) / R;
                                const double m = up < down ? up : down;
                                if (m < closest) closest = m;
                                break;
                            }
                        }
                    }
                    if (token < 0) token = last_pos;    /* rounding at the very top of the CDF */
                }
            }
            break;
        }
        accepted_len[b] = acc;
        next_token[b] = (int32_t)token;
        if (row_status) row_status[b] = status;
        if (margin) margin[b] = closest;
        free(f);
        free(q);
    }
    return 0;
}
