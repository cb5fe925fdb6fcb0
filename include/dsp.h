/*
 * dsp.h -- C ABI of the B200-native draft-and-verify core of DiffuSpec.
 *
 * One speculative step works on logits only (the two language models are the
 * caller's): dsp_lattice_build turns the diffusion drafter's [B,L,V] block
 * logits into the token lattice, dsp_cps_search picks one left-to-right path
 * through it, dsp_verify checks that path against the target model's
 * [B,Lt,V] logits, dsp_adl_update (host) sets the next draft length.
 *
 * Conventions
 *  - Every function returns 0 (DSP_OK) or a negative dsp_status.  Argument
 *    errors are detected on the host before anything is enqueued.
 *  - Unless marked "host", every pointer is a DEVICE pointer to memory the
 *    caller owns (inputs, outputs and the scratch workspace).  The library
 *    allocates nothing and keeps no device state between calls (exceptions:
 *    dsp_lattice_build_static holds its scratch in a static array,
 *    dsp_draft_verify_step keeps one stream and two events per device, and a
 *    dsp_step_graph is a CUDA graph object).
 *  - Device calls only enqueue work on `stream` (a cudaStream_t; NULL is the
 *    legacy default stream) and never synchronise.  Outputs are valid once
 *    the stream reaches the end of the call.  Two calls that share a
 *    workspace must be ordered (same stream, or an event between them).
 *  - Data-dependent conditions are reported per batch row in row_status[B]
 *    (bit flags below), never as a return code.
 *  - Tensors are row-major.  Logits have the vocabulary dimension contiguous;
 *    stride_b / stride_l are in elements.  dtype is DSP_F32 or DSP_BF16.
 *    Rows whose first element is 16-byte aligned are read with 128-bit loads;
 *    any other layout takes an element-wise CUDA path (slower, same results).
 *  - Positions, ranks and slots are 0-based (the paper counts from 1).
 *  - -inf logits are legal (masked tokens).  NaN or +inf logits, or a row with
 *    no finite logit, set DSP_ROW_NONFINITE_INPUT; that row's outputs are then
 *    unspecified but in bounds.  Finite logits must exceed -1e37.
 *  - The total order on tokens of one row is (logit descending, token id
 *    ascending): the lowest id wins every tie (-0.0 and +0.0 are equal).
 */
#ifndef DSP_H_
#define DSP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *dsp_stream_t;   /* a cudaStream_t */

enum dsp_status {
    DSP_OK = 0,
    DSP_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, bad stride ... */
    DSP_ERR_UNSUPPORTED = -2,   /* dtype, K_max, W or L beyond the compiled limits */
    DSP_ERR_WORKSPACE = -3,     /* workspace_bytes smaller than the query call's answer */
    DSP_ERR_CUDA = -4,          /* a CUDA runtime call failed; see dsp_last_cuda_error */
    DSP_ERR_STATIC_SCRATCH = -5 /* dsp_lattice_build_static: the problem needs more scratch than
                                   the library's built-in array of DSP_STATIC_WS_BYTES holds */
};

enum dsp_dtype { DSP_F32 = 0, DSP_BF16 = 1 };

/* row_status bit flags */
#define DSP_ROW_NONFINITE_INPUT 1u  /* NaN/+inf logit, or no finite logit, in a row of this batch row */
#define DSP_ROW_ZERO_RESIDUAL   2u  /* residual mass was 0: replacement = target argmax */
#define DSP_ROW_NO_BONUS_ROW    4u  /* whole path accepted and no target row path_len exists */
#define DSP_ROW_EOS_ACCEPTED    8u  /* an accepted token is EOS: the caller terminates decoding */
#define DSP_ROW_EOS_STOPPED     16u /* the path search stopped early at an EOS */
#define DSP_ROW_TIMEOUT         32u /* a bounded wait inside a kernel ran out (hardware fault or a
                                       defect of this library): the row's outputs are unspecified */

#define DSP_MAX_K 32      /* largest K_max (per-position candidate cap M_max) */
#define DSP_MAX_W 32      /* largest beam width */
#define DSP_MAX_L 1024    /* largest draft length */

/* Kernels whose launch dsp_profile_events can bracket with events. */
enum dsp_profile_point {
    DSP_PROFILE_LATTICE_SCAN = 0,   /* the pass over the draft logits inside dsp_lattice_build */
    DSP_PROFILE_TARGET_SCAN = 1     /* the pass over the target logits inside dsp_verify */
};

const char *dsp_strerror(int32_t status);   /* host; static string */
int32_t dsp_last_cuda_error(void);          /* host; the cudaError_t behind the last DSP_ERR_CUDA */
int32_t dsp_version(void);                  /* host; ABI version, currently 1 */

/* Measurement aid (host; not thread-safe; no counterpart in the paper).  While `start` and
 * `stop` (caller-owned cudaEvent_t handles created with timing enabled) are set for a point,
 * every later call that launches that kernel records `start` right before and `stop` right
 * after the launch on the call's stream, so that cudaEventElapsedTime gives the kernel's own
 * duration without the call's other work.  Two NULLs switch the point off again.
 * Errors: INVALID_ARG (unknown point, or only one of the two events given). */
int32_t dsp_profile_events(int32_t point, void *start, void *stop);

/* Measurement aid (no counterpart in the paper): a kernel that only reads `bytes` bytes (rounded
 * down to a multiple of 16) of device memory at `buffer` (device, 16-byte aligned) once, with
 * coalesced 128-bit loads, and keeps nothing.  Timed by the caller with events on `stream`, it
 * gives the read bandwidth this GPU reaches on a buffer of that size: the ceiling for the passes
 * over the logits, which read and hardly write.  `sink` (device, one uint32, caller-owned) is
 * written only if the folded data equals one fixed value; its content means nothing.
 * Enqueues on `stream` and returns.  Errors: INVALID_ARG (null or misaligned pointer,
 * bytes < 16), UNSUPPORTED (more than 2^31 - 1 pieces of 16 KB), CUDA. */
int32_t dsp_read_probe(const void *buffer, size_t bytes, uint32_t *sink, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Lattice build  (Sec. 3.2 "Lattice and pruning", Eq. 7; Alg. 1 stage 1;
 *                 the generation-length signal of Eq. 9)
 *
 * For every row (b,l) of draft_logits, in one pass over its V logits:
 *   lse      = log sum_v exp(x_v)                 (l^dlm(v) = x_v - lse)
 *   entropy  = lse - sum_v x_v exp(x_v - lse)     (nats; -inf logits add 0)
 *   the K = min(K_max, V) best tokens under the total order, -inf ones dropped
 *   (at least one is kept), with their exact logits and log-probabilities;
 *   cand_count = Eq. 7: the smallest m <= K whose cumulative full-vocabulary
 *   probability reaches tau, K if none does.  Pruning is off unless
 *   0 < tau <= 1.  If eos_id >= 0, EOS is not among the kept candidates and its
 *   logit is finite, EOS is appended as one extra slot ("always keep EOS");
 *   that slot is not counted in Eq. 7.
 *   gen_len[b] = number of positions before the first whose best token is
 *   eos_id (L if none, or if eos_id < 0)                          (Eq. 9)
 *
 * Inputs : draft_logits [B,L,V] (dtype), strides in elements.
 * Outputs: cand_id    int32 [B,L,KC]   KC = K_max + (eos_id >= 0 ? 1 : 0);
 *          cand_logit float [B,L,KC]   unused slots: id -1, logit -inf, logp -inf
 *          cand_logp  float [B,L,KC]
 *          cand_count int32 [B,L]
 *          lse        float [B,L]      (nullable)
 *          lse64      double[B,L]      the same value in double; dsp_cps_search
 *                                      and dsp_verify read it
 *          entropy    float [B,L]      (nullable)
 *          gen_len    int32 [B]
 *          row_status uint32[B]        overwritten
 * workspace: at least dsp_lattice_workspace_bytes(...) bytes, 256-byte aligned;
 *          contents need not be initialised and are garbage afterwards.  (The
 *          size of every workspace in this header depends on how rows are cut
 *          into slices, which follows the SM count of the current device: ask
 *          the query call with the device current on which the call will run.)
 * Errors : INVALID_ARG (null required pointer, B<0, L<1, V<1, stride < V ...),
 *          UNSUPPORTED (dtype, K_max outside 1..DSP_MAX_K, L > DSP_MAX_L),
 *          WORKSPACE, CUDA.  B == 0 is a no-op returning DSP_OK.
 */
int32_t dsp_lattice_workspace_bytes(int32_t B, int32_t L, int32_t V, int32_t dtype,
                                    int32_t K_max, size_t *bytes /* host, out */);

int32_t dsp_lattice_build(const void *draft_logits, int32_t dtype,
                          int32_t B, int32_t L, int32_t V,
                          int64_t stride_b, int64_t stride_l,
                          int32_t K_max, float tau, int32_t eos_id,
                          int32_t *cand_id, float *cand_logit, float *cand_logp,
                          int32_t *cand_count, float *lse, double *lse64, float *entropy,
                          int32_t *gen_len, uint32_t *row_status,
                          void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Lattice build without a caller-supplied workspace.  (The paper has no
 * counterpart: this entry point exists for the sake of deployment only.)
 *
 * Same inputs, outputs, results and argument errors as dsp_lattice_build, for
 * callers that cannot allocate device memory for the scratch workspace: code
 * that runs where cudaMalloc is not allowed or not reachable (inside another
 * framework's callback, on a thread that must not call allocating CUDA
 * routines, in a process whose device memory has all been handed out).  The
 * caller still owns and passes every input and output buffer.  The scratch is
 * an array of DSP_STATIC_WS_BYTES bytes that is part of the library image:
 * every GPU on which the library is loaded holds it until the process exits.
 *
 *  - This function calls no allocating routine (no cudaMalloc / cudaFree).
 *  - Limit: dsp_lattice_workspace_bytes(B, L, V, dtype, K_max) must not exceed
 *    DSP_STATIC_WS_BYTES, else DSP_ERR_STATIC_SCRATCH is returned and nothing
 *    is enqueued; this limit is checked first, the other argument errors of
 *    dsp_lattice_build after it.  (Layouts read with 128-bit loads need a few
 *    bytes per row; any other layout needs (24 + 8 K_max) bytes per row and
 *    slice: ask the query call.)
 *  - The first call on each device looks up the array's device address (a
 *    host-side, once-per-device step with that device current).  Make that
 *    first call outside any stream capture.
 *  - All calls on one device share the one array, which keeps what the last
 *    call left in it; each call clears on `stream` the part that has to start
 *    at zero.  Two calls whose GPU work may overlap (different streams with no
 *    ordering between them, or several host threads) race on it: order them.
 */
#define DSP_STATIC_WS_BYTES (4u << 20)

int32_t dsp_lattice_build_static(const void *draft_logits, int32_t dtype,
                                 int32_t B, int32_t L, int32_t V,
                                 int64_t stride_b, int64_t stride_l,
                                 int32_t K_max, float tau, int32_t eos_id,
                                 int32_t *cand_id, float *cand_logit, float *cand_logp,
                                 int32_t *cand_count, float *lse, double *lse64, float *entropy,
                                 int32_t *gen_len, uint32_t *row_status, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Causal-consistency path search  (Sec. 3.2 "Scoring and search", Eq. 8;
 *                                   Alg. 1 stage 2)
 *
 * Left-to-right beam search of width W over the lattice.  A path pi_1..pi_m
 * scores  S(pi) = sum_i [ lambda * l^dlm_i(pi_i) + (1-lambda) * l^ng(pi_{i-1}, pi_i) ]
 * with pi_0 = prev_token[b] (the last token of the prefix).  All live beams
 * have equal depth, so they are ranked on the fp32 quantity
 *   cum = sum_i step_i,  g = x - x_top1(i),
 *   step = fl( fl(lambda*g) + fl((1-lambda)*n) ),  cum = fl(cum + step),
 * (fl = round to fp32, no fused multiply-add, 1-lambda = fl(1 - lambda)), which
 * differs from Eq. 8 by a term common to all beams; survivors are the best
 * min(W, #expansions) under (cum descending, token id ascending, parent rank
 * ascending).  The search stops after the first depth at which the rank-0
 * survivor's new token is eos_id (row flag DSP_ROW_EOS_STOPPED).
 *
 * Causal proxy l^ng (the paper's n-gram model or small causal model, here
 * caller-supplied fp32 scores):
 *   proxy_kind 0: hashed table of 2^table_log2 entries, 1 <= table_log2 <= 31.
 *     With all arithmetic on uint32 modulo 2^32:
 *       h = prev * 0x9E3779B1;  h ^= cur + hash_seed;  h *= 0x9E3779B1;
 *       h ^= h >> 15;  h *= 0x9E3779B1;  h ^= h >> 13;
 *       l^ng = proxy_table[h >> (32 - table_log2)]
 *   proxy_kind 1: dense table [V,V]: l^ng = proxy_table[prev * V + cur]; a
 *     prev_token or candidate id outside [0, V) is clamped into it.
 *   proxy_kind 2: a tensor [B,L,KC,KC] of scores the caller computed for the
 *     lattice (a small causal model): l^ng of candidate slot k at position i
 *     after candidate slot p at position i-1 is proxy_table[b][i][p][k]; at
 *     position 0 row p = 0 is read.  prev_token, V, table_log2, hash_seed unused.
 *   proxy_kind 3: hashed trigram table of 2^table_log2 entries (the paper's
 *     proxy is a 3-gram model): l^ng(cur | prev2, prev) with
 *       g = prev2 * 0xC2B2AE35;  g ^= g >> 16;
 *       h = (prev ^ g) * 0x9E3779B1;  h ^= cur + hash_seed;  h *= 0x9E3779B1;
 *       h ^= h >> 15;  h *= 0x9E3779B1;  h ^= h >> 13;
 *       l^ng = proxy_table[h >> (32 - table_log2)]
 *     and prev_token int32 [B,2]: the prefix's last two tokens, oldest first.
 *
 * Inputs : cand_id, cand_logit, cand_count, lse64 as written by
 *          dsp_lattice_build (KC = their last dimension); prev_token int32 [B]
 *          ([B,2] for proxy_kind 3).
 * Outputs: path       int32 [B,L]   rank-0 path, -1 beyond path_len
 *          path_slot  int32 [B,L]   candidate slot of each path token, -1 beyond
 *          path_len   int32 [B]     m (0 if the first position has no candidate: the one
 *                                   surviving beam is then the empty path, score 0)
 *          path_score float [B]     Eq. 8 of the rank-0 path
 *          beam_ids   int32 [B,W,L] (nullable) all survivors by rank, -1 padded
 *          beam_score float [B,W]   (nullable) Eq. 8 per survivor, -inf if none
 *          beam_cum   float [B,W]   (nullable) the ranking quantity, -inf if none
 *          row_status uint32[B]     (nullable) flags OR-ed into existing content
 * Errors : INVALID_ARG, UNSUPPORTED (W outside 1..DSP_MAX_W, KC > DSP_MAX_K+1,
 *          L > DSP_MAX_L, proxy_kind), CUDA.
 */
int32_t dsp_cps_search(const int32_t *cand_id, const float *cand_logit,
                       const double *lse64, const int32_t *cand_count,
                       int32_t B, int32_t L, int32_t KC,
                       const int32_t *prev_token,
                       int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
                       uint32_t hash_seed, int32_t V,
                       int32_t W, float lambda, int32_t eos_id,
                       int32_t *path, int32_t *path_slot, int32_t *path_len, float *path_score,
                       int32_t *beam_ids, float *beam_score, float *beam_cum,
                       uint32_t *row_status, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Path search with a verifier-side term  (Sec. 6, future work ii: a scoring
 * that takes the verifier into account; the paper gives no rule, this is the
 * reading taken)
 *
 * dsp_cps_search with a third term in the path score,
 *   S(pi) = sum_i [ lambda * l^dlm_i(pi_i) + (1-lambda) * l^ng(pi_{i-1}, pi_i)
 *                   + mu * l^ver_i(pi_i) ],
 * where l^ver is a log-score of each lattice candidate from the verifier's
 * side (a distilled head, a cached verifier row, a unigram of the verifier:
 * the caller's choice), given slot by slot:
 *   ver_score float [B,L,KC] (device; nullable): entry [b,i,k] scores candidate
 *             slot k of position i; slots at or beyond cand_count are not read.
 *   mu        float: its weight (finite; any sign).
 * The ranking step becomes  step = fl( fl( fl(lambda*g) + fl((1-lambda)*n) )
 * + fl(mu * v) );  path_score and beam_score include the term.  With
 * ver_score null the call is dsp_cps_search bit for bit (mu is then ignored).
 * Everything else (arguments, outputs, order of ties, early stop, errors) is as
 * for dsp_cps_search; INVALID_ARG also for a NaN or infinite mu.
 * dsp_draft_verify_step and the step graph search without the term: a caller
 * that wants it makes the three calls.
 */
int32_t dsp_cps_search_biased(const int32_t *cand_id, const float *cand_logit,
                              const double *lse64, const int32_t *cand_count,
                              int32_t B, int32_t L, int32_t KC,
                              const int32_t *prev_token,
                              int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
                              uint32_t hash_seed, int32_t V,
                              int32_t W, float lambda, int32_t eos_id,
                              const float *ver_score, float mu,
                              int32_t *path, int32_t *path_slot, int32_t *path_len, float *path_score,
                              int32_t *beam_ids, float *beam_score, float *beam_cum,
                              uint32_t *row_status, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Verification  (Sec. 2: acceptance rule Eq. 1, residual resampling, accepted
 *                length Eq. 2; Sec. 4: greedy = temperature 0; Alg. 1 stage 3;
 *                the drafter probability q is the draft row's own softmax, the
 *                left-to-right proxy of Eq. 6 under one refinement step)
 *
 * mode[b] == 0 (greedy): token i < m is accepted iff it equals the argmax of
 *   target row i; the correction at the first rejection is that argmax.
 * mode[b] != 0 (stochastic): ratio_i = p_i(y_i) / q_i(y_i) evaluated in
 *   double; accepted iff u[b,i] < ratio_i; at the first rejection the
 *   replacement is the inverse-CDF draw, in token-id order with the single
 *   uniform u[b,L], from the residual max(0, p_i - q_i): the smallest v with
 *   positive residual whose cumulative residual reaches u * (total residual).
 *   A total of 0 gives the target argmax and DSP_ROW_ZERO_RESIDUAL.
 * accepted_len[b] = index of the first rejection, or m = path_len[b].
 * If all m are accepted and m < Lt, next_token is the bonus token from target
 * row m (argmax, or the same inverse-CDF draw from p_m); if m == Lt it is -1
 * and DSP_ROW_NO_BONUS_ROW is set.  An accepted EOS sets DSP_ROW_EOS_ACCEPTED.
 *
 * all_greedy != 0 promises that every row is greedy: mode, u, draft_logits,
 * cand_logit, path_slot and draft_lse64 may then be NULL, no exponentials are
 * evaluated and tgt_lse is not written.
 *
 * Inputs : target_logits [B,Lt,V], L <= Lt <= L+1; draft_logits [B,L,V] (same
 *          dtype); path, path_slot, path_len from dsp_cps_search; cand_logit
 *          [B,L,KC] and draft_lse64 [B,L] from dsp_lattice_build;
 *          mode uint8 [B]; u float [B,L+1] in [0,1).
 * Outputs: accepted_len int32 [B]; next_token int32 [B];
 *          ratio      float [B,L]   (nullable) p/q at every i < m of a stochastic
 *                                   row, -1 elsewhere
 *          tgt_argmax int32 [B,Lt]  (nullable)
 *          tgt_lse    float [B,Lt]  (nullable; only written if !all_greedy)
 *          row_status uint32[B]     flags OR-ed into existing content
 * workspace: at least dsp_verify_workspace_bytes(...) bytes, 256-byte aligned.
 * Errors : INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 */
int32_t dsp_verify_workspace_bytes(int32_t B, int32_t L, int32_t Lt, int32_t V, int32_t dtype,
                                   size_t *bytes /* host, out */);

int32_t dsp_verify(const void *target_logits, int32_t dtype,
                   int32_t B, int32_t L, int32_t Lt, int32_t V,
                   int64_t tstride_b, int64_t tstride_l,
                   const void *draft_logits, int64_t dstride_b, int64_t dstride_l,
                   const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                   const float *cand_logit, const double *draft_lse64, int32_t KC,
                   int32_t all_greedy, const uint8_t *mode, const float *u, int32_t eos_id,
                   int32_t *accepted_len, int32_t *next_token, float *ratio,
                   int32_t *tgt_argmax, float *tgt_lse, uint32_t *row_status,
                   void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * One whole step in one call  (Alg. 1 stages 1-3 on logits)
 *
 * dsp_lattice_build, dsp_cps_search and dsp_verify with the arguments and
 * results of the three calls (KC = K_max + (eos_id >= 0 ? 1 : 0); row_status is
 * overwritten by the lattice part and OR-ed into by the others; every output of
 * the three calls is written, nullable ones as there).  The one call lets the
 * pass over the target logits, which needs only those, run beside the lattice
 * build and the path search, one side on `stream` and the other on a second
 * stream of the library (of the highest priority the device has; on large
 * inputs it carries the build and the search, otherwise the target pass); the
 * decisions wait for both.  All work is ordered after what was enqueued on
 * `stream` before the call, and work enqueued on `stream` after it is ordered
 * after all of it.
 * The second stream and two events are created at the first call on each
 * device and kept until the process exits (host-side handles; no device
 * memory is allocated).  Calls from several host threads are safe: the
 * library holds a lock while one call enqueues its work.
 * lattice_workspace / verify_workspace: as for dsp_lattice_build / dsp_verify.
 * Errors: those of the three calls.
 */
int32_t dsp_draft_verify_step(
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
    void *verify_workspace, size_t verify_workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Lattice of a vocabulary-sharded drafter head  (Sec. 3.2 "Lattice and
 * pruning", Eq. 7, Eq. 9, computed from slices of the vocabulary; the paper
 * runs one GPU, a tensor-parallel output layer leaves every GPU one slice).
 *
 * dsp_lattice_shard reduces one slice [B,L,Vs] of the logits, holding the
 * tokens vocab_offset .. vocab_offset+Vs-1, to one record per row:
 *   sums[b,l] : S = sum 2^(x*log2e - c), T = sum 2^(x*log2e - c)*(x*log2e - c)
 *               over the slice, against the slice's reference exponent c (S = 0
 *               if the slice has no finite logit), and the logit of eos_id if
 *               the slice holds that token (NaN otherwise);
 *   keys[b,l,:]: the slice's best min(K_max, Vs) tokens as sortable 64-bit keys
 *               (logit, global token id), best first, 0 = none.
 * The records of all G slices, gathered slice-major into [G,B,L] / [G,B,L,K_max]
 * / [G,B] buffers in local memory (one all-gather of (24 + 8*K_max) bytes per
 * row and slice), go to dsp_lattice_merge, which writes the same outputs as
 * dsp_lattice_build on the whole rows [B,L,V]: identical candidates and counts
 * (integer compares on the keys), sums added in double.  K_max, eos_id must
 * agree between the calls; the slices must tile 0..V-1.
 * Records are plain data but their content is only meaningful to the merge.
 *
 * workspace: dsp_shard_workspace_bytes(B, L, Vs, dtype, K_max) for a slice,
 *            dsp_merge_workspace_bytes(B) for the merge; 256-byte aligned.
 * shard_status uint32 [B] (written): DSP_ROW_TIMEOUT; the merge ORs the slices'
 * flags into row_status and adds DSP_ROW_NONFINITE_INPUT as dsp_lattice_build.
 * Errors : as dsp_lattice_build; INVALID_ARG also for vocab_offset < 0, G < 1;
 *          UNSUPPORTED for G > 1024.
 */
typedef struct dsp_shard_sums {
    double S, T;
    float c;
    float eos_logit;
} dsp_shard_sums;

int32_t dsp_shard_workspace_bytes(int32_t B, int32_t L, int32_t Vs, int32_t dtype, int32_t K_max,
                                  size_t *bytes /* host, out */);
int32_t dsp_lattice_shard(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t Vs,
                          int64_t stride_b, int64_t stride_l, int32_t vocab_offset,
                          int32_t K_max, int32_t eos_id,
                          dsp_shard_sums *sums, uint64_t *keys, uint32_t *shard_status,
                          void *workspace, size_t workspace_bytes, dsp_stream_t stream);
int32_t dsp_merge_workspace_bytes(int32_t B, size_t *bytes /* host, out */);
int32_t dsp_lattice_merge(int32_t G, const dsp_shard_sums *sums, const uint64_t *keys,
                          const uint32_t *shard_status,
                          int32_t B, int32_t L, int32_t V, int32_t K_max, float tau, int32_t eos_id,
                          int32_t *cand_id, float *cand_logit, float *cand_logp,
                          int32_t *cand_count, float *lse, double *lse64, float *entropy,
                          int32_t *gen_len, uint32_t *row_status,
                          void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Verification with a vocabulary-sharded target head  (Sec. 2 Eq. 1, Eq. 2,
 * residual resampling; greedy decoding of Sec. 4 -- dsp_verify computed from
 * slices of the target's vocabulary, as a tensor-parallel verifier leaves them).
 *
 * 1. dsp_target_shard: every GPU reduces its slice [B,Lt,Vs] of the target
 *    logits to one record per row (as dsp_lattice_shard with one key: the
 *    slice's argmax; the record's probe logit is the target logit of the row's
 *    path token if the slice holds that token).  All-gather the records.
 * 2. dsp_verify_merge (every GPU, same result): argmax and log-sum-exp of every
 *    target row from the records, then the acceptance scan exactly as
 *    dsp_verify.  Greedy rows are finished (next_token).  For a stochastic row
 *    that needs a draw, job_trow[b] names the target row (b*Lt + i) to sample
 *    from and job_drow[b] the draft row (b*L + i) of the residual, or -1 for a
 *    bonus draw from p; job_trow[b] = -1: nothing to draw; next_token[b] = -1
 *    until step 3.  tgt_lse64 [B,Lt] (double) is an output the draw needs.
 * 3. The caller gathers, into local memory, the named rows' slices from all
 *    GPUs into whole rows target_rows [B,V] and draft_rows [B,V] (row b = batch
 *    row b's row; rows of batch rows without a job are not read; strides in
 *    elements), and dsp_residual_sample draws next_token[b] as dsp_verify does
 *    (inverse CDF of [p - q]_+ or of p with u[b,L]; DSP_ROW_ZERO_RESIDUAL).
 * The draft side (cand_logit, draft_lse64) comes from the lattice, sharded or
 * not.  Other arguments, outputs, flags and errors as dsp_verify.
 * workspace: dsp_shard_workspace_bytes(B, Lt, Vs, dtype, 1),
 *            dsp_verify_merge_workspace_bytes(B, Lt),
 *            dsp_residual_sample_workspace_bytes(B, V, dtype); 256-byte aligned.
 */
int32_t dsp_target_shard(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t Lt, int32_t Vs,
                         int64_t stride_b, int64_t stride_l, int32_t vocab_offset,
                         const int32_t *path, const int32_t *path_len,
                         dsp_shard_sums *sums, uint64_t *keys /* [B,Lt,1] */, uint32_t *shard_status,
                         void *workspace, size_t workspace_bytes, dsp_stream_t stream);
int32_t dsp_verify_merge_workspace_bytes(int32_t B, int32_t Lt, size_t *bytes /* host, out */);
int32_t dsp_verify_merge(int32_t G, const dsp_shard_sums *sums /* [G,B,Lt] */, const uint64_t *keys /* [G,B,Lt] */,
                         const uint32_t *shard_status /* [G,B] */,
                         int32_t B, int32_t L, int32_t Lt,
                         const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                         const float *cand_logit, const double *draft_lse64, int32_t KC,
                         int32_t all_greedy, const uint8_t *mode, const float *u, int32_t eos_id,
                         int32_t *accepted_len, int32_t *next_token, float *ratio /* nullable */,
                         int32_t *tgt_argmax, float *tgt_lse /* nullable */, double *tgt_lse64,
                         int32_t *job_trow, int32_t *job_drow, uint32_t *row_status,
                         void *workspace, size_t workspace_bytes, dsp_stream_t stream);
int32_t dsp_residual_sample_workspace_bytes(int32_t B, int32_t V, int32_t dtype, size_t *bytes /* host, out */);
int32_t dsp_residual_sample(const void *target_rows, const void *draft_rows, int32_t dtype,
                            int32_t B, int32_t L, int32_t Lt, int32_t V,
                            int64_t tstride, int64_t dstride,
                            const int32_t *job_trow, const int32_t *job_drow,
                            const double *tgt_lse64, const double *draft_lse64,
                            const int32_t *tgt_argmax, const float *u,
                            int32_t *next_token, uint32_t *row_status,
                            void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Several paths in one target pass  (Sec. 2 names tree-based parallel
 * verification as verifier-side engineering; the paper verifies the rank-0
 * path only -- this is the greedy rule of Sec. 4 applied along a token tree of
 * the beams dsp_cps_search leaves in beam_ids).
 *
 * dsp_beam_tree: beams that share a prefix share its nodes.  N = W*L node slots
 * per batch row; nodes are numbered in the order (beam rank, depth) of their
 * first use, so the rank-0 path is nodes 0 .. m-1 (m = path_len[b]).
 *   node_token / node_parent / node_depth int32 [B,N]: token, the node before
 *     it on its path (-1 at depth 0), depth; -1 in unused slots;
 *   beam_node int32 [B,W,L]: node of beam w at depth i, -1 where there is none;
 *   n_nodes int32 [B].
 * The caller runs the target model on the tree (tree attention) and supplies
 * target_logits [B, 1+N, V]: row 0 = the distribution after the prefix, row
 * 1+n = the distribution after node n (rows of unused slots are not read).
 * dsp_verify_tree walks from the root: the argmax (lowest id on ties) of the
 * current row picks the child that carries that token; the walk ends where no
 * child does.  accepted_len [B] = nodes walked, accepted_node int32 [B,L] = the
 * nodes in order (-1 beyond), next_token [B] = the argmax of the row where the
 * walk ended (correction, or bonus after a leaf), tgt_argmax int32 [B,1+N]
 * (-1 for unused rows), row_status (written): DSP_ROW_NONFINITE_INPUT if an
 * existing row holds NaN / +inf or no finite logit, DSP_ROW_TIMEOUT.
 * dsp_verify_tree_stochastic is the stochastic rule along the same tree (Sec. 2:
 * Eq. 1 with residual resampling, in its multi-branch form): the children of the
 * current node are tried in node order; child n with token x is accepted iff
 * u[b,n] < f(x) / q_i(x), where f is the node's current target distribution
 * (softmax of its target row at first) and q_i the softmax of draft row i, i the
 * node's depth (f(x) > 0 = q_i(x) accepts, f(x) = 0 rejects); a rejection replaces
 * f by [f - q_i]_+ / R (R its mass) before the next sibling is tried.  When no
 * child is left (all rejected, a leaf, depth L) next_token is the smallest v with
 * f(v) > 0 and sum_{w<=v} f(w) >= u[b,N] * sum_w f(w); R = 0 gives the argmax of
 * the node's target row and DSP_ROW_ZERO_RESIDUAL.  draft_logits [B,L,V];
 * u float [B,N+1] in [0,1).  At most DSP_MAX_W children of one node are tried (a
 * tree of dsp_beam_tree has no more).  The acceptance test is evaluated in double
 * from the two logits, the rows' log-sum-exp and the residual masses; the sums over
 * a row (log-sum-exp, residual mass, the cumulative sum of the emitted token) add
 * fp32 terms in double in a fixed order: a decision closer than about 1e-6
 * (relative) to going the other way may differ from exact arithmetic.  The draft
 * rows 0 .. min(L, N+1)-1 are read once more than the walk needs them (their
 * log-sum-exp is formed for all batch rows up front).
 * workspace: dsp_verify_tree_workspace_bytes(B, N, V, dtype), 256-byte aligned
 * (one size for both rules).
 * Errors : INVALID_ARG, UNSUPPORTED (W > DSP_MAX_W, L > DSP_MAX_L,
 *          N + 1 > DSP_MAX_L, dtype), WORKSPACE, CUDA.
 */
int32_t dsp_beam_tree(const int32_t *beam_ids, const int32_t *path_len, int32_t B, int32_t W, int32_t L,
                      int32_t *node_token, int32_t *node_parent, int32_t *node_depth,
                      int32_t *beam_node, int32_t *n_nodes, dsp_stream_t stream);
int32_t dsp_verify_tree_workspace_bytes(int32_t B, int32_t N, int32_t V, int32_t dtype,
                                        size_t *bytes /* host, out */);
int32_t dsp_verify_tree_stochastic(const void *target_logits, const void *draft_logits, int32_t dtype,
                                   int32_t B, int32_t N, int32_t L, int32_t V,
                                   int64_t tstride_b, int64_t tstride_l, int64_t dstride_b, int64_t dstride_l,
                                   const int32_t *node_token, const int32_t *node_parent, const int32_t *n_nodes,
                                   const float *u,
                                   int32_t *accepted_len, int32_t *accepted_node, int32_t *next_token,
                                   int32_t *tgt_argmax, uint32_t *row_status,
                                   void *workspace, size_t workspace_bytes, dsp_stream_t stream);
int32_t dsp_verify_tree(const void *target_logits, int32_t dtype, int32_t B, int32_t N, int32_t V,
                        int64_t stride_b, int64_t stride_l,
                        const int32_t *node_token, const int32_t *node_parent, const int32_t *n_nodes,
                        int32_t L, int32_t *accepted_len, int32_t *accepted_node, int32_t *next_token,
                        int32_t *tgt_argmax, uint32_t *row_status,
                        void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * Refinement step of the diffusion drafter  (Sec. 3.1, Eq. 5: iterative
 * refinement with the update set "top-K by confidence"; the paper's default
 * S = 1 needs a single call with n_update >= L, S > 1 is its ablation).
 *
 * logits [B,L,V] are the drafter's per-position conditionals for the block at
 * this refinement step.  For every position i of batch row b with
 * masked[b,i] != 0:
 *   a_i    = argmax_v x[b,i,v]            (lowest id on ties)
 *   conf_i = log q(a_i) = x_max - lse     (fp32; positions are compared in fp32)
 * The min(n_update, #masked) masked positions of largest conf (equal conf: the
 * lower position first) are revealed: tokens[b,i] = a_i, masked[b,i] = 0.
 * Rows of positions that are already revealed are not read.
 *
 * Inputs : logits (dtype, strides in elements, as for dsp_lattice_build);
 *          n_update >= 1.
 * In/out : tokens int32 [B,L], masked uint8 [B,L] (entries of revealed
 *          positions are left as they are).
 * Outputs: argmax int32 [B,L], confidence float [B,L]: a_i and conf_i of the
 *          positions masked on entry, -1 and -inf elsewhere;
 *          n_left int32 [B] = positions still masked on return;
 *          row_status uint32 [B] (written): DSP_ROW_NONFINITE_INPUT if a masked
 *          row holds NaN / +inf or no finite logit (that position takes
 *          conf = -inf; the batch row's outputs are then unspecified but in
 *          bounds), DSP_ROW_TIMEOUT.
 * workspace: dsp_unmask_workspace_bytes(B, L, V, dtype), 256-byte aligned.
 * Errors : INVALID_ARG (null pointer, sizes, strides, n_update < 1,
 *          alignment), UNSUPPORTED (dtype, L > DSP_MAX_L, V > 2^30), WORKSPACE,
 *          CUDA.
 */
int32_t dsp_unmask_workspace_bytes(int32_t B, int32_t L, int32_t V, int32_t dtype,
                                   size_t *bytes /* host, out */);
int32_t dsp_unmask_step(const void *logits, int32_t dtype, int32_t B, int32_t L, int32_t V,
                        int64_t stride_b, int64_t stride_l, int32_t n_update,
                        int32_t *tokens, uint8_t *masked, int32_t *argmax, float *confidence,
                        int32_t *n_left, uint32_t *row_status,
                        void *workspace, size_t workspace_bytes, dsp_stream_t stream);

/* -------------------------------------------------------------------------
 * A step recorded as a CUDA graph  (Alg. 1 stages 1-3 replayed; the draft
 * length changes between steps by Eq. 11, over few values: one graph each).
 *
 * dsp_step_graph_create records one dsp_draft_verify_step call (same
 * arguments, no stream) as a CUDA graph and returns a handle (host object,
 * owned by the caller until dsp_step_graph_destroy).  Nothing runs at creation.
 * dsp_step_graph_launch replays it on `stream`: same kernels, same results as
 * the direct call, with the host's launch work of two memsets and up to seven
 * kernels on two streams replaced by one graph launch.  The graph holds the
 * addresses, sizes and scalar arguments given at creation: keep every buffer
 * alive and in place while the handle lives, refresh inputs in place, and
 * order launches that share buffers or workspaces (same stream).  One graph
 * per draft length L (and per set of buffers); graphs of different L may
 * share input buffers (strides) and workspaces sized for the largest L.
 * Creation allocates (CUDA's graph objects), must not overlap another thread's
 * dsp_draft_verify_step on the same device, and is refused (UNSUPPORTED)
 * while events are set through dsp_profile_events.
 * Errors : create: those of dsp_draft_verify_step, INVALID_ARG (out is null),
 *          CUDA; launch: INVALID_ARG (null handle), CUDA; destroy: CUDA (a null
 *          handle is fine).
 */
typedef struct dsp_step_graph dsp_step_graph;

int32_t dsp_step_graph_create(
    dsp_step_graph **out /* host, out */,
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
    void *verify_workspace, size_t verify_workspace_bytes);
int32_t dsp_step_graph_launch(dsp_step_graph *graph, dsp_stream_t stream);
int32_t dsp_step_graph_destroy(dsp_step_graph *graph);

/* -------------------------------------------------------------------------
 * Adaptive draft length  (Sec. 3.3, Eq. 9-11; Alg. 1 init and stage 4) -- host.
 *
 * State is plain data owned by the caller (copy it to checkpoint it).
 *   init  : both moving averages 0, k = k_max.
 *   update: ema = (1-rho)*ema + rho*signal for the batch means of gen_len and
 *           accepted_len (batch 1 is the paper's setting), then
 *           k = clip(ceil(ema_gen + delta * [ema_acc >= ema_gen]), k_min, k_max),
 *           the ceiling first rounded up to a multiple of `granularity`
 *           (1 = the paper's rule).  All arithmetic in double.
 * accepted_len / gen_len are HOST pointers (the caller copies the two [B]
 * arrays back; that copy is the step's only device-to-host traffic).
 * Errors : INVALID_ARG (null pointer, B < 1, k_min < 1, k_min > k_max,
 *          rho outside (0,1], delta < 0, granularity < 1).
 */
typedef struct dsp_adl_params {
    int32_t k_min, k_max;
    double delta;
    double rho;
    int32_t granularity;
} dsp_adl_params;

typedef struct dsp_adl_state {
    double ema_gen, ema_acc;
    int32_t k;        /* draft length for the next step */
    int32_t steps;    /* updates so far */
} dsp_adl_state;

int32_t dsp_adl_init(dsp_adl_state *state, const dsp_adl_params *params);
int32_t dsp_adl_update(dsp_adl_state *state, const dsp_adl_params *params,
                       const int32_t *accepted_len, const int32_t *gen_len, int32_t B,
                       int32_t *next_L /* host, out, nullable */);

/* -------------------------------------------------------------------------
 * Breadth controller, host side  (Sec. 6, future work iii: joint control of
 * draft length and search / pruning breadth; the paper gives no rule, this
 * is the library's: the moving averages of Eq. 10 on two more signals)
 *
 * Per step, from the lattice build's entropy output and the two lengths that
 * dsp_adl_update takes (batch means; all pointers are HOST pointers):
 *   H = mean over batch rows b and positions i < max(1, gen_len[b]) of
 *       entropy[b,i]                                             (nats)
 *   s = mean over b of max(0, gen_len[b] - accepted_len[b]) / max(1, gen_len[b])
 *   ema = (1-rho) * ema + rho * signal            (both start at 0)
 *   K' = clip( ceil( exp(ema_H) ), K_min, K_max )  candidates per position for
 *        the next step (the drafter's perplexity)
 *   W' = clip( ceil( W_min + (W_max - W_min) * ema_s ), W_min, W_max )  beam width
 * dsp_breadth_init: averages 0, K = K_max, W = W_max.  All arithmetic in double.
 * entropy: float [B,L] (a host copy of dsp_lattice_build's output).
 * Errors : INVALID_ARG (null pointer, B < 1, L < 1, K_min < 1, K_min > K_max,
 *          K_max > DSP_MAX_K, W likewise with DSP_MAX_W, rho outside (0,1]).
 */
typedef struct dsp_breadth_params {
    int32_t K_min, K_max, W_min, W_max;
    double rho;
} dsp_breadth_params;

typedef struct dsp_breadth_state {
    double ema_entropy, ema_shortfall;
    int32_t K, W;     /* candidate cap and beam width for the next step */
    int32_t steps;    /* updates so far */
} dsp_breadth_state;

int32_t dsp_breadth_init(dsp_breadth_state *state, const dsp_breadth_params *params);
int32_t dsp_breadth_update(dsp_breadth_state *state, const dsp_breadth_params *params,
                           const float *entropy, const int32_t *accepted_len, const int32_t *gen_len,
                           int32_t B, int32_t L,
                           int32_t *next_K /* host, out, nullable */, int32_t *next_W /* host, out, nullable */);

#ifdef __cplusplus
}
#endif
#endif /* DSP_H_ */
