// dsp_cps_search: causal-consistency path search (Sec. 3.2 "Scoring and search", Eq. 8).
//
// One CTA per batch row walks the lattice left to right.  The step score of a candidate,
//   step = fl( fl(lambda * (x - x_top1)) + fl((1 - lambda) * l^ng(prev, cur)) ),
// (with a verifier-side score per candidate slot, dsp_cps_search_biased: fl(step + fl(mu * l^ver)))
// depends on the previous position's candidate slot and on its own slot but not on the beam, so
// for a window of depths the causal scores of all (depth, previous slot, slot) are gathered in
// parallel (asynchronous 4-byte copies straight into shared memory: one round trip however many
// entries a thread has) before the depths of the window are walked; the sequential part of a
// depth is then two shared-memory reads and three fp32 operations per expansion and the selection
// of the best W.  The work of a depth is bound by the latency of its instructions, not by their
// number of lanes: beams of up to 96 expansions are walked by one warp alone (no block barrier, no
// shared-memory atomic between depths), larger ones by the whole CTA.
// Expansions become unique 64-bit keys (cum | token-id rank | parent rank | slot) whose integer
// order is the beam order (cum desc, token id asc, parent rank asc).  The best W are found by
// pruning and ranking, not sorting: an expansion below the worst of the beams' own best
// expansions cannot be among the best W and is dropped; the few that remain count the keys
// above them (all pairs); the keys are unique, so the ranks below W name one key each.
// Back-pointers stay in shared memory; each surviving beam's slots are recovered by walking them
// and the token ids are then read by all threads at once (from shared memory if the search had
// one window).
#include "dsp_common.cuh"
#include "dsp_internal.h"

namespace dsp {

constexpr int kMaxKC = DSP_MAX_K + 1;
constexpr int kStepBudgetBytes = 48 * 1024;        // shared memory for one window of depths

struct CpsArgs {
    const int32_t *cand_id;
    const float *cand_logit;
    const double *lse64;
    const int32_t *cand_count;
    int B, L, KC;
    const int32_t *prev_token;
    int proxy_kind;
    const float *table;
    int table_log2;
    uint32_t hash_seed;
    int V;
    int W;
    float lambda;
    int eos_id;
    const float *ver_score;      // [B,L,KC] or null: the verifier-side term of the step score
    float mu;
    int32_t *path, *path_slot, *path_len;
    float *path_score;
    int32_t *beam_ids;
    float *beam_score, *beam_cum;
    uint32_t *row_status;
    int D;                       // depths per window
    int ver;                     // 1: ver_score is given
    int SW;                      // step-table entries per depth: KC * KC, or KC for the trigram proxy
};

// Depths per window and dynamic shared memory of a launch (SW = step-table entries per depth).
inline int cps_window_depths(int L, int KC, int SW, bool ver) {
    int d = kStepBudgetBytes / (SW * 4 + KC * (ver ? 21 : 17) + 16);   // everything a depth keeps in shared memory
    if (d < 1) d = 1;
    return d < L ? d : L;
}
inline size_t cps_smem_bytes(int L, int W, int KC, int D, int SW, bool ver) {
    size_t o = align_up((size_t)3 * L * W, 16);                 // back-pointers and walked slots
    o += (size_t)D * 8;                                         // log-sum-exp of each position (double)
    o += (size_t)D * SW * 4;                                    // step scores
    o += (size_t)(D + 1) * KC * 4;                              // candidate ids (and the depth before the window)
    o += (size_t)D * KC * 4;                                    // candidate logits
    o += (size_t)D * KC * 4 * (ver ? 2 : 1);                    // the drafter's and the verifier's weighted terms
    o += (size_t)(D + 1) * 4 + (size_t)D * 4;                   // candidate counts, their division constants
    o += (size_t)D * KC * 4;                                    // best step score after each previous slot
    o += align_up((size_t)D * KC, 4);                           // token-id ranks
    return o;
}

// Bigram proxies: the dense [V,V] table or the hashed table (the mix is part of the ABI).
__device__ __forceinline__ const float *proxy_entry(const CpsArgs &a, int prev, int cur) {
    if (a.proxy_kind == 1)                                   // ids outside [0, V) read the nearest row / column
        return &a.table[(long long)min(max(prev, 0), a.V - 1) * a.V + min(max(cur, 0), a.V - 1)];
    uint32_t h = (uint32_t)prev * 0x9E3779B1u;
    h ^= (uint32_t)cur + a.hash_seed;
    h *= 0x9E3779B1u;
    h ^= h >> 15;
    h *= 0x9E3779B1u;
    h ^= h >> 13;
    return &a.table[h >> (32 - a.table_log2)];
}
// One 4-byte asynchronous copy from global to shared memory (no register in between, so a thread
// can have any number of them in flight), and the wait for all copies this thread has issued.
__device__ __forceinline__ void copy4_async(void *dst_shared, const void *src_global) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)),
                 "l"(__cvta_generic_to_global(src_global))
                 : "memory");
}
__device__ __forceinline__ void copies_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Hashed trigram proxy (the mix is part of the ABI).
__device__ __forceinline__ float trigram_score(const CpsArgs &a, int prev2, int prev, int cur) {
    uint32_t g = (uint32_t)prev2 * 0xC2B2AE35u;
    g ^= g >> 16;
    uint32_t h = ((uint32_t)prev ^ g) * 0x9E3779B1u;
    h ^= (uint32_t)cur + a.hash_seed;
    h *= 0x9E3779B1u;
    h ^= h >> 15;
    h *= 0x9E3779B1u;
    h ^= h >> 13;
    return __ldg(&a.table[h >> (32 - a.table_log2)]);
}

constexpr int kMaxExpansions = DSP_MAX_W * kMaxKC;        // expansions of one depth

// floor(x / d) as a multiplication: m = floor(2^32 / d) + 1 is exact while x * d < 2^32
// (here x < 2^16 and d <= 33^2).
__device__ __forceinline__ unsigned long long div_magic(int d) { return (1ull << 32) / (unsigned)d + 1ull; }
__device__ __forceinline__ int div_by(int x, unsigned long long m) { return (int)(((unsigned long long)(unsigned)x * m) >> 32); }

// TRI: the hashed trigram proxy.  Its score depends on the beam's last two tokens, so it cannot be
// tabulated per window: every expansion gathers its own score in the depth loop (one more memory
// round trip per depth), the beams' best expansions are found with shared-memory atomics, and one
// more block barrier separates them from the pruning.
// EPL > 0: the beam is small enough (W * KC <= 32 * EPL) for one warp to hold every expansion of a
// depth, EPL per lane.  That warp then walks the depths of a window alone, with no block-wide
// barrier and no shared-memory atomic between them (the pruning floor and the best token travel by
// warp reductions), while the other warps wait for the end of the window; the work of a depth is
// too small to pay for two barriers among eight warps.
template <bool TRI, int EPL>
__global__ void __launch_bounds__(kThreads) cps_kernel(const CpsArgs a) {
    extern __shared__ __align__(16) unsigned char dyn[];
    // keys that can still be among the best W: two buffers in turn, the one not in use is zeroed
    // meanwhile, so that the slots after the last key read as "below every key"
    __shared__ __align__(16) unsigned long long surv[2][kMaxExpansions + 8];
    __shared__ float bcum[2][DSP_MAX_W];
    __shared__ int bslot[2][DSP_MAX_W];                // slot of each beam's last token
    __shared__ uint32_t s_floor[2];                    // smallest ord_bits among the beams' own best expansions
    __shared__ int s_nsurv[2];                         // survivors of this depth / of the next (in turn)
    __shared__ int s_top_tok;                          // token of the rank-0 survivor
    __shared__ int s_ctl[4];                           // what the walking warp hands back: m, stopped, live, cur
    // trigram proxy only: every expansion's key, each beam's last two tokens, each beam's best expansion
    __shared__ unsigned long long tkeys[TRI ? kMaxExpansions : 1];
    __shared__ int btok[2][TRI ? DSP_MAX_W : 1], btok2[2][TRI ? DSP_MAX_W : 1];
    __shared__ __align__(16) uint32_t tbest[2][TRI ? DSP_MAX_W : 4];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const int L = a.L, W = a.W, KC = a.KC, D = a.D;
    unsigned char *bp_parent = dyn;
    unsigned char *bp_slot = dyn + (size_t)L * W;
    unsigned char *walk = dyn + (size_t)2 * L * W;     // slot of beam w at depth i, after the walk
    double *slse = reinterpret_cast<double *>(dyn + align_up((size_t)3 * L * W, 16));
    float *step = reinterpret_cast<float *>(slse + D);
    int *cid = reinterpret_cast<int *>(step + (size_t)D * a.SW);   // row 0: the depth before the window
    float *clg = reinterpret_cast<float *>(cid + (size_t)(D + 1) * KC);
    float *glam = clg + (size_t)D * KC;                               // fl(lambda * (x - x_top1)) of each candidate
    float *vmu = glam + (size_t)D * KC;                               // fl(mu * l^ver) of each candidate, if given
    int *ccnt = reinterpret_cast<int *>(vmu + (a.ver ? (size_t)D * KC : 0));   // entry 0: the depth before the window
    unsigned *cinv = reinterpret_cast<unsigned *>(ccnt + D + 1);
    float *smax = reinterpret_cast<float *>(cinv + D);                // [d][previous slot]: best step score
    unsigned char *trank = reinterpret_cast<unsigned char *>(smax + (size_t)D * KC);
    const float lam = a.lambda;
    const float oml = __fsub_rn(1.0f, lam);
    const long long row0 = (long long)b * L;
    const int KK = KC * KC;
    const unsigned long long mKK = div_magic(KK), mKC = div_magic(KC);
    // The step score of candidate dk = d * KC + k from its causal score: fl( fl(lambda*g) + fl((1-lambda)*n) ),
    // then fl(. + fl(mu*v)) where a verifier-side score is given.
    auto score_at = [&](int dk, float ng) {
        const float st = __fadd_rn(glam[dk], __fmul_rn(oml, ng));
        return a.ver ? __fadd_rn(st, vmu[dk]) : st;
    };

    int live = 1, cur = 0, m = L, turn = 0;
    bool stopped = false;
    if (tid < 2 * DSP_MAX_W) {                          // both beam buffers: in-bounds values everywhere
        (&bcum[0][0])[tid] = 0.f;
        (&bslot[0][0])[tid] = 0;
    }
    if (tid < 2) s_nsurv[tid] = 0;
    if constexpr (TRI) {
        if (tid < 2 * DSP_MAX_W) {
            (&btok[0][0])[tid] = 0;
            (&btok2[0][0])[tid] = 0;
            (&tbest[0][0])[tid] = tid == 0 ? 0u : 0xFFFFFFFFu;      // one live beam at the start
        }
    }
    for (int x = tid; x < 2 * (kMaxExpansions + 8); x += kThreads) (&surv[0][0])[x] = 0ull;
    grid_dependency_wait();                            // the lattice is complete from here on
    if constexpr (TRI) {
        if (tid == 0) { btok2[0][0] = a.prev_token[2 * b]; btok[0][0] = a.prev_token[2 * b + 1]; }
    }

    double off = 0.0;                                   // this thread's part of sum_i (lse_i - x_top1,i), i < m
    for (int i0 = 0; i0 < L && m == L && !stopped; i0 += D) {
        const int nd = min(D, L - i0);
        // ---- window set-up: ids, logits and counts; step scores and token-id ranks; best steps ----
        // Everything that is only copied goes from global to shared memory asynchronously, so the
        // set-up costs one round trip for the lattice and one for the causal scores, however many
        // entries a thread handles.
        __syncthreads();
        for (int x = tid; x < nd * KC; x += kThreads) {
            copy4_async(&cid[KC + x], &a.cand_id[(row0 + i0) * KC + x]);
            copy4_async(&clg[x], &a.cand_logit[(row0 + i0) * KC + x]);
            if (a.ver) copy4_async(&vmu[x], &a.ver_score[(row0 + i0) * KC + x]);
        }
        for (int x = tid; x < KC; x += kThreads)
            copy4_async(&cid[x], i0 == 0 ? &a.prev_token[TRI ? 2 * b + 1 : b] : &a.cand_id[(row0 + i0 - 1) * KC + x]);
        for (int x = tid; x < nd; x += kThreads) {
            const int c = max(0, min(a.cand_count[row0 + i0 + x], KC));
            slse[x] = a.lse64[row0 + i0 + x];
            ccnt[1 + x] = c;
            cinv[x] = c > 0 ? 65536u / (unsigned)c + 1u : 0u;       // floor(e / c) = (e * cinv) >> 16 for e < 2048
        }
        if (tid == 0) {
            ccnt[0] = i0 == 0 ? 1 : max(0, min(a.cand_count[row0 + i0 - 1], KC));
            s_floor[cur] = 0xFFFFFFFFu;
        }
        copies_wait_all();
        __syncthreads();
        if constexpr (!TRI) {
            // the causal scores land in the step table as they are; the weighting happens where they are used
            const int total = nd * KK;
#pragma unroll 4
            for (int x = tid; x < total; x += kThreads) {
                const int d = div_by(x, mKK), rem = x - d * KK;
                const int p = div_by(rem, mKC), k = rem - p * KC;
                if (k < ccnt[1 + d] && p < ccnt[d])
                    copy4_async(&step[x], a.proxy_kind == 2 ? &a.table[(row0 + i0) * KK + x]   // [B,L,KC,KC]: x's order
                                                           : proxy_entry(a, cid[d * KC + p], cid[(d + 1) * KC + k]));
            }
        }
        for (int x = tid; x < nd * KC; x += kThreads) {         // meanwhile: the other terms, the rank of each token id
            const int d = div_by(x, mKC), k = x - d * KC;
            int r = 0;
            if (k < ccnt[1 + d]) {
                const int tok = cid[KC + x];
                for (int q = 0; q < ccnt[1 + d]; ++q) r += cid[(d + 1) * KC + q] < tok;
            }
            trank[x] = (unsigned char)r;
            glam[x] = __fmul_rn(lam, __fsub_rn(clg[x], clg[d * KC]));
            if (a.ver) vmu[x] = __fmul_rn(a.mu, vmu[x]);
        }
        copies_wait_all();
        __syncthreads();
        if constexpr (!TRI) {
            for (int x = tid; x < nd * KC; x += kThreads) {     // best step score after previous slot p
                const int d = div_by(x, mKC), p = x - d * KC;
                float best = -CUDART_INF_F;
                if (p < ccnt[d])
                    for (int k = 0; k < ccnt[1 + d]; ++k)
                        best = fmaxf(best, score_at(d * KC + k, step[x * KC + k]));
                smax[x] = best;
            }
            if (EPL == 0 && tid < live) {                       // the beams' best expansions at the window's first depth
                float best = -CUDART_INF_F;
                const int p = bslot[cur][tid];
                for (int k = 0; k < ccnt[1]; ++k)
                    best = fmaxf(best, score_at(k, step[p * KC + k]));
                atomicMin(&s_floor[cur], ord_bits(__fadd_rn(bcum[cur][tid], best)));
            }
        }
        __syncthreads();

        // ---- the depths of the window, one after the other ----
        if constexpr (EPL > 0) {
            if (warp == 0) {
                // the pruning floor of the window's first depth: the smallest of the beams' best expansions
                uint32_t floor_reg;
                {
                    uint32_t mine = 0xFFFFFFFFu;
                    if (lane < live) {
                        float best = -CUDART_INF_F;
                        const int p = bslot[cur][lane];
                        for (int k = 0; k < ccnt[1]; ++k) best = fmaxf(best, score_at(k, step[p * KC + k]));
                        mine = ord_bits(__fadd_rn(bcum[cur][lane], best));
                    }
                    floor_reg = __reduce_min_sync(0xFFFFFFFFu, mine);
                }
                unsigned long long *const sv = surv[0];
                for (int d = 0; d < nd; ++d) {
                    const int i = i0 + d;
                    const int cnt = ccnt[1 + d];
                    const int n = live * cnt;
                    if (n == 0) { m = i; break; }           // an empty position ends the lattice
                    const int keep = min(W, n);
                    const int nxt = cur ^ 1;
                    const uint32_t floor_ord = live >= keep ? floor_reg : 0u;
                    const unsigned inv = cinv[d];
                    // all loads of the lane's expansions first (they are independent), then the compaction
                    unsigned long long key[EPL];
                    bool in[EPL];
#pragma unroll
                    for (int j = 0; j < EPL; ++j) {
                        const int e = lane + 32 * j;
                        const bool valid = e < n;
                        const int ec = valid ? e : 0;
                        const int w = (int)(((unsigned)ec * inv) >> 16), k = ec - w * cnt;
                        const float cum = __fadd_rn(bcum[cur][w], score_at(d * KC + k, step[(d * KC + bslot[cur][w]) * KC + k]));
                        const uint32_t ob = ord_bits(cum);
                        in[j] = valid && ob >= floor_ord;
                        key[j] = ((unsigned long long)ob << 32) | ((unsigned long long)(255 - trank[d * KC + k]) << 24) |
                                 ((unsigned long long)(255 - w) << 16) | ((unsigned long long)(255 - k) << 8) | 1ull;
                    }
                    int S = 0;
#pragma unroll
                    for (int j = 0; j < EPL; ++j) {
                        const unsigned ballot = __ballot_sync(0xFFFFFFFFu, in[j]);
                        if (in[j]) sv[S + __popc(ballot & ((1u << lane) - 1u))] = key[j];
                        S += __popc(ballot);
                    }
                    if (lane < 8) sv[S + lane] = 0ull;      // the ranking reads eight keys a round
                    __syncwarp();
                    uint32_t next_floor = 0xFFFFFFFFu;
                    int top = -1;
                    const ulonglong2 *sp = reinterpret_cast<const ulonglong2 *>(sv);
                    for (int t = lane; t < S; t += 32) {
                        const unsigned long long q = sv[t];
                        int rank = 0;
                        for (int j = 0; j < S; j += 8) {
                            const ulonglong2 v0 = sp[(j >> 1) + 0], v1 = sp[(j >> 1) + 1], v2 = sp[(j >> 1) + 2],
                                             v3 = sp[(j >> 1) + 3];
                            rank += ((v0.x > q ? 1 : 0) + (v0.y > q ? 1 : 0)) + ((v1.x > q ? 1 : 0) + (v1.y > q ? 1 : 0)) +
                                    ((v2.x > q ? 1 : 0) + (v2.y > q ? 1 : 0)) + ((v3.x > q ? 1 : 0) + (v3.y > q ? 1 : 0));
                        }
                        if (rank < keep) {
                            const int w = 255 - (int)((q >> 16) & 0xFF), k = 255 - (int)((q >> 8) & 0xFF);
                            const float cum = ord_value((uint32_t)(q >> 32));
                            if (d + 1 < nd) next_floor = min(next_floor, ord_bits(__fadd_rn(cum, smax[(d + 1) * KC + k])));
                            if (rank == 0) top = cid[(d + 1) * KC + k];
                            bcum[nxt][rank] = cum;
                            bslot[nxt][rank] = k;
                            bp_parent[(size_t)i * W + rank] = (unsigned char)w;
                            bp_slot[(size_t)i * W + rank] = (unsigned char)k;
                        }
                    }
                    floor_reg = __reduce_min_sync(0xFFFFFFFFu, next_floor);
                    const int top_tok = __reduce_max_sync(0xFFFFFFFFu, top);
                    __syncwarp();
                    live = keep;
                    cur = nxt;
                    if (a.eos_id >= 0 && top_tok == a.eos_id) { m = i + 1; stopped = true; break; }
                }
                if (lane == 0) { s_ctl[0] = m; s_ctl[1] = stopped ? 1 : 0; s_ctl[2] = live; s_ctl[3] = cur; }
            }
            __syncthreads();
            m = s_ctl[0]; stopped = s_ctl[1] != 0; live = s_ctl[2]; cur = s_ctl[3];
        } else {
        for (int d = 0; d < nd; ++d, turn ^= 1) {
            const int i = i0 + d;
            const int cnt = ccnt[1 + d];
            const int n = live * cnt;
            if (n == 0) { m = i; break; }               // an empty position ends the lattice
            const int keep = min(W, n);
            const int nxt = cur ^ 1;
            // Every beam's best expansion is one of the n; with `keep` beams or more, the keep-th
            // best expansion is at least the smallest of those, so anything below it is out.
            uint32_t floor_ord = 0u;
            const unsigned inv = cinv[d];
            if constexpr (TRI) {
                // every expansion gathers its causal score; each beam's best expansion by atomicMax
                for (int e = tid; e < n; e += kThreads) {
                    const int w = (int)(((unsigned)e * inv) >> 16), k = e - w * cnt;
                    const float ng = trigram_score(a, btok2[cur][w], btok[cur][w], cid[(d + 1) * KC + k]);
                    const float cum = __fadd_rn(bcum[cur][w], score_at(d * KC + k, ng));
                    const uint32_t ob = ord_bits(cum);
                    atomicMax(&tbest[cur][w], ob);
                    tkeys[e] = ((unsigned long long)ob << 32) | ((unsigned long long)(255 - trank[d * KC + k]) << 24) |
                               ((unsigned long long)(255 - w) << 16) | ((unsigned long long)(255 - k) << 8) | 1ull;
                }
                if (tid < DSP_MAX_W) tbest[nxt][tid] = tid < keep ? 0u : 0xFFFFFFFFu;   // for the next depth
                __syncthreads();
                if (live >= keep) {
                    floor_ord = 0xFFFFFFFFu;
                    const uint4 *tb = reinterpret_cast<const uint4 *>(tbest[cur]);
#pragma unroll
                    for (int j = 0; j < DSP_MAX_W / 4; ++j) {
                        const uint4 v = tb[j];
                        floor_ord = min(min(floor_ord, min(v.x, v.y)), min(v.z, v.w));
                    }
                }
            } else {
                // Every beam's best expansion is one of the n; with `keep` beams or more, the keep-th
                // best expansion is at least the smallest of those, so anything below it is out.
                floor_ord = live >= keep ? s_floor[cur] : 0u;
                if (tid == 0) s_floor[nxt] = 0xFFFFFFFFu;
            }
            for (int e0 = warp * 32; e0 < n; e0 += kThreads) {
                const int e = e0 + lane;
                unsigned long long key = 0ull;
                bool in = false;
                if (e < n) {
                    if constexpr (TRI) {
                        key = tkeys[e];
                        in = (uint32_t)(key >> 32) >= floor_ord;
                    } else {
                        const int w = (int)(((unsigned)e * inv) >> 16), k = e - w * cnt;
                        const float cum = __fadd_rn(bcum[cur][w], score_at(d * KC + k, step[(d * KC + bslot[cur][w]) * KC + k]));
                        const uint32_t ob = ord_bits(cum);
                        in = ob >= floor_ord;
                        key = ((unsigned long long)ob << 32) | ((unsigned long long)(255 - trank[d * KC + k]) << 24) |
                              ((unsigned long long)(255 - w) << 16) | ((unsigned long long)(255 - k) << 8) | 1ull;
                    }
                }
                const unsigned ballot = __ballot_sync(0xFFFFFFFFu, in);
                int base = 0;
                if (lane == 0 && ballot) base = atomicAdd(&s_nsurv[turn], __popc(ballot));
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
                if (in) surv[turn][base + __popc(ballot & ((1u << lane) - 1u))] = key;
            }
            __syncthreads();
            // The survivors are ranked by counting (all pairs; the keys are unique): the ranks
            // below `keep` name the next beams, in order.
            const int S = s_nsurv[turn];
            if (tid == 0) s_nsurv[turn ^ 1] = 0;
            for (int x = tid; x < W * KC + 8; x += kThreads) surv[turn ^ 1][x] = 0ull;
            const ulonglong2 *sp = reinterpret_cast<const ulonglong2 *>(surv[turn]);
            for (int t = tid; t < S; t += kThreads) {
                const unsigned long long q = surv[turn][t];
                int rank = 0;
                for (int j = 0; j < S; j += 8) {            // eight keys a round; the slots after the last key are zero
                    const ulonglong2 v0 = sp[(j >> 1) + 0], v1 = sp[(j >> 1) + 1], v2 = sp[(j >> 1) + 2],
                                     v3 = sp[(j >> 1) + 3];
                    rank += ((v0.x > q ? 1 : 0) + (v0.y > q ? 1 : 0)) + ((v1.x > q ? 1 : 0) + (v1.y > q ? 1 : 0)) +
                            ((v2.x > q ? 1 : 0) + (v2.y > q ? 1 : 0)) + ((v3.x > q ? 1 : 0) + (v3.y > q ? 1 : 0));
                }
                if (rank < keep) {
                    const int w = 255 - (int)((q >> 16) & 0xFF), k = 255 - (int)((q >> 8) & 0xFF);
                    const float cum = ord_value((uint32_t)(q >> 32));    // as added up for the key (-0 reads as +0)
                    bcum[nxt][rank] = cum;
                    bslot[nxt][rank] = k;
                    if constexpr (TRI) {
                        btok2[nxt][rank] = btok[cur][w];
                        btok[nxt][rank] = cid[(d + 1) * KC + k];
                    } else {
                        if (d + 1 < nd) atomicMin(&s_floor[nxt], ord_bits(__fadd_rn(cum, smax[(d + 1) * KC + k])));
                    }
                    bp_parent[(size_t)i * W + rank] = (unsigned char)w;
                    bp_slot[(size_t)i * W + rank] = (unsigned char)k;
                    if (rank == 0) s_top_tok = cid[(d + 1) * KC + k];
                }
            }
            __syncthreads();
            live = keep;
            cur = nxt;
            if (a.eos_id >= 0 && s_top_tok == a.eos_id) { m = i + 1; stopped = true; break; }
        }
        }
        // the window's positions that are on the path: their part of the term Eq. 8 has beyond the ranking
        const int upto = (m == L && !stopped) ? i0 + nd : m;
        for (int x = tid; x < nd && i0 + x < upto; x += kThreads) off += slse[x] - (double)clg[x * KC];
    }
    __syncthreads();

    // ---- outputs ----
    // common term of Eq. 8 dropped from the ranking: lambda * sum_i (lse_i - x_top1,i), in double
    // (the verifier-side term, where given, is part of the ranking quantity already)
    __shared__ double s_off[kWarps];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) off += __shfl_xor_sync(0xFFFFFFFFu, off, o);
    if (lane == 0) s_off[warp] = off;
    // walk the back-pointers (shared memory only), one thread per surviving beam
    const int nlive = live;                            // m == 0: the one empty path, score 0
    if (tid < nlive) {
        int at = tid;
        for (int i = m - 1; i >= 0; --i) {
            walk[(size_t)i * W + tid] = bp_slot[(size_t)i * W + at];
            at = bp_parent[(size_t)i * W + at];
        }
    }
    __syncthreads();
    off = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) off += s_off[w];
    // token ids of every beam: all threads; a search of one window still has every id in shared memory
    const bool one_window = D >= L;
    for (int x = tid; x < W * L; x += kThreads) {
        const int w = x / L, i = x - w * L;
        int id = -1, slot = -1;
        if (w < nlive && i < m) {
            slot = walk[(size_t)i * W + w];
            id = one_window ? cid[(i + 1) * KC + slot] : a.cand_id[(row0 + i) * KC + slot];
        }
        if (a.beam_ids) a.beam_ids[((long long)b * W + w) * L + i] = id;
        if (w == 0) {
            a.path[row0 + i] = id;
            a.path_slot[row0 + i] = slot;
        }
    }
    if (tid < W) {
        const int w = tid;
        float score = -CUDART_INF_F, cumv = -CUDART_INF_F;
        if (w < nlive) {
            cumv = bcum[cur][w];
            score = (float)((double)cumv - (double)lam * off);
        }
        if (a.beam_score) a.beam_score[(long long)b * W + w] = score;
        if (a.beam_cum) a.beam_cum[(long long)b * W + w] = cumv;
        if (w == 0) {
            a.path_len[b] = m;
            a.path_score[b] = score;
            if (a.row_status && stopped) atomicOr(&a.row_status[b], DSP_ROW_EOS_STOPPED);
        }
    }
}

}  // namespace dsp

using namespace dsp;

int32_t dsp::cps_search_impl(const int32_t *cand_id, const float *cand_logit,
                                  const double *lse64, const int32_t *cand_count,
                                  int32_t B, int32_t L, int32_t KC,
                                  const int32_t *prev_token,
                                  int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
                                  uint32_t hash_seed, int32_t V,
                                  int32_t W, float lambda, int32_t eos_id,
                                  const float *ver_score, float mu,
                                  int32_t *path, int32_t *path_slot, int32_t *path_len,
                                  float *path_score,
                                  int32_t *beam_ids, float *beam_score, float *beam_cum,
                                  uint32_t *row_status, cudaStream_t stream) {
    if (B < 0 || L < 1 || KC < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (W < 1 || W > DSP_MAX_W || KC > DSP_MAX_K + 1 || L > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    if (proxy_kind < 0 || proxy_kind > 3) return DSP_ERR_UNSUPPORTED;
    if ((proxy_kind == 0 || proxy_kind == 3) && (table_log2 < 1 || table_log2 > 31)) return DSP_ERR_INVALID_ARG;
    if (!(lambda >= 0.f && lambda <= 1.f)) return DSP_ERR_INVALID_ARG;
    if (ver_score && !(fabsf(mu) <= 3.0e38f)) return DSP_ERR_INVALID_ARG;      // NaN or infinite weight
    if (B == 0) return DSP_OK;
    if (!cand_id || !cand_logit || !lse64 || !cand_count || !prev_token || !proxy_table || !path ||
        !path_slot || !path_len || !path_score)
        return DSP_ERR_INVALID_ARG;

    CpsArgs a;
    a.cand_id = cand_id; a.cand_logit = cand_logit; a.lse64 = lse64; a.cand_count = cand_count;
    a.B = B; a.L = L; a.KC = KC;
    a.prev_token = prev_token;
    a.proxy_kind = proxy_kind; a.table = proxy_table; a.table_log2 = table_log2;
    a.hash_seed = hash_seed; a.V = V; a.W = W; a.lambda = lambda; a.eos_id = eos_id;
    a.ver_score = ver_score; a.mu = mu; a.ver = ver_score != nullptr;
    a.path = path; a.path_slot = path_slot; a.path_len = path_len; a.path_score = path_score;
    a.beam_ids = beam_ids; a.beam_score = beam_score; a.beam_cum = beam_cum;
    a.row_status = row_status;
    const bool tri = proxy_kind == 3;
    a.SW = tri ? KC : KC * KC;
    a.D = cps_window_depths(L, KC, a.SW, a.ver != 0);
    const size_t dyn = cps_smem_bytes(L, W, KC, a.D, a.SW, a.ver != 0);
    {
        // raise the kernels' dynamic shared memory limit once per device (the attribute is per device)
        static bool done[64] = {};
        int dev = 0;
        DSP_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64 || !done[dev]) {
            // largest request of any shape: the back-pointers of the longest, widest search and a full
            // window (a window's arrays fill the budget up to one depth's worth of rounding)
            int most = (int)(align_up((size_t)3 * DSP_MAX_L * DSP_MAX_W, 16) + kStepBudgetBytes +
                             (size_t)kMaxKC * 8 + 64);
            for (void (*k)(CpsArgs) : {cps_kernel<false, 0>, cps_kernel<false, 1>, cps_kernel<false, 2>, cps_kernel<false, 3>,
                                       cps_kernel<true, 0>})
                DSP_CUDA_TRY(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, most));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    const int epl = (W * KC + 31) / 32;                 // expansions per lane if one warp took a whole depth
    void (*kernel)(CpsArgs) = tri        ? cps_kernel<true, 0>
                              : epl == 1 ? cps_kernel<false, 1>
                              : epl == 2 ? cps_kernel<false, 2>
                              : epl == 3 ? cps_kernel<false, 3>
                                         : cps_kernel<false, 0>;
    DSP_CUDA_TRY(launch_dependent(kernel, (unsigned)B, kThreads, dyn, stream, a,
                                  true));
    return DSP_OK;
}

extern "C" int32_t dsp_cps_search(const int32_t *cand_id, const float *cand_logit,
                                  const double *lse64, const int32_t *cand_count,
                                  int32_t B, int32_t L, int32_t KC,
                                  const int32_t *prev_token,
                                  int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
                                  uint32_t hash_seed, int32_t V,
                                  int32_t W, float lambda, int32_t eos_id,
                                  int32_t *path, int32_t *path_slot, int32_t *path_len,
                                  float *path_score,
                                  int32_t *beam_ids, float *beam_score, float *beam_cum,
                                  uint32_t *row_status, dsp_stream_t stream) {
    return cps_search_impl(cand_id, cand_logit, lse64, cand_count, B, L, KC, prev_token, proxy_kind, proxy_table,
                           table_log2, hash_seed, V, W, lambda, eos_id, nullptr, 0.f, path, path_slot, path_len,
                           path_score, beam_ids, beam_score, beam_cum, row_status,
                           reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int32_t dsp_cps_search_biased(const int32_t *cand_id, const float *cand_logit,
                                         const double *lse64, const int32_t *cand_count,
                                         int32_t B, int32_t L, int32_t KC,
                                         const int32_t *prev_token,
                                         int32_t proxy_kind, const float *proxy_table, int32_t table_log2,
                                         uint32_t hash_seed, int32_t V,
                                         int32_t W, float lambda, int32_t eos_id,
                                         const float *ver_score, float mu,
                                         int32_t *path, int32_t *path_slot, int32_t *path_len,
                                         float *path_score,
                                         int32_t *beam_ids, float *beam_score, float *beam_cum,
                                         uint32_t *row_status, dsp_stream_t stream) {
    return cps_search_impl(cand_id, cand_logit, lse64, cand_count, B, L, KC, prev_token, proxy_kind, proxy_table,
                           table_log2, hash_seed, V, W, lambda, eos_id, ver_score, mu, path, path_slot, path_len,
                           path_score, beam_ids, beam_score, beam_cum, row_status,
                           reinterpret_cast<cudaStream_t>(stream));
}
