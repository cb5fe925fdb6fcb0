// dsp_cps_search: causal-consistency path search (Sec. 3.2 "Scoring and search", Eq. 8).
//
// One CTA per batch row walks the lattice left to right.  The step score of a candidate,
//   step = fl( fl(lambda * (x - x_top1)) + fl((1 - lambda) * l^ng(prev, cur)) ),
// depends on the previous position's candidate slot and on its own slot but not on the beam, so
// for a window of depths all (depth, previous slot, slot) steps are gathered and computed in
// parallel before the depths of the window are walked; the sequential part of a depth is then
// one shared-memory read and one fp32 add per expansion and the selection of the best W.
// Expansions become unique 64-bit keys (cum | token-id rank | parent rank | slot) whose integer
// order is the beam order (cum desc, token id asc, parent rank asc); every warp sorts 32 keys
// with a bitonic network and the warps' lists are merged pairwise through shared memory.
// Back-pointers stay in shared memory; each surviving beam's slots are recovered by walking them
// and the token ids are then fetched by all threads at once.
#include "dsp_common.cuh"

namespace dsp {

constexpr int kMaxKC = DSP_MAX_K + 1;
constexpr int kStepBudgetBytes = 48 * 1024;        // shared memory for one window of step scores

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
    int32_t *path, *path_slot, *path_len;
    float *path_score;
    int32_t *beam_ids;
    float *beam_score, *beam_cum;
    uint32_t *row_status;
    int D;                       // depths per window
};

// Depths per window and dynamic shared memory of a launch.
inline int cps_window_depths(int L, int KC) {
    int d = kStepBudgetBytes / (KC * KC * 4);
    if (d < 1) d = 1;
    return d < L ? d : L;
}
inline size_t cps_smem_bytes(int L, int W, int KC, int D) {
    size_t o = align_up((size_t)3 * L * W, 16);                 // back-pointers and walked slots
    o += (size_t)D * KC * KC * 4;                               // step scores
    o += (size_t)D * KC * 4;                                    // candidate ids
    o += align_up((size_t)D * KC, 4);                           // token-id ranks
    o += (size_t)D * 4;                                         // candidate counts
    return o;
}

__device__ __forceinline__ float proxy_score(const CpsArgs &a, int prev, int cur) {
    if (a.proxy_kind == 1) return __ldg(&a.table[(long long)prev * a.V + cur]);
    uint32_t h = (uint32_t)prev * 0x9E3779B1u;
    h ^= (uint32_t)cur + a.hash_seed;
    h *= 0x9E3779B1u;
    h ^= h >> 15;
    h *= 0x9E3779B1u;
    h ^= h >> 13;
    return __ldg(&a.table[h >> (32 - a.table_log2)]);
}

__device__ __forceinline__ unsigned long long kmax(unsigned long long a, unsigned long long b) { return a > b ? a : b; }
__device__ __forceinline__ unsigned long long kmin(unsigned long long a, unsigned long long b) { return a < b ? a : b; }

// Sort 32 keys, one per lane, descending over the lanes (bitonic network).
__device__ __forceinline__ unsigned long long sort_keys_desc(unsigned long long v, int lane) {
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
            const bool up = (lane & k) == 0;
            const bool lower = (lane & j) == 0;
            v = (lower == up) ? kmax(v, o) : kmin(v, o);
        }
    }
    return v;
}
// Best 32 of this warp's descending list `a` and another descending list given reversed
// (`b_rev` = the other list's key of lane 31 - lane), descending: the lane-wise maximum is
// bitonic and holds the best 32; five compare-exchange stages sort it.
__device__ __forceinline__ unsigned long long merge_keys(unsigned long long a, unsigned long long b_rev, int lane) {
    unsigned long long v = kmax(a, b_rev);
#pragma unroll
    for (int j = 16; j > 0; j >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, v, j);
        v = (lane & j) == 0 ? kmax(v, o) : kmin(v, o);
    }
    return v;
}

__global__ void __launch_bounds__(kThreads) cps_kernel(const CpsArgs a) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ unsigned long long xch[2][kWarps][32];  // sorted keys of each warp, for the merges (two buffers in turn)
    __shared__ float bcum[2][DSP_MAX_W];
    __shared__ int bslot[2][DSP_MAX_W];                // slot of each beam's last token
    __shared__ int s_top_tok;                          // token of the rank-0 survivor

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;
    const int L = a.L, W = a.W, KC = a.KC, D = a.D;
    unsigned char *bp_parent = dyn;
    unsigned char *bp_slot = dyn + (size_t)L * W;
    unsigned char *walk = dyn + (size_t)2 * L * W;     // slot of beam w at depth i, after the walk
    float *step = reinterpret_cast<float *>(dyn + align_up((size_t)3 * L * W, 16));
    int *cid = reinterpret_cast<int *>(step + (size_t)D * KC * KC);
    unsigned char *trank = reinterpret_cast<unsigned char *>(cid + (size_t)D * KC);
    int *ccnt = reinterpret_cast<int *>(trank + align_up((size_t)D * KC, 4));
    const float lam = a.lambda;
    const float oml = __fsub_rn(1.0f, lam);
    const long long row0 = (long long)b * L;

    int live = 1, cur = 0, m = L;
    bool stopped = false;
    if (tid == 0) { bcum[0][0] = 0.f; bslot[0][0] = 0; }

    for (int i0 = 0; i0 < L && m == L && !stopped; i0 += D) {
        const int nd = min(D, L - i0);
        // ---- window set-up: ids and counts, then step scores and token-id ranks, in parallel ----
        __syncthreads();
        for (int x = tid; x < nd; x += kThreads) ccnt[x] = max(0, min(a.cand_count[row0 + i0 + x], KC));
        for (int x = tid; x < nd * KC; x += kThreads) cid[x] = a.cand_id[(row0 + i0) * KC + x];
        __syncthreads();
        for (int x = tid; x < nd * KC * KC; x += kThreads) {
            const int d = x / (KC * KC), rem = x - d * KC * KC;
            const int p = rem / KC, k = rem - p * KC;
            const int i = i0 + d;
            const int pc = i == 0 ? 1 : (d > 0 ? ccnt[d - 1] : max(0, min(a.cand_count[row0 + i - 1], KC)));
            if (k < ccnt[d] && p < pc) {
                const int prev = i == 0 ? a.prev_token[b]
                                        : (d > 0 ? cid[(d - 1) * KC + p] : a.cand_id[(row0 + i - 1) * KC + p]);
                const float *lg = a.cand_logit + (row0 + i) * KC;
                const float g = __fsub_rn(lg[k], lg[0]);
                const float ng = proxy_score(a, prev, cid[d * KC + k]);
                step[x] = __fadd_rn(__fmul_rn(lam, g), __fmul_rn(oml, ng));
            }
        }
        for (int x = tid; x < nd * KC; x += kThreads) {
            const int d = x / KC, k = x - d * KC;
            int r = 0;
            if (k < ccnt[d]) {
                const int tok = cid[x];
                for (int q = 0; q < ccnt[d]; ++q) r += cid[d * KC + q] < tok;
            }
            trank[x] = (unsigned char)r;
        }
        __syncthreads();

        // ---- the depths of the window, one after the other ----
        for (int d = 0; d < nd; ++d) {
            const int i = i0 + d;
            const int cnt = ccnt[d];
            const int n = live * cnt;
            if (n == 0) { m = i; break; }               // an empty position ends the lattice
            // every warp: its expansions, 32 at a time, sorted and merged into `best`
            unsigned long long best = 0ull;
            for (int base = warp * 32; base < n; base += kThreads) {
                const int e = base + lane;
                unsigned long long key = 0ull;
                if (e < n) {
                    const int w = e / cnt, k = e - w * cnt;
                    const float cum = __fadd_rn(bcum[cur][w], step[(d * KC + bslot[cur][w]) * KC + k]);
                    key = ((unsigned long long)ord_bits(cum) << 32) |
                          ((unsigned long long)(255 - trank[d * KC + k]) << 24) |
                          ((unsigned long long)(255 - w) << 16) | ((unsigned long long)(255 - k) << 8) | 1ull;
                }
                const unsigned long long sorted = sort_keys_desc(key, lane);
                best = base < kThreads ? sorted : merge_keys(best, __shfl_sync(0xFFFFFFFFu, sorted, 31 - lane), lane);
            }
            // pairwise merges of the warps' lists (only as many levels as n needs)
            int buf = 0;
#pragma unroll
            for (int span = 1; span < kWarps; span <<= 1) {
                if (n > 32 * span) {
                    xch[buf][warp][lane] = best;
                    __syncthreads();
                    if ((warp & (2 * span - 1)) == 0) best = merge_keys(best, xch[buf][warp + span][31 - lane], lane);
                    buf ^= 1;                           // the next level writes the other buffer
                }
            }
            // warp 0 holds the best min(32, n) expansions: the first min(W, n) survive
            const int keep = min(W, n);
            const int nxt = cur ^ 1;
            if (warp == 0 && lane < keep) {
                const int w = 255 - (int)((best >> 16) & 0xFF), k = 255 - (int)((best >> 8) & 0xFF);
                bcum[nxt][lane] = __fadd_rn(bcum[cur][w], step[(d * KC + bslot[cur][w]) * KC + k]);
                bslot[nxt][lane] = k;
                bp_parent[(size_t)i * W + lane] = (unsigned char)w;
                bp_slot[(size_t)i * W + lane] = (unsigned char)k;
                if (lane == 0) s_top_tok = cid[d * KC + k];
            }
            __syncthreads();
            live = keep;
            cur = nxt;
            if (a.eos_id >= 0 && s_top_tok == a.eos_id) { m = i + 1; stopped = true; break; }
        }
    }
    __syncthreads();

    // ---- outputs ----
    // common term of Eq. 8 dropped from the ranking: lambda * sum_i (lse_i - x_top1,i), in double
    __shared__ double s_off[kWarps];
    double off = 0.0;
    for (int i = tid; i < m; i += kThreads) off += a.lse64[row0 + i] - (double)a.cand_logit[(row0 + i) * KC];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) off += __shfl_xor_sync(0xFFFFFFFFu, off, o);
    if (lane == 0) s_off[warp] = off;
    // walk the back-pointers (shared memory only), one thread per surviving beam
    const int nlive = m > 0 ? live : 0;
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
    // token ids of every beam: all threads, independent loads
    for (int x = tid; x < W * L; x += kThreads) {
        const int w = x / L, i = x - w * L;
        int id = -1, slot = -1;
        if (w < nlive && i < m) {
            slot = walk[(size_t)i * W + w];
            id = a.cand_id[(row0 + i) * KC + slot];
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
    if (B < 0 || L < 1 || KC < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (W < 1 || W > DSP_MAX_W || KC > DSP_MAX_K + 1 || L > DSP_MAX_L) return DSP_ERR_UNSUPPORTED;
    if (proxy_kind != 0 && proxy_kind != 1) return DSP_ERR_UNSUPPORTED;
    if (proxy_kind == 0 && (table_log2 < 1 || table_log2 > 31)) return DSP_ERR_INVALID_ARG;
    if (!(lambda >= 0.f && lambda <= 1.f)) return DSP_ERR_INVALID_ARG;
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
    a.path = path; a.path_slot = path_slot; a.path_len = path_len; a.path_score = path_score;
    a.beam_ids = beam_ids; a.beam_score = beam_score; a.beam_cum = beam_cum;
    a.row_status = row_status;
    a.D = cps_window_depths(L, KC);
    const size_t dyn = cps_smem_bytes(L, W, KC, a.D);
    {
        // raise the kernel's dynamic shared memory limit once per device (the attribute is per device)
        static bool done[64] = {};
        int dev = 0;
        DSP_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64 || !done[dev]) {
            DSP_CUDA_TRY(cudaFuncSetAttribute(
                cps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                (int)cps_smem_bytes(DSP_MAX_L, DSP_MAX_W, kMaxKC, cps_window_depths(DSP_MAX_L, kMaxKC))));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    cps_kernel<<<B, kThreads, dyn, reinterpret_cast<cudaStream_t>(stream)>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
