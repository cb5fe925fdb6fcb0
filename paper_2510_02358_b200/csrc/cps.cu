// dsp_cps_search: causal-consistency path search (Sec. 3.2 "Scoring and search", Eq. 8).
//
// One CTA per batch row walks the lattice left to right.  At each depth the (live beams x
// candidates) expansions are scored in fp32 in a fixed operation order, ranked under
// (cum desc, token id asc, parent rank asc) by counting, and the best W survive with
// back-pointers kept in shared memory; paths are rebuilt by walking the back-pointers.
#include "dsp_common.cuh"

namespace dsp {

constexpr int kMaxExp = DSP_MAX_W * (DSP_MAX_K + 1);

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
};

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

__global__ void __launch_bounds__(kThreads) cps_kernel(const CpsArgs a) {
    extern __shared__ unsigned char bp[];              // [L][W] parent rank, then [L][W] slot
    __shared__ float ecum[kMaxExp];
    __shared__ int etok[kMaxExp];
    __shared__ float bcum[2][DSP_MAX_W];
    __shared__ int btok[2][DSP_MAX_W];
    __shared__ int cid[DSP_MAX_K + 1];
    __shared__ float clg[DSP_MAX_K + 1];

    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    const int L = a.L, W = a.W, KC = a.KC;
    unsigned char *bp_parent = bp;
    unsigned char *bp_slot = bp + (size_t)L * W;
    const float lam = a.lambda;
    const float oml = __fsub_rn(1.0f, lam);

    int live = 1, cur = 0, m = L;
    bool stopped = false;
    if (tid == 0) bcum[0][0] = 0.f;
    __syncthreads();

    for (int i = 0; i < L; ++i) {
        const long long r = (long long)b * L + i;
        int cnt = a.cand_count[r];
        cnt = max(0, min(cnt, KC));
        if (tid < cnt) {
            cid[tid] = a.cand_id[r * KC + tid];
            clg[tid] = a.cand_logit[r * KC + tid];
        }
        __syncthreads();
        const int n = live * cnt;
        if (n == 0) { m = i; break; }                   // an empty position ends the lattice
        const float top1 = clg[0];
        for (int e = tid; e < n; e += kThreads) {
            const int w = e / cnt, k = e - w * cnt;
            const int tok = cid[k];
            const float g = __fsub_rn(clg[k], top1);
            const int prev = i == 0 ? a.prev_token[b] : btok[cur][w];
            const float ng = proxy_score(a, prev, tok);
            const float step = __fadd_rn(__fmul_rn(lam, g), __fmul_rn(oml, ng));
            ecum[e] = __fadd_rn(bcum[cur][w], step);
            etok[e] = tok;
        }
        __syncthreads();
        const int nxt = cur ^ 1;
        for (int e = tid; e < n; e += kThreads) {
            const float s = ecum[e];
            const int tok = etok[e];
            int rank = 0;
            for (int f = 0; f < n; ++f) {
                const float sf = ecum[f];
                const int tf = etok[f];
                rank += (sf > s) || (sf == s && (tf < tok || (tf == tok && f < e)));
            }
            if (rank < W) {
                const int w = e / cnt;
                bcum[nxt][rank] = s;
                btok[nxt][rank] = tok;
                bp_parent[(size_t)i * W + rank] = (unsigned char)w;
                bp_slot[(size_t)i * W + rank] = (unsigned char)(e - w * cnt);
            }
        }
        __syncthreads();
        live = min(W, n);
        cur = nxt;
        if (a.eos_id >= 0 && btok[cur][0] == a.eos_id) { m = i + 1; stopped = true; break; }
    }
    __syncthreads();

    // common term of Eq. 8 dropped from the ranking: lambda * sum_i (lse_i - x_top1,i)
    double off = 0.0;
    for (int i = 0; i < m; ++i) {
        const long long r = (long long)b * L + i;
        off += a.lse64[r] - (double)a.cand_logit[r * KC];
    }
    if (tid < W) {
        const int w = tid;
        const bool alive = w < live && m > 0;
        float score = -CUDART_INF_F, cumv = -CUDART_INF_F;
        if (alive) {
            cumv = bcum[cur][w];
            score = (float)((double)cumv - (double)lam * off);
            int at = w;
            for (int i = m - 1; i >= 0; --i) {
                const int slot = bp_slot[(size_t)i * W + at];
                const int id = a.cand_id[((long long)b * L + i) * KC + slot];
                if (a.beam_ids) a.beam_ids[((long long)b * W + w) * L + i] = id;
                if (w == 0) {
                    a.path[(long long)b * L + i] = id;
                    a.path_slot[(long long)b * L + i] = slot;
                }
                at = bp_parent[(size_t)i * W + at];
            }
        }
        if (a.beam_ids)
            for (int i = alive ? m : 0; i < L; ++i) a.beam_ids[((long long)b * W + w) * L + i] = -1;
        if (a.beam_score) a.beam_score[(long long)b * W + w] = score;
        if (a.beam_cum) a.beam_cum[(long long)b * W + w] = cumv;
        if (w == 0) {
            for (int i = m; i < L; ++i) {
                a.path[(long long)b * L + i] = -1;
                a.path_slot[(long long)b * L + i] = -1;
            }
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
    const size_t dyn = (size_t)L * W * 2;
    static bool attr_set = false;
    if (!attr_set) {
        DSP_CUDA_TRY(cudaFuncSetAttribute(cps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          DSP_MAX_L * DSP_MAX_W * 2));
        attr_set = true;
    }
    cps_kernel<<<B, kThreads, dyn, reinterpret_cast<cudaStream_t>(stream)>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}
