// dsp_lattice_build: draft logits -> token lattice (Sec. 3.2 "Lattice and pruning", Eq. 7, Eq. 9).
//
// Rows whose layout is 16-byte aligned take one kernel: lattice_scan_kernel streams every row
// slice once from HBM (one CTA per slice, no block-wide barrier in the loop, see stream_core.cuh)
// and the CTA that is through with a row last adds up the sums, selects the exact top-K
// (row_engine.cuh) and finalises the row; gen_len and row_status, which belong to a batch row,
// are prepared before the kernel and updated by every row (atomicMin / atomicOr).
// Any other layout takes lattice_kernel: one CTA streams one slice element-wise and does the
// top-K on the way; a row split over several CTAs is finished by whichever CTA arrives last
// (atomic ticket): no CTA waits.  In both paths the CTA that finishes the last row of a batch
// row also writes gen_len and row_status.
#include "dsp_internal.h"
#include "lattice_rows.cuh"

namespace dsp {


// Both paths share the zeroed head; the rest is laid out for the element-wise path (partials,
// keys) and for the streaming path (column records and warp sums of rows cut into several
// slices) over the same bytes: a call takes one path.
struct LatticeWs {
    size_t off_row_ticket, off_b_ticket, off_b_status, zero_bytes, off_partials, off_keys;
    RowScratchLayout rs;
    size_t total;
};
static LatticeWs lattice_ws_layout(int64_t B, int64_t L, int nslices, int K) {
    LatticeWs w;
    size_t o = 0;
    w.off_row_ticket = o; o += align_up((size_t)(B * L) * 4, 256);
    w.off_b_ticket = o;   o += align_up((size_t)B * 4, 256);
    w.off_b_status = o;   o += align_up((size_t)B * 4, 256);
    w.zero_bytes = o;
    w.off_partials = o;   o += align_up((size_t)(B * L) * nslices * sizeof(SlicePartial), 256);
    w.off_keys = o;       o += align_up((size_t)(B * L) * nslices * K * 8, 256);
    w.rs = row_scratch_layout(w.zero_bytes, B * L, nslices);
    w.total = o > w.rs.end ? o : w.rs.end;
    return w;
}

template <typename DT, typename SY>
__device__ void lattice_finalise(const LatticeArgs &a, ScanSmem &sm, long long row, int b, const DT *rowp,
                                 float c, double S, double T);

// Everything after the scan of one slice: publish the slice's partial result, let the CTA that
// arrives last merge the row, finalise the row (Eq. 7 count, EOS slot, outputs) and, for the
// last row of a batch row, write gen_len and row_status.  `extra_status` is OR-ed into the
// batch row's status.
template <typename DT, typename SY>
__device__ void lattice_finish(const LatticeArgs &a, ScanSmem &sm, long long row, int slice, int b,
                               const DT *rowp, float c, double S, double T, unsigned extra_status) {
    const int tid = threadIdx.x;
    if (extra_status && tid == 0) atomicOr(&a.b_status[b], extra_status);
    if (a.nslices > 1) {
        SlicePartial *part = a.partials + row * a.nslices;
        unsigned long long *keys = a.keys + (row * a.nslices + slice) * a.K;
        const int nk = sm.cnt;
        if (tid < nk) keys[tid] = sm.cand[tid];
        if (tid == 0) {
            part[slice].S = S; part[slice].T = T; part[slice].c = c; part[slice].nkeys = nk;
        }
        __threadfence();
        SY::sync();
        if (tid == 0) sm.flag = (int)atomicAdd(&a.row_ticket[row], 1u);
        SY::sync();
        if (sm.flag != a.nslices - 1) return;
        __threadfence();
        // last CTA of this row: gather every slice's keys and sums
        if (tid == 0) sm.cnt = 0;
        SY::sync();
        for (int s = 0; s < a.nslices; ++s) {
            const int n = __ldcg(&part[s].nkeys);
            const unsigned long long *ks = a.keys + (row * a.nslices + s) * a.K;
            if (tid < n) sm.cand[s * a.K + tid] = __ldcg(&ks[tid]);
            else if (tid < a.K) sm.cand[s * a.K + tid] = 0ull;     // below every real key
        }
        if (tid == 0) sm.cnt = a.nslices * a.K;
        prune<SY>(sm, a.K);
        if (tid == 0) {
            int n = 0;                                  // drop the padding keys again
            while (n < sm.cnt && sm.cand[n] != 0ull) ++n;
            sm.cnt = n;
            merge_partials(part, a.nslices, c, S, T);
            sm.fin[0] = S; sm.fin[1] = T; sm.redc[0] = c;
        }
        SY::sync();
        S = sm.fin[0]; T = sm.fin[1]; c = sm.redc[0];
    }

    lattice_finalise<DT, SY>(a, sm, row, b, rowp, c, S, T);
}

// Finalise a row from its sorted best keys sm.cand[0 .. sm.cnt) and its whole-row sums (c, S, T):
// log-sum-exp, entropy, Eq. 7 count, EOS slot, candidate outputs; the CTA that finishes the last
// row of a batch row also writes gen_len (Eq. 9) and row_status.
template <typename DT, typename SY>
__device__ void lattice_finalise(const LatticeArgs &a, ScanSmem &sm, long long row, int b, const DT *rowp,
                                 float c, double S, double T) {
    const int tid = threadIdx.x;
    const int nk = sm.cnt;
    double lse, mean_x;
    const bool ok = row_log_stats(c, S, T, lse, mean_x) && nk > 0;
    if (tid < nk) sm.pk[tid] = exp((double)key_value(sm.cand[tid]) - lse);
    SY::sync();
    if (tid == 0) {
        int count = nk;
        if (a.tau > 0.f && a.tau <= 1.f && ok) {       // Eq. 7 on full-vocabulary probabilities
            const double tau = (double)a.tau;
            double cum = 0.0;
            for (int k = 0; k < nk; ++k) {
                cum += sm.pk[k];
                if (cum >= tau) { count = k + 1; break; }
            }
        }
        int eos_slot = -1;
        float eos_x = 0.f;
        if (a.eos_id >= 0 && a.eos_id < a.V) {          // always keep EOS
            bool has = false;
            for (int k = 0; k < count; ++k) has |= key_id(sm.cand[k]) == a.eos_id;
            if (!has) {
                eos_x = Elem<DT>::load1(rowp + a.eos_id);
                if (eos_x > -CUDART_INF_F && eos_x < CUDART_INF_F) eos_slot = count;
            }
        }
        sm.flag = count;
        sm.overflow = eos_slot;
        sm.thr_v = eos_x;
        a.cand_count[row] = count + (eos_slot >= 0 ? 1 : 0);
        if (a.lse) a.lse[row] = (float)lse;
        a.lse64[row] = lse;
        if (a.entropy) a.entropy[row] = (float)(lse - mean_x);
        if (!ok) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    }
    SY::sync();
    if (tid < a.KC) {
        const int count = sm.flag, eos_slot = sm.overflow;
        int id = -1;
        float x = -CUDART_INF_F, lp = -CUDART_INF_F;
        if (tid < count) {
            id = key_id(sm.cand[tid]);
            x = key_value(sm.cand[tid]);
            lp = (float)((double)x - lse);
        } else if (tid == eos_slot) {
            id = a.eos_id;
            x = sm.thr_v;
            lp = (float)((double)x - lse);
        }
        const long long o = row * a.KC + tid;
        a.cand_id[o] = id;
        a.cand_logit[o] = x;
        a.cand_logp[o] = lp;
    }
    // ---- last row of this batch row: generation length (Eq. 9) and status ----
    __threadfence();
    SY::sync();
    if (tid == 0) {
        const unsigned t = atomicAdd(&a.b_ticket[b], 1u);
        if (t == (unsigned)a.L - 1) {
            __threadfence();
            int g = a.L;
            if (a.eos_id >= 0) {
                for (int i = 0; i < a.L; ++i) {
                    if (__ldcg(&a.cand_id[((long long)b * a.L + i) * a.KC]) == a.eos_id) { g = i; break; }
                }
            }
            a.gen_len[b] = g;
            a.row_status[b] = atomicOr(&a.b_status[b], 0u);
        }
    }
}


// Element-wise kernel: any layout (rows need not be 16-byte aligned).
template <typename DT>
__global__ void __launch_bounds__(kThreads, 4) lattice_kernel(const LatticeArgs a) {
    __shared__ ScanSmem sm;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    const int s0 = slice * a.slice_elems;
    const int s1 = min(a.V, s0 + a.slice_elems);
    float c;
    double S, T;
    scan_slice<DT, true>(rowp, s0, s1, a.K, sm, c, S, T);
    lattice_finish<DT, SyncAll>(a, sm, row, slice, b, rowp, c, S, T, 0u);
}

// Streaming path: one CTA per row slice; the CTA that is through with a row last finalises it
// (log-sum-exp, entropy, Eq. 7 count, EOS slot, candidate outputs, its part of gen_len (Eq. 9)
// and row_status).
template <typename DT>
__global__ void __launch_bounds__(kThreads, 3) lattice_scan_kernel(const LatticeArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ StreamBars bars;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.L), l = (int)(row - (long long)b * a.L);
    const DT *rowp = reinterpret_cast<const DT *>(a.logits) + b * a.stride_b + l * a.stride_l;
    stream_begin(bars, a.nstages);
    grid_launch_dependents();
    RowResult r;
    if (!row_engine<DT>(rowp, a.V, a.K, true, row, slice, a.nslices, a.ntiles_row, a.nstages, a.rs, &a.row_status[b],
                        bars, ring, r))
        return;
    warp_finalise_row(a, row, b, l, r.key, r.stats_ok && !r.nonfinite, r.lse, r.mean_x, 0u, threadIdx.x & 31,
                      [&]() { return Elem<DT>::load1(rowp + a.eos_id); });
}

template <typename DT>
static int32_t launch_lattice(LatticeArgs &a, void *workspace, size_t workspace_bytes, cudaStream_t st) {
    const long long nrows = (long long)a.B * a.L;
    const SlicePlan plan = plan_slices<DT>(nrows, a.V, slice_target_ctas());
    a.nslices = plan.nslices;
    a.slice_elems = plan.slice_elems;
    a.ntiles_row = (a.V + tile_elems<DT>() - 1) / tile_elems<DT>();
    const LatticeWs w = lattice_ws_layout(a.B, a.L, a.nslices, a.K);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(workspace);
    a.row_ticket = reinterpret_cast<unsigned *>(ws + w.off_row_ticket);
    a.b_ticket = reinterpret_cast<unsigned *>(ws + w.off_b_ticket);
    a.b_status = reinterpret_cast<unsigned *>(ws + w.off_b_status);
    a.partials = reinterpret_cast<SlicePartial *>(ws + w.off_partials);
    a.keys = reinterpret_cast<unsigned long long *>(ws + w.off_keys);
    a.rs.row_ticket = a.row_ticket;
    a.rs.cols = reinterpret_cast<uint2 *>(ws + w.rs.off_cols);
    a.rs.wpart = reinterpret_cast<WarpPartial *>(ws + w.rs.off_wpart);
    // tickets and status words of the workspace start at zero, row_status at 0, gen_len at L
    PrepareArgs prep;
    prep.zero_a = reinterpret_cast<uint32_t *>(ws); prep.n_a = (long long)(w.zero_bytes / 4);
    prep.zero_b = a.row_status; prep.n_b = a.B;
    prep.fill = a.gen_len; prep.n_fill = a.B; prep.fill_value = a.L;
    DSP_CUDA_TRY(launch_prepare(prep, st));
    const long long nblocks = nrows * a.nslices;
    if (nblocks > 0x7FFFFFFFLL) return DSP_ERR_UNSUPPORTED;
    if (a.nslices <= kMaxSlices && nrows <= 0x7FFFFFFFLL && stream_layout_ok<DT>(a.logits, a.V, a.stride_b, a.stride_l)) {
        static RingSmemDone smem_done;                       // one per element type
        DSP_CUDA_TRY(allow_ring_smem(lattice_scan_kernel<DT>, smem_done));
        a.nstages = ring_stages(nblocks);
        const ProfileEvents pe = g_profile[DSP_PROFILE_LATTICE_SCAN];
        if (pe.start) DSP_CUDA_TRY(cudaEventRecord(pe.start, st));
        // the streaming kernel may start beside the preparation: it waits for it after its rows are streamed
        DSP_CUDA_TRY(launch_dependent(lattice_scan_kernel<DT>, (unsigned)nblocks, kThreads, (size_t)a.nstages * kTileBytes, st, a,
                                      !pe.start));
        if (pe.stop) DSP_CUDA_TRY(cudaEventRecord(pe.stop, st));
    } else {
        lattice_kernel<DT><<<(unsigned)nblocks, kThreads, 0, st>>>(a);
    }
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

template <typename DT>
static size_t lattice_ws_bytes(int B, int L, int V, int K) {
    const SlicePlan plan = plan_slices<DT>((long long)B * L, V, slice_target_ctas());
    return lattice_ws_layout(B, L, plan.nslices, K).total;
}

}  // namespace dsp

using namespace dsp;

static int32_t check_lattice_shape(int32_t B, int32_t L, int32_t V, int32_t dtype, int32_t K_max) {
    if (B < 0 || L < 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (K_max < 1 || K_max > DSP_MAX_K || L > DSP_MAX_L || V > (1 << 30)) return DSP_ERR_UNSUPPORTED;
    return DSP_OK;
}

extern "C" int32_t dsp_lattice_workspace_bytes(int32_t B, int32_t L, int32_t V, int32_t dtype,
                                               int32_t K_max, size_t *bytes) {
    if (!bytes) return DSP_ERR_INVALID_ARG;
    const int32_t rc = check_lattice_shape(B, L, V, dtype, K_max);
    if (rc != DSP_OK) return rc;
    const int K = K_max < V ? K_max : V;
    const int Bq = B > 0 ? B : 1;
    *bytes = dtype == DSP_BF16 ? lattice_ws_bytes<__nv_bfloat16>(Bq, L, V, K)
                               : lattice_ws_bytes<float>(Bq, L, V, K);
    return DSP_OK;
}

int32_t dsp::lattice_build_impl(const void *draft_logits, int32_t dtype,
                                int32_t B, int32_t L, int32_t V,
                                int64_t stride_b, int64_t stride_l,
                                int32_t K_max, float tau, int32_t eos_id,
                                int32_t *cand_id, float *cand_logit, float *cand_logp,
                                int32_t *cand_count, float *lse, double *lse64, float *entropy,
                                int32_t *gen_len, uint32_t *row_status,
                                void *workspace, size_t workspace_bytes, cudaStream_t st) {
    const int32_t rc = check_lattice_shape(B, L, V, dtype, K_max);
    if (rc != DSP_OK) return rc;
    if (B == 0) return DSP_OK;
    if (!draft_logits || !cand_id || !cand_logit || !cand_logp || !cand_count || !lse64 ||
        !gen_len || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (stride_l < V || stride_b < 0 || (B > 1 && stride_b < (int64_t)(L - 1) * stride_l + V))
        return DSP_ERR_INVALID_ARG;
    if (tau != tau) return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(draft_logits) & (es - 1)) != 0) return DSP_ERR_INVALID_ARG;

    LatticeArgs a;
    a.logits = draft_logits;
    a.B = B; a.L = L; a.V = V;
    a.stride_b = stride_b; a.stride_l = stride_l;
    a.K = K_max < V ? K_max : V;
    a.K_max = K_max;
    a.KC = K_max + (eos_id >= 0 ? 1 : 0);
    a.tau = tau;
    a.eos_id = eos_id;
    a.cand_id = cand_id; a.cand_logit = cand_logit; a.cand_logp = cand_logp;
    a.cand_count = cand_count; a.lse = lse; a.lse64 = lse64; a.entropy = entropy;
    a.gen_len = gen_len; a.row_status = row_status;
    return dtype == DSP_BF16 ? launch_lattice<__nv_bfloat16>(a, workspace, workspace_bytes, st)
                             : launch_lattice<float>(a, workspace, workspace_bytes, st);
}

extern "C" int32_t dsp_lattice_build(const void *draft_logits, int32_t dtype,
                                     int32_t B, int32_t L, int32_t V,
                                     int64_t stride_b, int64_t stride_l,
                                     int32_t K_max, float tau, int32_t eos_id,
                                     int32_t *cand_id, float *cand_logit, float *cand_logp,
                                     int32_t *cand_count, float *lse, double *lse64, float *entropy,
                                     int32_t *gen_len, uint32_t *row_status,
                                     void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    return lattice_build_impl(draft_logits, dtype, B, L, V, stride_b, stride_l, K_max, tau, eos_id, cand_id,
                              cand_logit, cand_logp, cand_count, lse, lse64, entropy, gen_len, row_status,
                              workspace, workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

// ---- dsp_lattice_build_static: the same build for callers that cannot allocate ----------------
//
// The scratch workspace lives in this translation unit as a file-scope device array, so a caller
// that has no way to obtain device memory for it (a plug-in running inside a host process whose
// memory pool is closed to it, a callback on a thread where CUDA allocation calls are forbidden,
// code that runs after the memory budget has been handed out) passes only inputs and outputs.
#include <mutex>

namespace {

constexpr size_t kStaticWsBytes = (size_t)DSP_STATIC_WS_BYTES;
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_ws_mutex;
void *g_static_ws_addr[kMaxDevices];    // device address of g_static_ws on each device, 0 = not asked yet

// In host code `g_static_ws` only names the symbol; the address a kernel can use has to be asked
// for, once per device and with that device current.
int32_t static_ws_address(void **out) {
    int dev = -1;
    DSP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return DSP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_ws_mutex);
    if (!g_static_ws_addr[dev]) {
        void *p = nullptr;
        DSP_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_ws));
        if (!p) return dsp::cuda_fail(cudaErrorInvalidSymbol);
        g_static_ws_addr[dev] = p;
    }
    *out = g_static_ws_addr[dev];
    return DSP_OK;
}

}  // namespace

extern "C" int32_t dsp_lattice_build_static(const void *draft_logits, int32_t dtype,
                                            int32_t B, int32_t L, int32_t V,
                                            int64_t stride_b, int64_t stride_l,
                                            int32_t K_max, float tau, int32_t eos_id,
                                            int32_t *cand_id, float *cand_logit, float *cand_logp,
                                            int32_t *cand_count, float *lse, double *lse64,
                                            float *entropy, int32_t *gen_len, uint32_t *row_status,
                                            dsp_stream_t stream) {
    size_t need = 0;
    const int32_t rc = dsp_lattice_workspace_bytes(B, L, V, dtype, K_max, &need);
    if (rc != DSP_OK) return rc;
    if (need > kStaticWsBytes) return DSP_ERR_STATIC_SCRATCH;
    if (B == 0) return DSP_OK;
    void *ws = nullptr;
    const int32_t rs = static_ws_address(&ws);
    if (rs != DSP_OK) return rs;
    // The build zeroes the part of the scratch that must start at zero on `stream` before its
    // kernel runs, so what the previous call left in the array does not matter.
    return dsp_lattice_build(draft_logits, dtype, B, L, V, stride_b, stride_l, K_max, tau, eos_id,
                             cand_id, cand_logit, cand_logp, cand_count, lse, lse64, entropy,
                             gen_len, row_status, ws, kStaticWsBytes, stream);
}
