// dsp_verify: verification of the chosen path against the target logits
// (Sec. 2: Eq. 1 acceptance, residual resampling, Eq. 2 accepted length; greedy = temperature 0).
//
// Every target row is streamed once (argmax; log-sum-exp terms only for stochastic batch rows):
// 16-byte aligned layouts by target_scan_kernel (one CTA per row slice, no block-wide barrier in
// the loop, see stream_core.cuh; the CTA that is through with a row last takes the argmax and
// adds up the sums, see row_engine.cuh), any other layout by target_kernel (element-wise, slices
// merged by the CTA arriving last).  Every batch row's left-to-right acceptance scan (one warp)
// then either gives the next token (greedy) or a sampling job (stochastic: residual at the first
// rejection, or bonus from row m).  The first part needs only the target logits:
// dsp_draft_verify_step (step.cu) runs it beside the lattice finish and the path search.
// residual_kernel: for each job, one more pass over ONE target row (and ONE draft row):
// per-chunk sums of max(0, p - q) in token order; the CTA arriving last inverts the CDF.
// When every row is greedy the scans run in accept_kernel and that is all; otherwise they run
// inside residual_kernel (each CTA scans its own batch row first): one launch less in the chain.
#include "dsp_internal.h"
#include "row_engine.cuh"

namespace dsp {

struct SampleJob {
    int trow;        // target row index b*Lt + i, or -1: no job
    int drow;        // draft row index b*L + i, or -1: draw from p itself (bonus token)
    float u;
    int fallback;    // target argmax of that row (used when the residual mass is 0); jobs of the
                     // acceptance scan leave it unset: their kernel reads the row's argmax itself
};

struct VerifyArgs {
    const void *target;
    const void *draft;
    int B, L, Lt, V;
    long long tstride_b, tstride_l, dstride_b, dstride_l;
    const int32_t *path, *path_slot, *path_len;
    const float *cand_logit;
    const double *draft_lse64;
    int KC;
    int all_greedy;
    const uint8_t *mode;
    const float *u;
    int eos_id;
    int32_t *accepted_len, *next_token;
    float *ratio;
    int32_t *tgt_argmax;
    float *tgt_lse;
    uint32_t *row_status;
    int nslices, slice_elems;
    // workspace
    unsigned *row_ticket;      // [B*Lt]  zeroed per call
    unsigned *b_ticket;        // [B]     zeroed per call
    unsigned *res_ticket;      // [B]     zeroed per call
    unsigned *b_status;        // [B]     zeroed per call
    SlicePartial *partials;    // [B*Lt, nslices]
    unsigned long long *keys;  // [B*Lt, nslices]
    int32_t *argmax;           // [B*Lt]
    double *tlse64;            // [B*Lt]
    RowScratch rs;             // records of rows cut into several slices (streaming path)
    int ntiles_row;            // tiles of a whole row
    int nstages;               // ring depth of the streaming kernel
    SampleJob *jobs;           // [B]
    double *chunk_sums;        // [B, nchunks]
    int nchunks, res_slices, chunks_per_slice;
    // sharded target head (dsp_verify_merge): the path tokens' target logits come from the slices' records,
    // and the rows to sample from are reported to the caller
    const float *xt_probe;     // [B*Lt] or null
    int32_t *job_trow, *job_drow;   // [B] or null
};

template <typename DT>
__device__ __forceinline__ const DT *trow_ptr(const VerifyArgs &a, long long trow) {
    const long long b = trow / a.Lt, i = trow - b * a.Lt;
    return reinterpret_cast<const DT *>(a.target) + b * a.tstride_b + i * a.tstride_l;
}
template <typename DT>
__device__ __forceinline__ const DT *drow_ptr(const VerifyArgs &a, long long drow) {
    const long long b = drow / a.L, i = drow - b * a.L;
    return reinterpret_cast<const DT *>(a.draft) + b * a.dstride_b + i * a.dstride_l;
}

// Left-to-right acceptance of batch row b by one warp (Eq. 1, Eq. 2).  Returns (in lane 0) the
// sampling job of the row (trow < 0: none); with `write` it also writes the row's outputs
// (without: the same decisions, no side effects: for CTAs that only need the job).
template <typename DT>
__device__ SampleJob accept_row(const VerifyArgs &a, int b, bool write) {
    const int lane = threadIdx.x & 31;
    const int L = a.L, Lt = a.Lt;
    const int m_raw = __ldcg(&a.path_len[b]);
    const bool stoch = !a.all_greedy && a.mode[b] != 0;
    // the first 32 positions' path entries are fetched beside the path length, not after it
    int y_first = -1, slot_first = 0;
    if (lane < L) {
        y_first = __ldcg(&a.path[(long long)b * L + lane]);
        if (stoch) slot_first = __ldcg(&a.path_slot[(long long)b * L + lane]);
    }
    const int m = max(0, min(m_raw, L));
    int acc = m;
    bool eos_seen_before_acc = false;
    for (int i0 = 0; i0 < L; i0 += 32) {
        const int i = i0 + lane;
        bool rej = false;
        float rt_out = -1.f;
        if (i < m) {
            const int y = i0 == 0 ? y_first : __ldcg(&a.path[(long long)b * L + i]);
            if (!stoch) {
                rej = y != __ldcg(&a.argmax[(long long)b * Lt + i]);
            } else {
                const int slot = i0 == 0 ? slot_first : __ldcg(&a.path_slot[(long long)b * L + i]);
                const double xt = a.xt_probe ? (double)__ldcg(&a.xt_probe[(long long)b * Lt + i])
                                             : (double)Elem<DT>::load1(trow_ptr<DT>(a, (long long)b * Lt + i) + y);
                const double xd = (double)__ldcg(&a.cand_logit[((long long)b * L + i) * a.KC + slot]);
                const double lp = xt - __ldcg(&a.tlse64[(long long)b * Lt + i]);
                const double lq = xd - __ldcg(&a.draft_lse64[(long long)b * L + i]);
                const double rt = exp(lp - lq);
                rej = !((double)a.u[(long long)b * (L + 1) + i] < rt);
                rt_out = (float)rt;
            }
        }
        if (write && a.ratio && i < L) a.ratio[(long long)b * L + i] = rt_out;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, rej);
        if (bal && acc == m) acc = i0 + __ffs(bal) - 1;
    }
    if (a.eos_id >= 0) {
        for (int i0 = 0; i0 < acc; i0 += 32) {
            const int i = i0 + lane;
            const bool e = i < acc && __ldcg(&a.path[(long long)b * L + i]) == a.eos_id;
            if (__ballot_sync(0xFFFFFFFFu, e)) eos_seen_before_acc = true;
        }
    }
    SampleJob job;
    job.trow = -1; job.drow = -1; job.u = 0.f; job.fallback = -1;
    if (lane == 0) {
        unsigned status = write ? atomicOr(&a.b_status[b], 0u) : 0u;
        if (eos_seen_before_acc) status |= DSP_ROW_EOS_ACCEPTED;
        int nt = -1;
        const int at = acc < m ? acc : m;              // row the next token comes from
        if (acc < m || m < Lt) {
            if (!stoch) {
                nt = __ldcg(&a.argmax[(long long)b * Lt + at]);
            } else {                                   // the fallback (the row's argmax) is read where it is needed
                job.trow = b * Lt + at;
                job.drow = acc < m ? b * L + at : -1;
                job.u = a.u[(long long)b * (L + 1) + L];
            }
        } else {
            status |= DSP_ROW_NO_BONUS_ROW;
        }
        if (write) {
            a.accepted_len[b] = acc;
            a.next_token[b] = nt;
            if (!a.all_greedy) a.jobs[b] = job;
            if (a.job_trow) { a.job_trow[b] = job.trow; a.job_drow[b] = job.drow; }
            if (status) atomicOr(&a.row_status[b], status);
        }
    }
    return job;
}

template <typename DT, typename SY>
__device__ void target_finish_row(const VerifyArgs &a, ScanSmem &sm, long long row, int b, bool sums,
                                  unsigned long long best, float c, double S, double T);

// Everything after the scan of one slice of a target row: publish the slice's best key and
// sums, let the CTA arriving last finish the row (argmax, log-sum-exp), and let the CTA that
// finishes the last row of a batch row run that row's acceptance scan.
template <typename DT, typename SY>
__device__ void target_finish(const VerifyArgs &a, ScanSmem &sm, long long row, int slice, int b,
                              bool sums, float c, double S, double T, unsigned extra_status) {
    const int tid = threadIdx.x;
    if (extra_status && tid == 0) atomicOr(&a.b_status[b], extra_status);
    unsigned long long best = sm.cnt > 0 ? sm.cand[0] : 0ull;
    if (a.nslices > 1) {
        SlicePartial *part = a.partials + row * a.nslices;
        unsigned long long *keys = a.keys + row * a.nslices;
        if (tid == 0) {
            keys[slice] = best;
            part[slice].S = S; part[slice].T = T; part[slice].c = c; part[slice].nkeys = sm.cnt;
            __threadfence();
            sm.flag = (int)atomicAdd(&a.row_ticket[row], 1u);
        }
        SY::sync();
        if (sm.flag != a.nslices - 1) return;
        __threadfence();
        if (tid == 0) {
            best = 0ull;
            for (int s = 0; s < a.nslices; ++s) {
                const unsigned long long k = __ldcg(&keys[s]);
                best = k > best ? k : best;
            }
            if (sums) merge_partials(part, a.nslices, c, S, T);
        }
    }
    target_finish_row<DT, SY>(a, sm, row, b, sums, best, c, S, T);
}

// A target row is complete (thread 0 holds its best key and, with `sums`, its whole-row sums):
// write argmax and log-sum-exp.
template <typename DT, typename SY>
__device__ void target_finish_row(const VerifyArgs &a, ScanSmem &sm, long long row, int b, bool sums,
                                  unsigned long long best, float c, double S, double T) {
    const int tid = threadIdx.x;
    if (tid == 0) {
        const int am = best ? key_id(best) : 0;
        a.argmax[row] = am;
        if (a.tgt_argmax) a.tgt_argmax[row] = am;
        bool ok = best != 0ull;
        if (sums) {
            double lse, mean_x;
            ok = row_log_stats(c, S, T, lse, mean_x) && ok;
            a.tlse64[row] = lse;
            if (a.tgt_lse) a.tgt_lse[row] = (float)lse;
        } else if (a.tgt_lse && !a.all_greedy) {
            a.tgt_lse[row] = CUDART_NAN_F;             // greedy row of a mixed batch: not computed
        }
        if (!ok) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    }
}


// Element-wise kernel: any layout.
template <typename DT>
__global__ void __launch_bounds__(kThreads, 4) target_kernel(const VerifyArgs a) {
    __shared__ ScanSmem sm;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.Lt);
    const DT *rowp = trow_ptr<DT>(a, row);
    const int s0 = slice * a.slice_elems;
    const int s1 = min(a.V, s0 + a.slice_elems);
    const bool sums = !a.all_greedy && a.mode[b] != 0;
    float c;
    double S, T;
    if (sums) scan_slice<DT, true>(rowp, s0, s1, 1, sm, c, S, T);
    else      scan_slice<DT, false>(rowp, s0, s1, 1, sm, c, S, T);
    target_finish<DT, SyncAll>(a, sm, row, slice, b, sums, c, S, T, 0u);
}

// Streaming path: one CTA per row slice; the CTA that is through with a row last writes its
// argmax (lowest id on ties) and, for a stochastic batch row, its log-sum-exp.
template <typename DT>
__global__ void __launch_bounds__(kThreads, 3) target_scan_kernel(const VerifyArgs a) {
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ StreamBars bars;
    const long long row = blockIdx.x / a.nslices;
    const int slice = blockIdx.x - (int)(row * a.nslices);
    const int b = (int)(row / a.Lt);
    const DT *rowp = trow_ptr<DT>(a, row);
    const bool sums = !a.all_greedy && a.mode[b] != 0;
    stream_begin(bars, a.nstages);
    grid_launch_dependents();
    RowResult r;
    if (!row_engine<DT>(rowp, a.V, 1, sums, row, slice, a.nslices, a.ntiles_row, a.nstages, a.rs, &a.b_status[b], bars,
                        ring, r))
        return;
    if ((threadIdx.x & 31) == 0) {
        const unsigned long long best = r.key;           // lane 0: the row's best key
        const int am = best ? key_id(best) : 0;
        a.argmax[row] = am;
        if (a.tgt_argmax) a.tgt_argmax[row] = am;
        bool ok = best != 0ull && !r.nonfinite;
        if (sums) {
            ok = r.stats_ok && ok;
            a.tlse64[row] = r.lse;
            if (a.tgt_lse) a.tgt_lse[row] = (float)r.lse;
        } else if (a.tgt_lse && !a.all_greedy) {
            a.tgt_lse[row] = CUDART_NAN_F;             // greedy row of a mixed batch: not computed
        }
        if (!ok) atomicOr(&a.b_status[b], DSP_ROW_NONFINITE_INPUT);
    }
}

// The left-to-right acceptance of every batch row (Eq. 1, Eq. 2), one warp per batch row, once
// the target statistics of all rows are there.
template <typename DT>
__global__ void __launch_bounds__(kThreads) accept_kernel(const VerifyArgs a) {
    grid_dependency_wait();                            // target statistics and path are complete from here on
    grid_launch_dependents();
    const int b = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b < a.B) accept_row<DT>(a, b, true);
}

// ---- residual / bonus sampling -------------------------------------------------------------

__device__ __forceinline__ float residual(float xt, float xd, const RowProb &pt, const RowProb &pd, bool has_q) {
    const float p = prob(xt, pt);
    const float q = has_q ? prob(xd, pd) : 0.f;
    const float r = __fsub_rn(p, q);
    return r > 0.f ? r : 0.f;                  // NaN -> 0
}

// ACCEPT: the kernel follows the target statistics directly and every CTA first runs its batch
// row's acceptance scan itself (one warp; the row's first CTA writes the scan's outputs), which
// takes the acceptance kernel and its launch out of the chain; otherwise the jobs are read from
// a.jobs, written by an earlier kernel.
template <typename DT, bool ACCEPT>
__global__ void __launch_bounds__(kThreads, 4) residual_kernel(const VerifyArgs a) {
    constexpr int N = Elem<DT>::N;
    constexpr int CE = 32 * N;                  // elements per chunk: one warp-wide vector load
    __shared__ double s_scan[kThreads];
    __shared__ double s_wtot[kWarps];
    __shared__ double s_total;
    __shared__ int s_found;
    __shared__ int s_flag;
    __shared__ SampleJob s_job;
    grid_dependency_wait();                            // what the kernels before wrote is complete from here on
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / a.res_slices;
    const int rs = blockIdx.x - b * a.res_slices;
    if constexpr (ACCEPT) {
        if (warp == 0) {
            const SampleJob j = accept_row<DT>(a, b, rs == 0);
            if (lane == 0) s_job = j;
        }
        __syncthreads();
    }
    const SampleJob job = ACCEPT ? s_job : a.jobs[b];
    if (job.trow < 0) return;
    const bool has_q = job.drow >= 0;
    const DT *tp = trow_ptr<DT>(a, job.trow);
    const DT *dp = has_q ? drow_ptr<DT>(a, job.drow) : tp;
    const bool aligned = ((reinterpret_cast<uintptr_t>(tp) | reinterpret_cast<uintptr_t>(dp)) & 15) == 0;
    double *sums = a.chunk_sums + (long long)b * a.nchunks;
    const int V = a.V;
    const int c0 = rs * a.chunks_per_slice, c1 = min(a.nchunks, c0 + a.chunks_per_slice);
    constexpr int kChunkBatch = 4;              // chunks whose loads a warp has in flight together
    uint4 vt[kChunkBatch], vd[kChunkBatch];
    auto load_batch = [&](int ch0) {
#pragma unroll
        for (int u = 0; u < kChunkBatch; ++u) {
            const int ch = ch0 + u * kWarps;
            if (ch < c1) {
                const int e0 = ch * CE + lane * N;
                vt[u] = load_vec<DT>(tp, e0, V, aligned);
                vd[u] = has_q ? load_vec<DT>(dp, e0, V, aligned) : vt[u];
            }
        }
    };
    load_batch(c0 + warp);                      // in flight while the rows' constants are fetched and formed
    const double tl = __ldcg(&a.tlse64[job.trow]);
    const double dl = has_q ? __ldcg(&a.draft_lse64[job.drow]) : 0.0;
    const RowProb pt = row_prob(tl);
    const RowProb pd = has_q ? row_prob(dl) : pt;

    for (int ch0 = c0 + warp; ch0 < c1; ch0 += kWarps * kChunkBatch) {
        if (ch0 != c0 + warp) load_batch(ch0);
#pragma unroll
        for (int u = 0; u < kChunkBatch; ++u) {
            const int ch = ch0 + u * kWarps;
            if (ch < c1) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < N; ++e)
                    s = __fadd_rn(s, residual(Elem<DT>::get(vt[u], e), Elem<DT>::get(vd[u], e), pt, pd, has_q));
                const double cs = warp_sum((double)s);
                if (lane == 0) sums[ch] = cs;
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = (int)atomicAdd(&a.res_ticket[b], 1u);
    __syncthreads();
    if (s_flag != a.res_slices - 1) return;
    __threadfence();

    // ---- last CTA of this job: invert the CDF ----
    const int per = (a.nchunks + kThreads - 1) / kThreads;     // consecutive chunks per thread
    const int k0 = min(a.nchunks, tid * per), k1 = min(a.nchunks, k0 + per);
    constexpr int kKept = 4;                    // chunk sums a thread keeps in registers for its second look
    double kept[kKept];
#pragma unroll
    for (int j = 0; j < kKept; ++j) kept[j] = k0 + j < k1 ? __ldcg(&sums[k0 + j]) : 0.0;
    double mine = 0.0;
#pragma unroll
    for (int j = 0; j < kKept; ++j) mine += kept[j];            // k0 + j >= k1: + 0.0, which changes nothing
    for (int k = k0 + kKept; k < k1; ++k) mine += __ldcg(&sums[k]);
    if (tid == 0) s_found = 0x7FFFFFFF;
    // exclusive prefix of the 256 thread sums, in a fixed order: inside each warp, then over the warps
    double tincl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xFFFFFFFFu, tincl, o);
        if (lane >= o) tincl += up;
    }
    const double upto = __shfl_up_sync(0xFFFFFFFFu, tincl, 1);
    if (lane == 31) s_wtot[warp] = tincl;
    __syncthreads();
    double wbase = 0.0;
    for (int w = 0; w < warp; ++w) wbase += s_wtot[w];
    s_scan[tid] = lane == 0 ? wbase : wbase + upto;
    if (tid == kThreads - 1) s_total = wbase + tincl;
    __syncthreads();
    const double R = s_total;
    if (!(R > 0.0)) {
        if (tid == 0) {
            a.next_token[b] = ACCEPT ? __ldcg(&a.argmax[job.trow]) : job.fallback;
            atomicOr(&a.row_status[b], DSP_ROW_ZERO_RESIDUAL);
        }
        return;
    }
    const double thr = (double)job.u * R;
    {
        // The first chunk at which the running sum reaches the threshold; the thread that finds it
        // leaves the sum of everything before that chunk in its slot of s_scan.
        double run = s_scan[tid];
        bool found = false;
#pragma unroll
        for (int j = 0; j < kKept; ++j) {
            if (!found && k0 + j < k1) {
                const double cs = kept[j];
                if (cs > 0.0 && run + cs >= thr) {
                    atomicMin(&s_found, k0 + j);
                    s_scan[tid] = run;
                    found = true;
                }
                run += cs;
            }
        }
        for (int k = k0 + kKept; k < k1 && !found; ++k) {
            const double cs = __ldcg(&sums[k]);
            if (cs > 0.0 && run + cs >= thr) {
                atomicMin(&s_found, k);
                s_scan[tid] = run;
                found = true;
            }
            run += cs;
        }
    }
    __syncthreads();
    int ch = s_found;
    const bool at_top = ch == 0x7FFFFFFF;
    if (at_top) {                               // rounding at the very top: last chunk with mass
        if (tid == 0) {
            int last = -1;
            for (int k = a.nchunks - 1; k >= 0; --k)
                if (__ldcg(&sums[k]) > 0.0) { last = k; break; }
            s_found = last;
        }
        __syncthreads();
        ch = s_found;
    }
    if (warp != 0) return;
    // prefix of everything before chunk ch: as its finder left it, else added up the same way
    double before = 0.0;
    {
        const int owner = min(kThreads - 1, ch / per);
        before = s_scan[owner];
        if (at_top)
            for (int k = owner * per; k < ch; ++k) before += __ldcg(&sums[k]);
    }
    const int e0 = ch * CE + lane * N;
    const uint4 ct = load_vec<DT>(tp, e0, V, aligned);
    const uint4 cd = has_q ? load_vec<DT>(dp, e0, V, aligned) : ct;
    float r[N];
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) {
        r[e] = residual(Elem<DT>::get(ct, e), Elem<DT>::get(cd, e), pt, pd, has_q);
        s = __fadd_rn(s, r[e]);
    }
    // exclusive prefix over lanes (double)
    double incl = (double)s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    double run = before + (incl - (double)s);
    int hit = -1, lastpos = -1;
#pragma unroll
    for (int e = 0; e < N; ++e) {
        run += (double)r[e];
        if (r[e] > 0.f && e0 + e < V) {
            lastpos = e0 + e;
            if (hit < 0 && run >= thr) hit = e0 + e;
        }
    }
    const unsigned bal = __ballot_sync(0xFFFFFFFFu, hit >= 0);
    int tok;
    if (bal) {
        tok = __shfl_sync(0xFFFFFFFFu, hit, __ffs(bal) - 1);
    } else {
        const unsigned bl = __ballot_sync(0xFFFFFFFFu, lastpos >= 0);
        tok = bl ? __shfl_sync(0xFFFFFFFFu, lastpos, 31 - __clz(bl))
                 : (ACCEPT ? __ldcg(&a.argmax[job.trow]) : job.fallback);
    }
    if (lane == 0) a.next_token[b] = tok;
}

struct VerifyWs {
    size_t off_row_ticket, off_b_ticket, off_res_ticket, off_b_status, zero_bytes;
    size_t off_partials, off_keys, off_argmax, off_tlse, off_jobs, off_chunks;
    RowScratchLayout rs;
    size_t total;
};
static VerifyWs verify_ws_layout(int64_t B, int64_t Lt, int nslices, int nchunks) {
    VerifyWs w;
    size_t o = 0;
    w.off_row_ticket = o; o += align_up((size_t)(B * Lt) * 4, 256);
    w.off_b_ticket = o;   o += align_up((size_t)B * 4, 256);
    w.off_res_ticket = o; o += align_up((size_t)B * 4, 256);
    w.off_b_status = o;   o += align_up((size_t)B * 4, 256);
    w.zero_bytes = o;
    w.off_partials = o;   o += align_up((size_t)(B * Lt) * nslices * sizeof(SlicePartial), 256);
    w.off_keys = o;       o += align_up((size_t)(B * Lt) * nslices * 8, 256);
    w.off_argmax = o;     o += align_up((size_t)(B * Lt) * 4, 256);
    w.off_tlse = o;       o += align_up((size_t)(B * Lt) * 8, 256);
    w.off_jobs = o;       o += align_up((size_t)B * sizeof(SampleJob), 256);
    w.off_chunks = o;     o += align_up((size_t)B * nchunks * 8, 256);
    w.rs = row_scratch_layout(o, B * Lt, nslices);
    w.total = w.rs.end;
    return w;
}

template <typename DT>
static int nchunks_of(int V) { return (V + 32 * Elem<DT>::N - 1) / (32 * Elem<DT>::N); }

template <typename DT>
static size_t verify_ws_bytes(int B, int Lt, int V) {
    const SlicePlan plan = plan_slices<DT>((long long)B * Lt, V, slice_target_ctas());
    return verify_ws_layout(B, Lt, plan.nslices, nchunks_of<DT>(V)).total;
}

template <typename DT>
static int32_t launch_verify(VerifyArgs &a, void *workspace, size_t workspace_bytes, cudaStream_t st,
                             int phases) {
    const long long nrows = (long long)a.B * a.Lt;
    const SlicePlan plan = plan_slices<DT>(nrows, a.V, slice_target_ctas());
    a.nslices = plan.nslices;
    a.slice_elems = plan.slice_elems;
    a.nchunks = nchunks_of<DT>(a.V);
    a.ntiles_row = (a.V + tile_elems<DT>() - 1) / tile_elems<DT>();
    const VerifyWs w = verify_ws_layout(a.B, a.Lt, a.nslices, a.nchunks);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(workspace);
    a.row_ticket = reinterpret_cast<unsigned *>(ws + w.off_row_ticket);
    a.b_ticket = reinterpret_cast<unsigned *>(ws + w.off_b_ticket);
    a.res_ticket = reinterpret_cast<unsigned *>(ws + w.off_res_ticket);
    a.b_status = reinterpret_cast<unsigned *>(ws + w.off_b_status);
    a.partials = reinterpret_cast<SlicePartial *>(ws + w.off_partials);
    a.keys = reinterpret_cast<unsigned long long *>(ws + w.off_keys);
    a.argmax = reinterpret_cast<int32_t *>(ws + w.off_argmax);
    a.tlse64 = reinterpret_cast<double *>(ws + w.off_tlse);
    a.jobs = reinterpret_cast<SampleJob *>(ws + w.off_jobs);
    a.rs.row_ticket = a.row_ticket;
    a.rs.cols = reinterpret_cast<uint2 *>(ws + w.rs.off_cols);
    a.rs.wpart = reinterpret_cast<WarpPartial *>(ws + w.rs.off_wpart);
    a.chunk_sums = reinterpret_cast<double *>(ws + w.off_chunks);
    // residual pass: about 4 CTAs per SM over all jobs, at least one chunk per warp
    int rsl = (device_sm_count() * 4 + a.B - 1) / a.B;
    const int max_rsl = (a.nchunks + kWarps - 1) / kWarps;
    if (rsl > max_rsl) rsl = max_rsl;
    if (rsl < 1) rsl = 1;
    a.chunks_per_slice = (a.nchunks + rsl - 1) / rsl;
    a.res_slices = (a.nchunks + a.chunks_per_slice - 1) / a.chunks_per_slice;

    const long long nblocks = nrows * a.nslices;
    if (nblocks > 0x7FFFFFFFLL) return DSP_ERR_UNSUPPORTED;
    if (phases & kVerifyStats) {
    // tickets and status words of the workspace start at zero
    PrepareArgs prep = PrepareArgs();
    prep.zero_a = reinterpret_cast<uint32_t *>(ws); prep.n_a = (long long)(w.zero_bytes / 4);
    DSP_CUDA_TRY(launch_prepare(prep, st));
    if (a.nslices <= kMaxSlices && nrows <= 0x7FFFFFFFLL && stream_layout_ok<DT>(a.target, a.V, a.tstride_b, a.tstride_l)) {
        static RingSmemDone smem_done;                       // one per element type
        DSP_CUDA_TRY(allow_ring_smem(target_scan_kernel<DT>, smem_done));
        a.nstages = ring_stages(nblocks);
        const ProfileEvents pe = g_profile[DSP_PROFILE_TARGET_SCAN];
        if (pe.start) DSP_CUDA_TRY(cudaEventRecord(pe.start, st));
        // the streaming kernel may start beside the preparation: it waits for it after its rows are streamed
        DSP_CUDA_TRY(launch_dependent(target_scan_kernel<DT>, (unsigned)nblocks, kThreads, (size_t)a.nstages * kTileBytes, st, a,
                                      !pe.start));
        if (pe.stop) DSP_CUDA_TRY(cudaEventRecord(pe.stop, st));
    } else {
        target_kernel<DT><<<(unsigned)nblocks, kThreads, 0, st>>>(a);
    }
    DSP_CUDA_TRY(cudaGetLastError());
    }
    if (phases & kVerifyDecide) {
        const bool early = true;
        if (a.all_greedy)
            DSP_CUDA_TRY(launch_dependent(accept_kernel<DT>, (unsigned)((a.B + kWarps - 1) / kWarps), kThreads, 0, st, a, early));
        else           // the acceptance scan runs inside the residual kernel
            DSP_CUDA_TRY(launch_dependent(residual_kernel<DT, true>, (unsigned)(a.B * a.res_slices), kThreads, 0, st, a, early));
    }
    return DSP_OK;
}

// ---- sharded target head: statistics from the slices' records, sampling from gathered rows ----

struct TargetMergeArgs {
    int G, B, Lt;
    const dsp_shard_sums *sums;        // [G,B,Lt]
    const unsigned long long *keys;    // [G,B,Lt] (one key per slice and row)
    const uint32_t *shard_status;      // [G,B]
    int32_t *argmax;                   // [B*Lt]
    double *tlse64;                    // [B*Lt]
    float *xt;                         // [B*Lt] target logit of the row's path token (NaN: none)
    int32_t *tgt_argmax;
    float *tgt_lse;
    unsigned *b_status;
};

// One warp per target row: argmax = the best of the slices' keys, log-sum-exp from the slices'
// sums against a common reference exponent, the path token's logit from the slice that holds it.
__global__ void __launch_bounds__(kThreads) target_merge_kernel(const TargetMergeArgs m) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long nrows = (long long)m.B * m.Lt;
    const long long row = (long long)blockIdx.x * kWarps + warp;
    if (row >= nrows) return;
    const int b = (int)(row / m.Lt);
    float cm = kRefFloor, xt = CUDART_NAN_F;
    unsigned long long best = 0ull;
    for (int g = lane; g < m.G; g += 32) {
        const dsp_shard_sums r = m.sums[g * nrows + row];
        if (r.S > 0.0 || !(r.S == r.S)) cm = fmaxf(cm, r.c);
        if (r.eos_logit == r.eos_logit) xt = r.eos_logit;
        const unsigned long long k = m.keys[g * nrows + row];
        best = k > best ? k : best;
    }
    cm = warp_max(cm);
    best = warp_max(best);
    double S = 0.0, T = 0.0;
    for (int g = lane; g < m.G; g += 32) {
        const dsp_shard_sums r = m.sums[g * nrows + row];
        if (r.S != 0.0) {
            const double d = (double)r.c - (double)cm;
            const double w = exp2(d);
            S += w * r.S;
            T += w * (r.T + r.S * d);
        }
    }
    S = warp_sum(S);
    T = warp_sum(T);
    const unsigned has = __ballot_sync(0xFFFFFFFFu, xt == xt);
    xt = has ? __shfl_sync(0xFFFFFFFFu, xt, __ffs(has) - 1) : CUDART_NAN_F;
    if (lane == 0) {
        double lse, mean_x;
        const bool ok = row_log_stats(cm, S, T, lse, mean_x) && best != 0ull;
        const int am = best ? key_id(best) : 0;
        m.argmax[row] = am;
        m.tlse64[row] = lse;
        m.xt[row] = xt;
        if (m.tgt_argmax) m.tgt_argmax[row] = am;
        if (m.tgt_lse) m.tgt_lse[row] = (float)lse;
        unsigned st = ok ? 0u : DSP_ROW_NONFINITE_INPUT;
        if (row == (long long)b * m.Lt)
            for (int g = 0; g < m.G; ++g) st |= m.shard_status[(long long)g * m.B + b];
        if (st) atomicOr(&m.b_status[b], st);
    }
}

struct SampleArgs {
    int B, L, Lt;
    const int32_t *job_trow, *job_drow;    // [B]
    const double *tgt_lse64, *draft_lse64; // [B*Lt], [B*L]
    const int32_t *tgt_argmax;             // [B*Lt]
    const float *u;                        // [B,L+1]
    SampleJob *jobs;                       // [B]
    double *tlse_g, *dlse_g;               // [B]
};
// Jobs over the gathered rows: row b of the gathered arrays is batch row b's row to sample from.
__global__ void sample_prepare_kernel(const SampleArgs s) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= s.B) return;
    SampleJob job;
    job.trow = -1; job.drow = -1; job.u = 0.f; job.fallback = -1;
    const int tr = s.job_trow[b], dr = s.job_drow[b];
    double tl = 0.0, dl = 0.0;
    if (tr >= 0) {
        job.trow = b;
        job.drow = dr >= 0 ? b : -1;
        job.u = s.u[(long long)b * (s.L + 1) + s.L];
        job.fallback = s.tgt_argmax[tr];
        tl = s.tgt_lse64[tr];
        if (dr >= 0) dl = s.draft_lse64[dr];
    }
    s.jobs[b] = job;
    s.tlse_g[b] = tl;
    s.dlse_g[b] = dl;
}

struct MergeWs {
    size_t off_b_status, zero_bytes, off_argmax, off_tlse, off_xt, off_jobs, total;
};
static MergeWs verify_merge_ws_layout(int64_t B, int64_t Lt) {
    MergeWs w;
    size_t o = 0;
    w.off_b_status = o; o += align_up((size_t)B * 4, 256);
    w.zero_bytes = o;
    w.off_argmax = o;   o += align_up((size_t)(B * Lt) * 4, 256);
    w.off_tlse = o;     o += align_up((size_t)(B * Lt) * 8, 256);
    w.off_xt = o;       o += align_up((size_t)(B * Lt) * 4, 256);
    w.off_jobs = o;     o += align_up((size_t)B * sizeof(SampleJob), 256);
    w.total = o;
    return w;
}

struct SampleWs {
    size_t off_res_ticket, zero_bytes, off_jobs, off_tlse, off_dlse, off_chunks, total;
};
static SampleWs sample_ws_layout(int64_t B, int nchunks) {
    SampleWs w;
    size_t o = 0;
    w.off_res_ticket = o; o += align_up((size_t)B * 4, 256);
    w.zero_bytes = o;
    w.off_jobs = o;       o += align_up((size_t)B * sizeof(SampleJob), 256);
    w.off_tlse = o;       o += align_up((size_t)B * 8, 256);
    w.off_dlse = o;       o += align_up((size_t)B * 8, 256);
    w.off_chunks = o;     o += align_up((size_t)B * nchunks * 8, 256);
    w.total = o;
    return w;
}

template <typename DT>
static int32_t launch_sample(VerifyArgs &a, SampleArgs &s, void *workspace, size_t workspace_bytes, cudaStream_t st) {
    a.nchunks = nchunks_of<DT>(a.V);
    const SampleWs w = sample_ws_layout(a.B, a.nchunks);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    char *ws = reinterpret_cast<char *>(workspace);
    a.res_ticket = reinterpret_cast<unsigned *>(ws + w.off_res_ticket);
    a.jobs = reinterpret_cast<SampleJob *>(ws + w.off_jobs);
    a.tlse64 = reinterpret_cast<double *>(ws + w.off_tlse);
    s.tlse_g = a.tlse64;
    s.dlse_g = reinterpret_cast<double *>(ws + w.off_dlse);
    a.draft_lse64 = s.dlse_g;
    s.jobs = a.jobs;
    a.chunk_sums = reinterpret_cast<double *>(ws + w.off_chunks);
    int rsl = (device_sm_count() * 4 + a.B - 1) / a.B;
    const int max_rsl = (a.nchunks + kWarps - 1) / kWarps;
    if (rsl > max_rsl) rsl = max_rsl;
    if (rsl < 1) rsl = 1;
    a.chunks_per_slice = (a.nchunks + rsl - 1) / rsl;
    a.res_slices = (a.nchunks + a.chunks_per_slice - 1) / a.chunks_per_slice;
    DSP_CUDA_TRY(cudaMemsetAsync(ws, 0, w.zero_bytes, st));
    sample_prepare_kernel<<<(unsigned)((a.B + 127) / 128), 128, 0, st>>>(s);
    DSP_CUDA_TRY(cudaGetLastError());
    residual_kernel<DT, false><<<(unsigned)(a.B * a.res_slices), kThreads, 0, st>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

}  // namespace dsp

using namespace dsp;

static int32_t check_verify_shape(int32_t B, int32_t L, int32_t Lt, int32_t V, int32_t dtype) {
    if (B < 0 || L < 1 || V < 1 || Lt < L || Lt > L + 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (L > DSP_MAX_L || V > (1 << 30)) return DSP_ERR_UNSUPPORTED;
    return DSP_OK;
}

extern "C" int32_t dsp_verify_workspace_bytes(int32_t B, int32_t L, int32_t Lt, int32_t V,
                                              int32_t dtype, size_t *bytes) {
    if (!bytes) return DSP_ERR_INVALID_ARG;
    const int32_t rc = check_verify_shape(B, L, Lt, V, dtype);
    if (rc != DSP_OK) return rc;
    const int Bq = B > 0 ? B : 1;
    *bytes = dtype == DSP_BF16 ? verify_ws_bytes<__nv_bfloat16>(Bq, Lt, V)
                               : verify_ws_bytes<float>(Bq, Lt, V);
    return DSP_OK;
}

int32_t dsp::verify_impl(const void *target_logits, int32_t dtype,
                         int32_t B, int32_t L, int32_t Lt, int32_t V,
                         int64_t tstride_b, int64_t tstride_l,
                         const void *draft_logits, int64_t dstride_b, int64_t dstride_l,
                         const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                         const float *cand_logit, const double *draft_lse64, int32_t KC,
                         int32_t all_greedy, const uint8_t *mode, const float *u, int32_t eos_id,
                         int32_t *accepted_len, int32_t *next_token, float *ratio,
                         int32_t *tgt_argmax, float *tgt_lse, uint32_t *row_status,
                         void *workspace, size_t workspace_bytes, cudaStream_t st, int phases) {
    const int32_t rc = check_verify_shape(B, L, Lt, V, dtype);
    if (rc != DSP_OK) return rc;
    if (B == 0) return DSP_OK;
    if (!target_logits || !path || !path_len || !accepted_len || !next_token || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (!all_greedy) {
        if (!draft_logits || !path_slot || !cand_logit || !draft_lse64 || !mode || !u)
            return DSP_ERR_INVALID_ARG;
        if (KC < 1 || KC > DSP_MAX_K + 1) return DSP_ERR_UNSUPPORTED;
        if (dstride_l < V || dstride_b < 0 || (B > 1 && dstride_b < (int64_t)(L - 1) * dstride_l + V))
            return DSP_ERR_INVALID_ARG;
    }
    if (tstride_l < V || tstride_b < 0 || (B > 1 && tstride_b < (int64_t)(Lt - 1) * tstride_l + V))
        return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(target_logits) & (es - 1)) != 0) return DSP_ERR_INVALID_ARG;
    if (draft_logits && (reinterpret_cast<uintptr_t>(draft_logits) & (es - 1)) != 0)
        return DSP_ERR_INVALID_ARG;

    VerifyArgs a;
    a.target = target_logits; a.draft = draft_logits;
    a.B = B; a.L = L; a.Lt = Lt; a.V = V;
    a.tstride_b = tstride_b; a.tstride_l = tstride_l;
    a.dstride_b = dstride_b; a.dstride_l = dstride_l;
    a.path = path; a.path_slot = path_slot; a.path_len = path_len;
    a.cand_logit = cand_logit; a.draft_lse64 = draft_lse64; a.KC = KC;
    a.all_greedy = all_greedy ? 1 : 0; a.mode = mode; a.u = u; a.eos_id = eos_id;
    a.accepted_len = accepted_len; a.next_token = next_token; a.ratio = ratio;
    a.tgt_argmax = tgt_argmax; a.tgt_lse = tgt_lse; a.row_status = row_status;
    a.xt_probe = nullptr; a.job_trow = nullptr; a.job_drow = nullptr;
    return dtype == DSP_BF16 ? launch_verify<__nv_bfloat16>(a, workspace, workspace_bytes, st, phases)
                             : launch_verify<float>(a, workspace, workspace_bytes, st, phases);
}

extern "C" int32_t dsp_verify(const void *target_logits, int32_t dtype,
                              int32_t B, int32_t L, int32_t Lt, int32_t V,
                              int64_t tstride_b, int64_t tstride_l,
                              const void *draft_logits, int64_t dstride_b, int64_t dstride_l,
                              const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                              const float *cand_logit, const double *draft_lse64, int32_t KC,
                              int32_t all_greedy, const uint8_t *mode, const float *u, int32_t eos_id,
                              int32_t *accepted_len, int32_t *next_token, float *ratio,
                              int32_t *tgt_argmax, float *tgt_lse, uint32_t *row_status,
                              void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    return verify_impl(target_logits, dtype, B, L, Lt, V, tstride_b, tstride_l, draft_logits, dstride_b,
                       dstride_l, path, path_slot, path_len, cand_logit, draft_lse64, KC, all_greedy, mode, u,
                       eos_id, accepted_len, next_token, ratio, tgt_argmax, tgt_lse, row_status, workspace,
                       workspace_bytes, reinterpret_cast<cudaStream_t>(stream), kVerifyStats | kVerifyDecide);
}

// ---- dsp_verify_merge / dsp_residual_sample: verification with a vocabulary-sharded target head ----

extern "C" int32_t dsp_verify_merge_workspace_bytes(int32_t B, int32_t Lt, size_t *bytes) {
    if (!bytes || B < 0 || Lt < 1) return DSP_ERR_INVALID_ARG;
    *bytes = verify_merge_ws_layout(B > 0 ? B : 1, Lt).total;
    return DSP_OK;
}

extern "C" int32_t dsp_verify_merge(int32_t G, const dsp_shard_sums *sums, const uint64_t *keys,
                                    const uint32_t *shard_status,
                                    int32_t B, int32_t L, int32_t Lt,
                                    const int32_t *path, const int32_t *path_slot, const int32_t *path_len,
                                    const float *cand_logit, const double *draft_lse64, int32_t KC,
                                    int32_t all_greedy, const uint8_t *mode, const float *u, int32_t eos_id,
                                    int32_t *accepted_len, int32_t *next_token, float *ratio,
                                    int32_t *tgt_argmax, float *tgt_lse, double *tgt_lse64,
                                    int32_t *job_trow, int32_t *job_drow, uint32_t *row_status,
                                    void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (G < 1 || B < 0 || L < 1 || Lt < L || Lt > L + 1) return DSP_ERR_INVALID_ARG;
    if (L > DSP_MAX_L || G > 1024) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!sums || !keys || !shard_status || !path || !path_len || !accepted_len || !next_token || !tgt_argmax ||
        !tgt_lse64 || !job_trow || !job_drow || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (!all_greedy) {
        if (!path_slot || !cand_logit || !draft_lse64 || !mode || !u) return DSP_ERR_INVALID_ARG;
        if (KC < 1 || KC > DSP_MAX_K + 1) return DSP_ERR_UNSUPPORTED;
    }
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const MergeWs w = verify_merge_ws_layout(B, Lt);
    if (workspace_bytes < w.total) return DSP_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    char *ws = reinterpret_cast<char *>(workspace);
    DSP_CUDA_TRY(cudaMemsetAsync(ws, 0, w.zero_bytes, st));
    TargetMergeArgs m;
    m.G = G; m.B = B; m.Lt = Lt;
    m.sums = sums;
    m.keys = reinterpret_cast<const unsigned long long *>(keys);
    m.shard_status = shard_status;
    m.argmax = reinterpret_cast<int32_t *>(ws + w.off_argmax);
    m.tlse64 = tgt_lse64;
    m.xt = reinterpret_cast<float *>(ws + w.off_xt);
    m.tgt_argmax = tgt_argmax;
    m.tgt_lse = tgt_lse;
    m.b_status = reinterpret_cast<unsigned *>(ws + w.off_b_status);
    const long long nrows = (long long)B * Lt;
    target_merge_kernel<<<(unsigned)((nrows + kWarps - 1) / kWarps), kThreads, 0, st>>>(m);
    DSP_CUDA_TRY(cudaGetLastError());
    VerifyArgs a = VerifyArgs();
    a.B = B; a.L = L; a.Lt = Lt; a.V = 1;
    a.path = path; a.path_slot = path_slot; a.path_len = path_len;
    a.cand_logit = cand_logit; a.draft_lse64 = draft_lse64; a.KC = KC;
    a.all_greedy = all_greedy ? 1 : 0; a.mode = mode; a.u = u; a.eos_id = eos_id;
    a.accepted_len = accepted_len; a.next_token = next_token; a.ratio = ratio;
    a.row_status = row_status;
    a.argmax = m.argmax; a.tlse64 = tgt_lse64; a.xt_probe = m.xt;
    a.b_status = m.b_status;
    a.jobs = reinterpret_cast<SampleJob *>(ws + w.off_jobs);
    a.job_trow = job_trow; a.job_drow = job_drow;
    accept_kernel<float><<<(unsigned)((B + kWarps - 1) / kWarps), kThreads, 0, st>>>(a);
    DSP_CUDA_TRY(cudaGetLastError());
    return DSP_OK;
}

extern "C" int32_t dsp_residual_sample_workspace_bytes(int32_t B, int32_t V, int32_t dtype, size_t *bytes) {
    if (!bytes || B < 0 || V < 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    const int Bq = B > 0 ? B : 1;
    *bytes = sample_ws_layout(Bq, dtype == DSP_BF16 ? nchunks_of<__nv_bfloat16>(V) : nchunks_of<float>(V)).total;
    return DSP_OK;
}

extern "C" int32_t dsp_residual_sample(const void *target_rows, const void *draft_rows, int32_t dtype,
                                       int32_t B, int32_t L, int32_t Lt, int32_t V,
                                       int64_t tstride, int64_t dstride,
                                       const int32_t *job_trow, const int32_t *job_drow,
                                       const double *tgt_lse64, const double *draft_lse64,
                                       const int32_t *tgt_argmax, const float *u,
                                       int32_t *next_token, uint32_t *row_status,
                                       void *workspace, size_t workspace_bytes, dsp_stream_t stream) {
    if (B < 0 || L < 1 || Lt < L || Lt > L + 1 || V < 1) return DSP_ERR_INVALID_ARG;
    if (dtype != DSP_F32 && dtype != DSP_BF16) return DSP_ERR_UNSUPPORTED;
    if (V > (1 << 30)) return DSP_ERR_UNSUPPORTED;
    if (B == 0) return DSP_OK;
    if (!target_rows || !draft_rows || !job_trow || !job_drow || !tgt_lse64 || !draft_lse64 || !tgt_argmax || !u ||
        !next_token || !row_status || !workspace)
        return DSP_ERR_INVALID_ARG;
    if (tstride < V || dstride < V) return DSP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0) return DSP_ERR_INVALID_ARG;
    const size_t es = dtype == DSP_BF16 ? 2 : 4;
    if (((reinterpret_cast<uintptr_t>(target_rows) | reinterpret_cast<uintptr_t>(draft_rows)) & (es - 1)) != 0)
        return DSP_ERR_INVALID_ARG;
    VerifyArgs a = VerifyArgs();
    a.target = target_rows; a.draft = draft_rows;
    a.B = B; a.L = 1; a.Lt = 1; a.V = V;               // the gathered arrays hold one row per batch row
    a.tstride_b = tstride; a.tstride_l = tstride;
    a.dstride_b = dstride; a.dstride_l = dstride;
    a.next_token = next_token; a.row_status = row_status;
    SampleArgs s;
    s.B = B; s.L = L; s.Lt = Lt;
    s.job_trow = job_trow; s.job_drow = job_drow;
    s.tgt_lse64 = tgt_lse64; s.draft_lse64 = draft_lse64;
    s.tgt_argmax = tgt_argmax; s.u = u;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    return dtype == DSP_BF16 ? launch_sample<__nv_bfloat16>(a, s, workspace, workspace_bytes, st)
                             : launch_sample<float>(a, s, workspace, workspace_bytes, st);
}
