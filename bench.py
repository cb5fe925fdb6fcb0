#!/usr/bin/env python
"""Benchmark of the draft-and-verify step (lattice build -> path search -> verify [-> ADL]).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic
logits.  The headline workload is configuration 4 (B=64, L=32, V=152064, bf16,
Eq. 7 pruning, mixed greedy/stochastic rows): 623 MB per logits tensor, far
larger than L2, so every step streams from HBM.  Smaller configurations rotate
over several input sets for the same reason.  Rank 0 prints ONE JSON line.

Batch rows are independent, so with N GPUs every rank runs the same per-GPU
workload on its own rows (weak scaling, no collective on the data path); the
time is the maximum over ranks and the value the steps all ranks completed per
second.

Beside the contract's keys the line carries: per-stage times and logits GB/s
(as fractions of the nominal 8 TB/s, of the measured copy bandwidth and of
``read_probe``, a read-only pass over the same logits timed in the same run),
the other four workloads, and ``parity``: the timed binary's outputs on a timed
input set compared with the oracle on sampled batch rows, near-ties counted.

--impl reference times the CPU oracle (plain C, as it stands) on a bounded
sample of the same workload on this machine's host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_02358_b200 import workloads as wl  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
HEADLINE = 4
# DRAM bytes (read + write) of one launch each of the two streaming kernels from an ncu capture of this
# workload (see profiles/); absent = not captured since the kernels last changed.
NCU_TRAFFIC_BYTES = {4: 640_400_000 + 626_800_000}


# The streaming kernels' own time is sampled inside the timed region on one step in this many
# (the events on both streams cost such a step 20 us or more), and on 32 steps right after it.
PROFILE_EVERY = 16


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, power = [], [], []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        seen = set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2])); power.append(float(c[3]))
            except ValueError:
                continue
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    seen.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm),
                       power_w_max=max(power))
        out["reasons"] = sorted(seen)
        return out


def params_of(w):
    return dict(K=w.K, W=w.W, tau=w.tau, lam=w.lam, eos_id=w.eos_id)


class GpuStep:
    """Pre-allocated outputs and workspaces for one workload; ``run(inp)`` enqueues one step."""

    def __init__(self, w, device):
        from paper_2510_02358_b200 import binding as dsp
        self.dsp, self.w, self.dev = dsp, w, device
        dt = dsp.DSP_BF16 if w.dtype == torch.bfloat16 else dsp.DSP_F32
        self.lat = dsp.lattice_outputs(w.B, w.L, w.K, w.eos_id, device)
        self.cps = dsp.cps_outputs(w.B, w.L, w.W, device, beams=True)
        self.ver = dsp.verify_outputs(w.B, w.L, w.Lt, device)
        self.ws_l = dsp.alloc_workspace(dsp.dsp_lattice_workspace_bytes(w.B, w.L, w.V, dt, w.K), device)
        self.ws_v = dsp.alloc_workspace(dsp.dsp_verify_workspace_bytes(w.B, w.L, w.Lt, w.V, dt), device)
        self.all_greedy = w.verify == "greedy"
        # two preparing kernels, the pass over the draft logits, the path search, the pass over the target
        # logits, accept (greedy) or residual with the acceptance scan inside (stochastic rows)
        self.kernels_per_step = 6

    def step(self, inp):
        """One step through the single-call entry point (what `value` and `e2e` time)."""
        dsp, w = self.dsp, self.w
        dsp.dsp_draft_verify_step(
            inp["draft"], inp["target"], inp["prev_token"], inp["table"], K_max=w.K, W=w.W, lam=w.lam,
            tau=w.tau, eos_id=w.eos_id, table_log2=inp["table_log2"], hash_seed=inp["hash_seed"],
            mode=None if self.all_greedy else inp["mode"], u=None if self.all_greedy else inp["u"],
            all_greedy=self.all_greedy, lat=self.lat, cps=self.cps, ver=self.ver,
            lattice_workspace=self.ws_l, verify_workspace=self.ws_v)

    def graph(self, inp):
        """The single-call step on ``inp`` recorded as a CUDA graph (same outputs and workspaces)."""
        dsp, w = self.dsp, self.w
        return dsp.dsp_step_graph_create(
            inp["draft"], inp["target"], inp["prev_token"], inp["table"], K_max=w.K, W=w.W, lam=w.lam,
            tau=w.tau, eos_id=w.eos_id, table_log2=inp["table_log2"], hash_seed=inp["hash_seed"],
            mode=None if self.all_greedy else inp["mode"], u=None if self.all_greedy else inp["u"],
            all_greedy=self.all_greedy, lat=self.lat, cps=self.cps, ver=self.ver,
            lattice_workspace=self.ws_l, verify_workspace=self.ws_v)

    def run(self, inp, ev=None):
        """The same step as three calls, with an event after each (the per-stage times)."""
        dsp, w = self.dsp, self.w
        if ev:
            ev[0].record()
        dsp.dsp_lattice_build(inp["draft"], w.K, w.tau, w.eos_id, out=self.lat, workspace=self.ws_l)
        if ev:
            ev[1].record()
        dsp.dsp_cps_search(self.lat, inp["prev_token"], inp["table"], W=w.W, lam=w.lam, eos_id=w.eos_id,
                           table_log2=inp["table_log2"], hash_seed=inp["hash_seed"], V=w.V,
                           out=self.cps, row_status=self.lat.row_status)
        if ev:
            ev[2].record()
        if self.all_greedy:
            dsp.dsp_verify(inp["target"], None, self.cps, None, eos_id=w.eos_id, all_greedy=True,
                           row_status=self.lat.row_status, out=self.ver, workspace=self.ws_v)
        else:
            dsp.dsp_verify(inp["target"], inp["draft"], self.cps, self.lat, mode=inp["mode"], u=inp["u"],
                           eos_id=w.eos_id, row_status=self.lat.row_status, out=self.ver,
                           workspace=self.ws_v)
        if ev:
            ev[3].record()


def reduce_max_ms(ms: float, dist, device) -> float:
    """Slowest rank's time (the job's time); identity on one rank."""
    if dist is None:
        return ms
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_steps_per_s(world: int, steps: int, ms: float) -> float:
    """Every rank completes ``steps`` steps on its own batch rows in ``ms`` (max over ranks)."""
    return world * steps / (ms * 1e-3)


def rank_seed_base(rank: int) -> int:
    """Each rank draws its own batch rows: disjoint seed ranges per rank."""
    return rank * 1000


def input_sets(w, device, seed_base=0):
    step_bytes = wl.step_logits_bytes(w)
    n = 1 if step_bytes > 4 * L2_BYTES else min(16, -(-4 * L2_BYTES // step_bytes))
    return [wl.make_inputs(w, step=seed_base + i, device=device) for i in range(n)]


def time_workload(w, device, steps, warmup, dist=None, stages=True, seed_base=0, one_set=False):
    """Device-timed throughput of one workload; returns a dict of measurements.  ``one_set``: the
    same input set every step (inputs smaller than L2 then stay in it)."""
    sets = input_sets(w, device, seed_base)
    if one_set:
        sets = sets[:1]
    st = GpuStep(w, device)
    dsp = st.dsp
    for i in range(warmup):
        st.step(sets[i % len(sets)])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    # the two streaming kernels' own time: on sampled timed steps each launch is bracketed by a pair of
    # events inside the library (on the stream the kernel is launched on, inside the timed region).
    # In the one-call step the two kernels run side by side, so what is reported is the window from
    # the start of the pass over the draft logits to the end of the later of the two passes.
    scan_evs = []

    def profiled_step(inp):
        evs4 = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        for e in evs4:
            e.record()                                   # torch creates an event at its first record
        dsp.dsp_profile_events(dsp.PROFILE_LATTICE_SCAN, evs4[0], evs4[1])
        dsp.dsp_profile_events(dsp.PROFILE_TARGET_SCAN, evs4[2], evs4[3])
        scan_evs.append(evs4)
        st.step(inp)
        dsp.dsp_profile_events(dsp.PROFILE_LATTICE_SCAN, None, None)
        dsp.dsp_profile_events(dsp.PROFILE_TARGET_SCAN, None, None)

    every = PROFILE_EVERY if steps >= 8 * PROFILE_EVERY else max(steps, 1)    # a short run: its first step only
    e0.record()
    for i in range(steps):
        if stages and i % every == 0:                    # one timed step in `every` carries the events
            profiled_step(sets[i % len(sets)])
        else:
            st.step(sets[i % len(sets)])
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    in_region = len(scan_evs)
    if stages:                                           # and a series right after the timed region, for the statistics
        for i in range(32):
            profiled_step(sets[i % len(sets)])
        torch.cuda.synchronize()
    out = dict(ms_total=ms, ms_per_step=ms / steps, sets=len(sets), kernels_per_step=st.kernels_per_step)
    if scan_evs:
        win = sorted(max(e[0].elapsed_time(e[1]), e[0].elapsed_time(e[3])) for e in scan_evs)
        out.update(ms_scan_window=sum(win) / len(win), ms_scan_window_min=win[0],
                   ms_scan_window_median=win[len(win) // 2], scan_samples=len(win), scan_samples_in_region=in_region,
                   ms_lattice_scan=sum(e[0].elapsed_time(e[1]) for e in scan_evs) / len(scan_evs),
                   ms_target_scan=sum(e[2].elapsed_time(e[3]) for e in scan_evs) / len(scan_evs))
    if stages:
        # per-stage times: the same step as three calls with an event after each (outside the timed region)
        n = min(steps, 200)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n)]
        for i in range(n):
            st.run(sets[i % len(sets)], evs[i])
        torch.cuda.synchronize()
        tl = [e[0].elapsed_time(e[1]) for e in evs]
        tc = [e[1].elapsed_time(e[2]) for e in evs]
        tv = [e[2].elapsed_time(e[3]) for e in evs]
        out.update(ms_lattice=sum(tl) / n, ms_cps=sum(tc) / n, ms_verify=sum(tv) / n,
                   ms_lattice_min=min(tl), ms_verify_min=min(tv))
    out["mean_accepted_len"] = st.ver.accepted_len.float().mean().item()
    out["mean_path_len"] = st.cps.path_len.float().mean().item()
    if stages:
        # the same step replayed from CUDA graphs (one per input set: a graph holds its addresses)
        # This is the timed region of the headline value: the same warm-up, exactly `steps` replays between
        # a barrier and a synchronise on both sides.
        graphs = [st.graph(inp) for inp in sets]
        for i in range(max(warmup, 3)):
            graphs[i % len(graphs)].launch()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for i in range(steps):
            graphs[i % len(graphs)].launch()
        g1.record()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        out["ms_graph_total"] = g0.elapsed_time(g1)
        out["ms_graph_step"] = out["ms_graph_total"] / steps
        for g in graphs:
            g.destroy()
    return out, st, sets


def time_proxies(w, st, sets, device, reps=50):
    """dsp_cps_search on the headline workload's lattice with each causal proxy (device time per call)."""
    dsp = st.dsp
    inp = sets[0]
    st.run(inp)
    KC = st.lat.cand_id.shape[2]
    g = torch.Generator(device=device).manual_seed(3)
    tensor = -6.0 * torch.rand((w.B, w.L, KC, KC), generator=g, device=device)
    prev2 = torch.stack([inp["prev_token"], inp["prev_token"]], dim=1).contiguous()
    ver = -4.0 * torch.rand((w.B, w.L, KC), generator=g, device=device)     # a verifier-side score per candidate slot
    cases = {"hashed_bigram": (0, inp["table"], inp["prev_token"], None), "tensor": (2, tensor, inp["prev_token"], None),
             "hashed_trigram": (3, inp["table"], prev2, None),
             "hashed_bigram_with_verifier_term": (0, inp["table"], inp["prev_token"], ver)}
    out = {}
    for name, (kind, table, prev, vs) in cases.items():
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for r in range(reps + 3):
            if r == 3:
                e0.record()
            dsp.dsp_cps_search_biased(st.lat, prev, table, W=w.W, lam=w.lam, ver_score=vs, mu=0.5, eos_id=w.eos_id,
                                      proxy_kind=kind, table_log2=inp["table_log2"], hash_seed=inp["hash_seed"], V=w.V,
                                      out=st.cps)
        e1.record()
        torch.cuda.synchronize()
        out[name] = e0.elapsed_time(e1) / reps
    return out


def time_sharded(w, device, G=4, reps=40):
    """One rank's share of the lattice of a drafter head sharded G ways over the vocabulary, on the
    headline workload's logits: dsp_lattice_shard on a V/G slice and dsp_lattice_merge of G records
    (the all-gather between them is not timed: one GPU here)."""
    from paper_2510_02358_b200 import binding as dsp
    x = input_sets(w, device, 9)[0]["draft"]
    Vs = w.V // G // 8 * 8
    dt = dsp.DSP_BF16 if w.dtype == torch.bfloat16 else dsp.DSP_F32
    ws = dsp.alloc_workspace(dsp.dsp_shard_workspace_bytes(w.B, w.L, Vs, dt, w.K), device)
    sl = x[:, :, :Vs]
    rec = dsp.dsp_lattice_shard(sl, 0, w.K, w.eos_id, workspace=ws)
    stack = lambda t: torch.stack([t] * G, dim=0).contiguous()
    sums, keys, status = stack(rec.sums), stack(rec.keys), stack(rec.status)
    out = dsp.lattice_outputs(w.B, w.L, w.K, w.eos_id, device)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    ts, tm = 0.0, 0.0
    for r in range(reps + 3):
        ev[0].record()
        dsp.dsp_lattice_shard(sl, 0, w.K, w.eos_id, out=rec, workspace=ws)
        ev[1].record()
        dsp.dsp_lattice_merge(sums, keys, status, w.V, w.K, w.tau, w.eos_id, out=out)
        ev[2].record()
        torch.cuda.synchronize()
        if r >= 3:
            ts += ev[0].elapsed_time(ev[1])
            tm += ev[1].elapsed_time(ev[2])
    nbytes = w.B * w.L * Vs * (2 if w.dtype == torch.bfloat16 else 4)
    return {"G": G, "slice_V": Vs, "shard_ms": ts / reps, "merge_ms": tm / reps,
            "slice_logits_gbs": nbytes / (ts / reps * 1e-3) / 1e9,
            "record_bytes_per_row_and_slice": 24 + 8 * w.K, "workload": "draft logits of %s" % w.name}


def vocab_slice(V: int, G: int, r: int):
    """Slice r of G of the vocabulary: [lo, hi), whole multiples of 8 tokens except the last slice."""
    per = -(-V // G) // 8 * 8 or 8
    lo = min(V, r * per)
    return lo, (V if r == G - 1 else min(V, lo + per))


def sharded_exchange_leg(shard, gather, merge, timer, reps, dist):
    """The vocabulary-sharded lattice as its three stages on every rank: shard() reduces the rank's
    slice to records, gather() brings every slice's records to every rank (the path's one exchange
    step), merge() finishes the rows.  ``timer()`` returns an object with record() / elapsed_ms(other)
    (CUDA events on a GPU).  Returns mean times per stage, the maximum over ranks."""
    tot = [0.0, 0.0, 0.0]
    for r in range(reps + 2):
        t = [timer() for _ in range(4)]
        t[0].record()
        rec = shard()
        t[1].record()
        allrec = gather(rec)
        t[2].record()
        merge(allrec)
        t[3].record()
        t[3].sync()
        if r >= 2:
            for k in range(3):
                tot[k] += t[k].elapsed_ms(t[k + 1])
    ms = [x / reps for x in tot]
    if dist is not None:
        tt = torch.tensor(ms, dtype=torch.float64, device=timer.device)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms = tt.tolist()
    return {"shard_ms": ms[0], "gather_ms": ms[1], "merge_ms": ms[2]}


class CudaTimer:
    device = None

    def __init__(self):
        self.e = torch.cuda.Event(enable_timing=True)

    def record(self):
        self.e.record()

    def sync(self):
        self.e.synchronize()

    def elapsed_ms(self, other):
        return self.e.elapsed_time(other.e)


def time_sharded_exchange(w, device, dist, rank, world, reps=20):
    """With several GPUs: every rank holds slice `rank` of the vocabulary of the SAME draft logits (a
    tensor-parallel drafter head), dsp_lattice_shard -> all-gather of the records into local memory
    (NCCL; no kernel reads a peer's memory) -> dsp_lattice_merge on every rank."""
    from paper_2510_02358_b200 import binding as dsp
    x = wl.make_inputs(w, step=77, device=device)["draft"]          # the same seed on every rank
    lo, hi = vocab_slice(w.V, world, rank)
    sl = x[:, :, lo:hi]
    dt = dsp.DSP_BF16 if w.dtype == torch.bfloat16 else dsp.DSP_F32
    ws = dsp.alloc_workspace(dsp.dsp_shard_workspace_bytes(w.B, w.L, hi - lo, dt, w.K), device)
    out = dsp.lattice_outputs(w.B, w.L, w.K, w.eos_id, device)
    CudaTimer.device = device
    res = sharded_exchange_leg(
        lambda: dsp.dsp_lattice_shard(sl, lo, w.K, w.eos_id, workspace=ws),
        lambda rec: dsp.gather_shard_records(rec),
        lambda a: dsp.dsp_lattice_merge(a.sums, a.keys, a.status, w.V, w.K, w.tau, w.eos_id, out=out),
        CudaTimer, reps, dist)
    res.update(G=world, record_bytes_per_row_and_slice=24 + 8 * w.K,
               gathered_bytes_per_rank=world * w.B * w.L * (24 + 8 * w.K),
               workload="draft logits of %s, vocabulary slice per rank" % w.name)
    return res


def time_unmask(w, device, reps=40):
    """The drafter's refinement step (dsp_unmask_step) on logits of the headline workload's shape:
    S = 1 (every position masked, one call) and S = 4 (four calls, a quarter of the block each;
    rows revealed earlier are not read)."""
    from paper_2510_02358_b200 import binding as dsp
    sets = input_sets(w, device, 7)
    dt = dsp.DSP_BF16 if w.dtype == torch.bfloat16 else dsp.DSP_F32
    ws = dsp.alloc_workspace(dsp.dsp_unmask_workspace_bytes(w.B, w.L, w.V, dt), device)
    out = None
    res = {}
    row_bytes = w.V * (2 if w.dtype == torch.bfloat16 else 4)
    for S in (1, 4):
        n = -(-w.L // S)
        tokens = torch.zeros((w.B, w.L), dtype=torch.int32, device=device)
        masked = torch.empty((w.B, w.L), dtype=torch.uint8, device=device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        total, rows_read = 0.0, 0
        for r in range(reps + 3):
            x = sets[r % len(sets)]["draft"]
            masked.fill_(1)
            e0.record()
            for s in range(S):
                out = dsp.dsp_unmask_step(x, tokens, masked, n, out=out, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            if r >= 3:
                total += e0.elapsed_time(e1)
        rows_read = sum(max(w.L - s * n, 0) for s in range(S)) * w.B
        ms = total / reps
        res["S%d" % S] = {"ms": ms, "calls": S, "rows_read": rows_read,
                          "logits_gbs": rows_read * row_bytes / (ms * 1e-3) / 1e9}
        assert int(masked.sum().item()) == 0
    res["workload"] = "logits of %s" % w.name
    return res


def time_tree(w, device, reps=30):
    """The beams of the path search verified as one token tree in a single target pass (dsp_beam_tree,
    then dsp_verify_tree for the greedy rule or dsp_verify_tree_stochastic for the sampling rule) on a
    batch of 8 rows of the headline workload's vocabulary: draft length 16, 8 candidates, 4 beams,
    64 node slots per batch row.  The target rows are synthetic: the draft row of the node's depth plus noise."""
    from paper_2510_02358_b200 import binding as dsp
    tw = w.scaled(B=8, L=16, K=8, W=4, tau=0.0, name="tree_B8_L16_W4")
    inp = wl.make_inputs(tw, step=11, device=device)
    lat = dsp.dsp_lattice_build(inp["draft"], tw.K)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=tw.W, lam=tw.lam, table_log2=inp["table_log2"],
                             hash_seed=inp["hash_seed"], V=tw.V)
    tree = dsp.dsp_beam_tree(cps)
    N = tw.W * tw.L
    g = torch.Generator(device=device).manual_seed(5)
    depth = torch.cat([torch.zeros((tw.B, 1), dtype=torch.long, device=device),
                       (tree.node_depth.long() + 1).clamp_(0, tw.L - 1)], dim=1)          # row 0: after the prefix
    target = torch.empty((tw.B, 1 + N, tw.V), dtype=tw.dtype, device=device)
    for b in range(tw.B):
        target[b] = (inp["draft"][b, depth[b]].float() +
                     0.5 * torch.randn((1 + N, tw.V), generator=g, device=device)).to(tw.dtype)
    u = torch.rand((tw.B, N + 1), generator=g, device=device)
    res = {"workload": tw.name, "node_slots": N, "nodes_mean": float(tree.n_nodes.float().mean().item()),
           "target_bytes": target.numel() * target.element_size()}
    calls = {"beam_tree": lambda: dsp.dsp_beam_tree(cps),
             "verify_tree_greedy": lambda: dsp.dsp_verify_tree(target, tree, tw.L),
             "verify_tree_stochastic": lambda: dsp.dsp_verify_tree_stochastic(target, inp["draft"], tree, u)}
    for name, call in calls.items():
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        out = None
        for r in range(reps + 3):
            if r == 3:
                e0.record()
            out = call()
        e1.record()
        torch.cuda.synchronize()
        res[name + "_ms"] = e0.elapsed_time(e1) / reps
        if name != "beam_tree":
            res[name + "_mean_accepted_len"] = float(out.accepted_len.float().mean().item())
    return res


def time_e2e(w, st, sets, device, steps):
    """Same step through the public calls with HOST buffers: pinned logits are copied to the
    device inside the timed region and the step's results are read back every step."""
    inp = sets[0]
    host = {k: inp[k].cpu().pin_memory() for k in ("draft", "target", "prev_token", "mode", "u")}
    dev = {k: torch.empty_like(inp[k]) for k in host}
    res_host = torch.empty((3, w.B), dtype=torch.int32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = res_host.numel() * 4
    staged = dict(inp)

    def one():
        for k in host:
            dev[k].copy_(host[k], non_blocking=True)
        staged.update(dev)
        st.step(staged)
        res_host[0].copy_(st.ver.accepted_len, non_blocking=True)
        res_host[1].copy_(st.ver.next_token, non_blocking=True)
        res_host[2].copy_(st.lat.gen_len, non_blocking=True)
        torch.cuda.current_stream().synchronize()          # the caller needs the result to go on

    one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    wall = (time.perf_counter() - t0) * 1e3
    ms = max(e0.elapsed_time(e1), wall)
    return dict(value=steps / (ms / 1e3), unit="steps/s", h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                steps=steps, ms_per_step=ms / steps)


def oracle_step(w, inp_cpu, rows):
    """The oracle's whole step on the first ``rows`` batch rows; returns seconds."""
    import oracle
    sl = slice(0, rows)
    d, t = inp_cpu["draft"][sl].contiguous(), inp_cpu["target"][sl].contiguous()
    t0 = time.perf_counter()
    lat = oracle.lattice_build(d, w.K, tau=w.tau, eos_id=w.eos_id)
    cps = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count,
                            inp_cpu["prev_token"][sl], inp_cpu["table"], W=w.W, lam=w.lam, eos_id=w.eos_id,
                            table_log2=inp_cpu["table_log2"], hash_seed=inp_cpu["hash_seed"], V=w.V)
    if w.verify == "greedy":
        oracle.verify(t, None, cps.path, cps.path_len, None, None, eos_id=w.eos_id)
    else:
        oracle.verify(t, d, cps.path, cps.path_len, inp_cpu["mode"][sl], inp_cpu["u"][sl], eos_id=w.eos_id)
    return time.perf_counter() - t0


def cpu_inputs(inp, rows):
    """CPU copies of the first ``rows`` batch rows of one input set."""
    out = {}
    for k, v in inp.items():
        if isinstance(v, torch.Tensor):
            out[k] = v.cpu() if k == "table" else v[:rows].cpu().contiguous()
        else:
            out[k] = v
    return out


def cpu_baseline(w, inp, budget_s=12.0):
    """Oracle (kind=oracle) timed on a bounded sample of the workload: whole steps on the first
    ``rows`` batch rows, repeated until about ``budget_s`` seconds of CPU wall-clock are spent."""
    import oracle
    oracle.build()
    cores = oracle.threads()
    rows = w.B
    cpu = cpu_inputs(inp, rows)
    t = oracle_step(w, cpu, rows)
    if t > budget_s and rows > cores:                 # one step is already too long: fewer rows
        rows = max(cores, int(rows * budget_s / t) // cores * cores)
        cpu = cpu_inputs(inp, rows)
        t = oracle_step(w, cpu, rows)
    n, total = 1, t
    while total < budget_s and n < 1000:
        total += oracle_step(w, cpu, rows)
        n += 1
    step_s = total / n * w.B / rows
    return dict(value=1.0 / step_s, unit="steps/s", cores=cores, kind="oracle",
                sample="first %d of %d batch rows, %d steps, %.1f s of CPU wall-clock; scaled by B/rows"
                       % (rows, w.B, n, total))


def parity_recheck(w, st, inp, max_rows):
    """The timed binary against the oracle inside the benchmark run: one more step on a timed
    input set, then up to ``max_rows`` evenly spaced batch rows compared field by field by the
    same comparison the tests use (integers exact, log-probabilities within 1e-3, near-ties of
    the floating-point decisions counted).  Part of the CPU-baseline leg: it runs the oracle."""
    from types import SimpleNamespace
    tdir = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tests")
    if tdir not in sys.path:
        sys.path.insert(0, tdir)
    from parity import check_step
    st.step(inp)
    torch.cuda.synchronize()
    n = min(w.B, max_rows)
    rows = sorted({round(i * (w.B - 1) / max(1, n - 1)) for i in range(n)})
    idx = torch.as_tensor(rows, dtype=torch.long, device=inp["draft"].device)
    take = lambda v: v[idx].cpu() if isinstance(v, torch.Tensor) and v.dim() >= 1 and v.shape[0] == w.B else v
    small = {k: (v if k == "table" else take(v)) for k, v in inp.items()}
    g = SimpleNamespace(**{name: SimpleNamespace(**{k: take(v) for k, v in vars(getattr(st, name)).items()})
                           for name in ("lat", "cps", "ver")})
    out = {"rows_checked": len(rows), "of_rows": w.B}
    try:
        rep = check_step(g, small, K=w.K, W=w.W, tau=w.tau, lam=w.lam, eos_id=w.eos_id,
                         all_greedy=w.verify == "greedy")
        out.update(status="ok", near_tau=rep["near_tau"], near_accept=rep["near_accept"],
                   near_token=rep["near_token"], max_abs_err=rep["max_err"])
    except AssertionError as e:
        out.update(status="FAILED", detail=str(e)[:300])
    return out


def time_read_probe(sets, device, reps=40):
    """Read bandwidth of this GPU on the timed logits themselves: dsp_read_probe (a kernel that only
    reads, coalesced 128-bit loads) over the draft tensors of the input sets in turn."""
    from paper_2510_02358_b200 import binding as dsp
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    bufs = [s["draft"] for s in sets] + ([s["target"] for s in sets] if len(sets) == 1 else [])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for r in range(reps + 3):
        if r == 3:
            e0.record()
        dsp.dsp_read_probe(bufs[r % len(bufs)], sink)
    e1.record()
    torch.cuda.synchronize()
    nbytes = bufs[0].numel() * bufs[0].element_size()
    us = e0.elapsed_time(e1) / reps * 1e3
    return {"gbs": nbytes / us / 1e3, "us_per_launch": us, "bytes_per_launch": nbytes,
            "note": "dsp_read_probe over the draft logits of the timed input sets, back to back launches"}


def time_adl_loop(device, n_steps=256):
    """Workload 2 as the closed loop the controller runs in (Sec. 3.3): every step's draft length
    is the one dsp_adl_update asked for after the step before, from that step's accepted and
    generated lengths copied to the host (the step's one device-to-host crossing, with a stream
    synchronisation).  Fresh logits every step (seed = step), drawn beforehand at the longest
    length with EOS as the drafter's top-1 from a seeded random-walk position on; a step of length
    L reads their first L rows.  Wall-clock over the loop, the synchronisations included."""
    from paper_2510_02358_b200 import binding as dsp
    base = wl.CONFIGS[2]
    walk = wl.eos_walk(n_steps)
    lengths = (8, 16, 24, 32)
    sets = [wl.make_inputs(base.scaled(L=32, eos_from=c if c < 32 else -1), step=t, device=device)
            for t, c in enumerate(walk)]
    steps = {L: GpuStep(base.scaled(L=L), device) for L in lengths}
    host = torch.empty((2,), dtype=torch.int32).pin_memory()
    view = lambda inp, L: dict(inp, draft=inp["draft"][:, :L], target=inp["target"][:, :L], u=inp["u"])

    def loop(n):
        st, prm = dsp.dsp_adl_init(**wl.ADL_C2)
        hist, acc, gen = {L: 0 for L in lengths}, 0, 0
        for t in range(n):
            L = st.k
            g = steps[L]
            g.step(view(sets[t], L))
            host[0:1].copy_(g.ver.accepted_len, non_blocking=True)
            host[1:2].copy_(g.lat.gen_len, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            dsp.dsp_adl_update(st, prm, host[0:1], host[1:2])
            hist[L] += 1
            acc += int(host[0])
            gen += int(host[1])
        return hist, acc, gen

    loop(16)                                          # warm-up
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    hist, acc, gen = loop(n_steps)
    dt = time.perf_counter() - t0
    return {"steps": n_steps, "steps_per_s": n_steps / dt, "us_per_step": dt / n_steps * 1e6,
            "draft_length_histogram": hist, "mean_draft_length": sum(L * c for L, c in hist.items()) / n_steps,
            "mean_accepted_len": acc / n_steps, "mean_gen_len": gen / n_steps,
            "controller": wl.ADL_C2,
            "note": "dsp_draft_verify_step + copy of 2 int32 to the host + synchronise + dsp_adl_update per step"}


def config_of(w, world, sets=None):
    """The `config` object of the JSON line: the same for the timed arm and the reference arm."""
    step_bytes = wl.step_logits_bytes(w)
    nsets = sets if sets is not None else (1 if step_bytes > 4 * L2_BYTES else min(16, -(-4 * L2_BYTES // step_bytes)))
    return {"workload": w.name, "B": w.B * world, "B_per_gpu": w.B, "L": w.L, "V": w.V,
            "logits_dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "K": w.K, "W": w.W,
            "tau": w.tau, "verify": w.verify, "parallelism": "batch rows sharded, no collective",
            "l2": "inputs larger than L2" if nsets == 1 else "rotating %d input sets" % nsets}


def run_reference(args, rank, world):
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = wl.CONFIGS[args.config]
    cores = oracle.threads()
    rows = min(w.B, max(1, cores))
    inp = wl.make_inputs(w.scaled(B=rows), step=0, device="cpu")
    for _ in range(args.warmup):
        oracle_step(w, inp, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(w, inp, rows)
    t = (time.perf_counter() - t0) / args.steps
    step_s = t * w.B / rows
    val = 1.0 / step_s
    sample = "each step = first %d of %d batch rows (same recipe and seed), scaled by B/rows" % (rows, w.B)
    print(json.dumps({
        "impl": "reference", "metric": "draft-verify steps/s", "value": val, "unit": "steps/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": config_of(w, max(1, args.gpus)),
        "cpu_baseline": {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=HEADLINE, choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="dsp", choices=["dsp", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the other four workloads and the CPU baseline")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "dsp" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    from paper_2510_02358_b200 import build
    build.build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    w = wl.CONFIGS[args.config]
    sampler = ClockSampler(local) if rank == 0 else None
    m, st, sets = time_workload(w, device, args.steps, args.warmup, dist, seed_base=rank_seed_base(rank))
    clocks = sampler.stop() if sampler else None
    # The headline times the step the way a decoding loop runs it: recorded once per input set
    # (dsp_step_graph_create) and replayed (dsp_step_graph_launch).  The same step enqueued call by
    # call (dsp_draft_verify_step) is timed beside it; its region carries the sampled events of `roofline`.
    ms = reduce_max_ms(m["ms_graph_total"], dist, device)
    ms_direct = reduce_max_ms(m["ms_total"], dist, device)
    e2e = time_e2e(w, st, sets, device, min(args.steps, 10))
    if dist is not None:
        e2e["ms_per_step"] = reduce_max_ms(e2e["ms_per_step"], dist, device)
        e2e["value"] = whole_job_steps_per_s(world, 1, e2e["ms_per_step"])
        e2e["h2d_bytes_per_step"] *= world
        e2e["d2h_bytes_per_step"] *= world
    sharded = time_sharded_exchange(w, device, dist, rank, world) if dist is not None else None
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    probe = time_read_probe(sets, device)
    tensor_bytes = w.logits_bytes
    gbs_lat = tensor_bytes / (m["ms_lattice"] * 1e-3) / 1e9
    gbs_ver = tensor_bytes / (m["ms_verify"] * 1e-3) / 1e9
    gbs_both = 2 * tensor_bytes / ((m["ms_lattice"] + m["ms_verify"]) * 1e-3) / 1e9
    # the two streaming kernels of the step run side by side: both tensors over the window they span
    gbs_scan = 2 * tensor_bytes / (m["ms_scan_window"] * 1e-3) / 1e9
    gbs_step = 2 * tensor_bytes / (ms / args.steps * 1e-3) / 1e9
    line = {
        "metric": "draft-verify steps/s", "value": whole_job_steps_per_s(world, args.steps, ms), "unit": "steps/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": config_of(w, world, m["sets"]),
        "timed_call": "dsp_step_graph_launch (one graph per input set, recorded by dsp_step_graph_create)",
        "logits_gbs": {"lattice_build": gbs_lat, "verify": gbs_ver, "lattice_plus_verify": gbs_both,
                       "frac_of_8000": gbs_both / 8000.0, "frac_of_%s_copy_peak" % peak_kind: gbs_both / peak,
                       "frac_of_read_probe": gbs_both / probe["gbs"]},
        "stage_ms": {"lattice_build": m["ms_lattice"], "cps_search": m["ms_cps"], "verify": m["ms_verify"],
                     "note": "the three calls one after the other; `value` times the single-call step, "
                             "which overlaps the target statistics with the path search"},
        "direct_call": {"ms_per_step": ms_direct / args.steps,
                        "steps_per_s": whole_job_steps_per_s(world, args.steps, ms_direct),
                        "note": "the same step enqueued call by call through dsp_draft_verify_step, the same number of "
                                "steps between the same barriers; some of them carry the events of `roofline`"},
        "mean_accepted_len": m["mean_accepted_len"], "mean_path_len": m["mean_path_len"],
        "roofline": {"bound": "hbm", "kernel": "lattice_scan_kernel + target_scan_kernel (side by side in the step)",
                     "achieved": gbs_scan, "peak": peak,
                     "peak_kind": "%s copy bandwidth" % peak_kind, "unit": "GB/s", "frac": gbs_scan / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.cid),
                     "algorithmic_bytes_per_launch": 2 * tensor_bytes,
                     "launch_us": m["ms_scan_window"] * 1e3, "launch_us_median": m["ms_scan_window_median"] * 1e3,
                     "launch_us_min": m["ms_scan_window_min"] * 1e3, "launches_timed": m["scan_samples"],
                     "launches_timed_in_region": m["scan_samples_in_region"],
                     "sampled_in": "the direct_call region (a recorded graph takes no caller events) and 32 steps after it",
                     "frac_of_read_probe": gbs_scan / probe["gbs"],
                     "frac_of_8000": gbs_scan / 8000.0,
                     "call_level": {"gbs": gbs_both, "frac_of_8000": gbs_both / 8000.0,
                                    "note": "(draft + target bytes) / (dsp_lattice_build + dsp_verify), the three calls"},
                     "step_level": {"gbs": gbs_step, "frac_of_8000": gbs_step / 8000.0,
                                    "note": "(draft + target bytes) / ms_per_step of the one-call step, path search and "
                                            "residual draw included"}},
        "read_probe": probe,
        "row_steps_per_s": whole_job_steps_per_s(world, args.steps, ms) * w.B,
        "e2e": e2e,
        "gpu_launches": m["kernels_per_step"] * args.steps,
        "clocks": clocks,
    }
    if sharded is not None:
        line["vocab_sharded_exchange"] = sharded
    if not args.no_extras and world == 1:
        line["cpu_baseline"] = cpu_baseline(w, sets[0])
        line["parity"] = parity_recheck(w, st, sets[0], 16)
        line["cps_proxies_ms"] = time_proxies(w, st, sets, device)
        extras = {}
        del st, sets
        torch.cuda.empty_cache()
        for cid in sorted(wl.CONFIGS):
            if cid == args.config:
                continue
            variants = [wl.CONFIGS[cid]] if cid != 2 else [wl.CONFIGS[2].scaled(L=L, name="c2_L%d" % L)
                                                             for L in (8, 16, 24, 32)]
            for wv in variants:
                n = 20 if cid == 5 else 200
                mm, s2, i2 = time_workload(wv, device, n, 5)
                tb = wv.logits_bytes
                extras[wv.name] = {
                    "steps_per_s": 1e3 / mm["ms_per_step"], "ms_per_step": mm["ms_per_step"],
                    "graph_ms_per_step": mm.get("ms_graph_step"),
                    "stage_ms": {"lattice_build": mm["ms_lattice"], "cps_search": mm["ms_cps"],
                                 "verify": mm["ms_verify"]},
                    "logits_gbs": 2 * tb / ((mm["ms_lattice"] + mm["ms_verify"]) * 1e-3) / 1e9,
                    "frac_of_8000": 2 * tb / ((mm["ms_lattice"] + mm["ms_verify"]) * 1e-3) / 1e9 / 8000.0,
                    "input_sets": mm["sets"], "mean_accepted_len": mm["mean_accepted_len"],
                    "parity": parity_recheck(wv, s2, i2[0], 4 if cid == 5 else 16)}
                if 2 * tb < L2_BYTES:                   # also with the one input set left in L2
                    mw, s3, i3 = time_workload(wv, device, n, 5, stages=False, one_set=True)
                    extras[wv.name]["ms_per_step_inputs_in_l2"] = mw["ms_per_step"]
                    del s3, i3
                del s2, i2
                torch.cuda.empty_cache()
        line["workloads"] = extras
        line["adl_closed_loop_c2"] = time_adl_loop(device)
        line["unmask_step"] = time_unmask(w, device)
        line["tree_verification"] = time_tree(w, device)
        line["vocab_sharded_lattice"] = time_sharded(w, device)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
