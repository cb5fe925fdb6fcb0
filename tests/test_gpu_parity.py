"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same bytes."""
import math
from types import SimpleNamespace

import pytest
import numpy as np
import torch

import oracle
from paper_2510_02358_b200 import binding as dsp
from paper_2510_02358_b200 import workloads as wl
from parity import check_step, gpu_step

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _to(inp, dev=DEV):
    return {k: (v.to(dev) if isinstance(v, torch.Tensor) else v) for k, v in inp.items()}


def _params(w):
    return dict(K=w.K, W=w.W, tau=w.tau, lam=w.lam, eos_id=w.eos_id, all_greedy=(w.verify == "greedy"))


# ---- the five workloads at sizes the oracle finishes in seconds (several tiles + ragged tail) ----
SMALL = {
    1: dict(B=2, L=8, V=32000),
    2: dict(B=1, L=16, V=152064, eos_from=9),
    3: dict(B=4, L=6, V=152064),
    4: dict(B=6, L=8, V=50021),         # odd V: rows are not 16-byte aligned -> element-wise path
    5: dict(B=3, L=5, V=256000),
}


@pytest.mark.parametrize("cid", [1, 2, 3, 4, 5])
def test_workloads_small(cid):
    w = wl.CONFIGS[cid].scaled(**SMALL[cid])
    inp = wl.make_inputs(w, step=1, device=DEV)
    g = gpu_step(inp, **_params(w))
    rep = check_step(g, inp, **_params(w))
    print(cid, rep)
    assert rep["near_accept"] + rep["near_token"] + rep["near_tau"] <= 2


# ---- the benchmark's own launch configuration at full size, oracle on sampled batch rows ----
@pytest.mark.parametrize("cid,rows", [(1, None), (2, None), (3, [0, 7, 15]), (4, [0, 1, 33, 62, 63]),
                                      (5, [0, 101, 255])])
def test_workloads_full_size_sampled_rows(cid, rows):
    w = wl.CONFIGS[cid]
    if cid == 2:
        w = w.scaled(eos_from=21)
    inp = wl.make_inputs(w, step=0, device=DEV)
    g = gpu_step(inp, **_params(w))
    rep = check_step(g, inp, rows=rows, **_params(w))
    print(cid, rep)
    # properties that hold for every row at any size
    m = g.cps.path_len
    assert ((g.ver.accepted_len >= 0) & (g.ver.accepted_len <= m) & (m <= w.L)).all()
    bc = g.cps.beam_cum
    assert (bc[:, :-1] >= bc[:, 1:]).all()
    assert (g.lat.cand_count >= 1).all() and (g.lat.cand_count <= w.K + (w.eos_id >= 0)).all()
    assert torch.isfinite(g.lat.lse).all() and (g.lat.entropy > 0).all()
    assert (g.lat.entropy <= math.log(w.V) + 1e-3).all()
    if w.verify == "greedy":
        am = g.ver.tgt_argmax
        for b in range(w.B):
            mm = int(m[b])
            match = (g.cps.path[b, :mm] == am[b, :mm]).tolist()
            assert int(g.ver.accepted_len[b]) == (match.index(False) if False in match else mm)
    del inp
    torch.cuda.empty_cache()


# ---- edge shapes ----
@pytest.mark.parametrize("B,L,V,K,W,dtype", [
    (2, 3, 5, 8, 4, torch.float32),          # V < K
    (1, 1, 1, 1, 1, torch.float32),          # one token
    (3, 2, 37, 4, 3, torch.bfloat16),        # V not a multiple of 8
    (2, 100, 300, 3, 2, torch.float32),      # long draft
    (2, 4, 8200, 1, 1, torch.bfloat16),      # K = 1, W = 1, just over one tile
    (2, 3, 4099, 32, 32, torch.float32),     # largest K and W
    (5, 7, 1000, 15, 3, torch.bfloat16),     # the paper's defaults M_max = 15, beam 3
    (2, 3, 8192, 32, 32, torch.bfloat16),    # largest K and W on a 16-byte aligned layout (streaming kernels)
    (1, 2, 1048576, 16, 8, torch.bfloat16),  # a million-token vocabulary: rows cut into long slices
    (3, 2, 12288, 8, 4, torch.float32),      # fp32 rows of exactly three tiles
])
def test_edge_shapes(B, L, V, K, W, dtype):
    inp = _to(wl.tiny_random(B, L, V, dtype=dtype, seed=B * 100 + L))
    for tau, eos in ((0.0, -1), (0.8, V - 1)):
        p = dict(K=K, W=W, tau=tau, lam=0.5, eos_id=eos)
        rep = check_step(gpu_step(inp, **p), inp, **p)
        assert rep["near_accept"] + rep["near_token"] + rep["near_tau"] <= 1


@pytest.mark.parametrize("seed", range(6))
def test_whole_step_on_random_shapes(seed):
    """Seeded random shapes through the three calls and through the single call: both dtypes, aligned and
    unaligned vocabularies, one to several tiles, pruning on and off, EOS, greedy / mixed batches."""
    rng = np.random.default_rng(500 + seed)
    near = 0
    for case in range(4):
        B = int(rng.integers(1, 6))
        L = int(rng.integers(1, 20))
        V = int(rng.choice([7, 100, 1000, 4096, 6151, 12288, 20000, 33000]))
        K = int(rng.choice([1, 3, 8, 16, 32]))
        W = int(rng.choice([1, 2, 4, 8, 16]))
        dtype = torch.bfloat16 if rng.integers(0, 2) else torch.float32
        tau = float(rng.choice([0.0, 0.5, 0.8, 0.95]))
        eos = int(V - 1) if rng.integers(0, 2) else -1
        greedy = bool(rng.integers(0, 3) == 0)
        inp = _to(wl.tiny_random(B, L, V, dtype=dtype, seed=seed * 10 + case, sigma_t=float(rng.choice([0.2, 0.7, 1.5]))))
        p = dict(K=K, W=W, tau=tau, lam=float(rng.choice([0.25, 0.5, 0.75])), eos_id=eos, all_greedy=greedy)
        for fused in (False, True):
            rep = check_step(gpu_step(inp, fused=fused, **p), inp, **p)
            near += rep["near_accept"] + rep["near_token"] + rep["near_tau"]
    assert near <= 4


@pytest.mark.parametrize("V,dtype", [(12288 + 64, torch.bfloat16), (6144 + 32, torch.float32),
                                     (3 * 12288 + 8, torch.bfloat16)])
def test_short_ragged_tail_in_a_slice_of_its_own(V, dtype):
    """Few rows, so every tile is a slice of its own, and the last tile holds only a few vectors: most
    threads of its CTA see nothing at all, which must neither count in the sums nor disturb them."""
    inp = _to(wl.tiny_random(1, 4, V, dtype=dtype, seed=V % 97))
    for tau, eos in ((0.0, -1), (0.8, 5)):
        p = dict(K=8, W=4, tau=tau, lam=0.5, eos_id=eos)
        for fused in (False, True):
            rep = check_step(gpu_step(inp, fused=fused, **p), inp, **p)
            assert rep["max_err"]["lse64"] < 5e-6 and rep["max_err"]["entropy"] < 5e-5


def test_dense_proxy_ids_out_of_range_are_clamped():
    B, L, K, V = 2, 5, 4, 50
    g = torch.Generator().manual_seed(4)
    lat = _hand_lattice(B, L, K, V, seed=3)
    table = torch.round(torch.randn((V, V), generator=g) * 8) / 8
    dlat = SimpleNamespace(**{k: v.to(DEV) for k, v in vars(lat).items()})
    kw = dict(W=3, lam=0.5, eos_id=-1, V=V, proxy_kind=1)
    out = {}
    for name, prev in (("low", [-7, V + 100]), ("clamped", [0, V - 1])):
        c = dsp.dsp_cps_search(dlat, torch.tensor(prev, dtype=torch.int32, device=DEV), table.to(DEV), **kw)
        torch.cuda.synchronize()
        out[name] = c
    for f in ("path", "path_len", "beam_ids", "beam_cum"):
        assert torch.equal(getattr(out["low"], f), getattr(out["clamped"], f)), f
    o = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, torch.tensor([0, V - 1], dtype=torch.int32),
                          table, **kw)
    assert torch.equal(out["clamped"].path.cpu(), o.path) and torch.equal(out["clamped"].beam_cum.cpu(), o.beam_cum)


def test_single_call_step_from_two_host_threads():
    """Two host threads, each with its own stream and buffers, call the one-call step at the same time."""
    import threading
    w = wl.CONFIGS[3].scaled(B=3, L=6, V=40000)
    p = _params(w)
    inps = [wl.make_inputs(w, step=s, device=DEV) for s in (11, 12)]
    want = [gpu_step(i, fused=True, **p) for i in inps]
    got, errs = [None, None], []

    def work(k):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for _ in range(20):
                    got[k] = gpu_step(inps[k], fused=True, **p)
        except Exception as e:                                      # surfaced below
            errs.append(e)
    ts = [threading.Thread(target=work, args=(k,)) for k in (0, 1)]
    [t.start() for t in ts]
    [t.join() for t in ts]
    assert not errs, errs
    for k in (0, 1):
        _same_outputs(want[k], got[k])


def test_target_with_bonus_row_and_all_greedy():
    B, L, V = 4, 5, 3000
    inp = _to(wl.tiny_random(B, L, V, dtype=torch.bfloat16, seed=3))
    extra = (inp["target"][:, :1].float() * 0.5).to(torch.bfloat16)
    inp["target"] = torch.cat([inp["target"], extra], dim=1).contiguous()      # Lt = L + 1
    inp["target"][:, :L] = inp["draft"]                                         # everything accepted
    for ag in (False, True):
        p = dict(K=4, W=4, lam=1.0, all_greedy=ag)
        g = gpu_step(inp, **p)
        check_step(g, inp, **p)
        greedy = torch.ones(B, dtype=torch.bool) if ag else (inp["mode"].cpu() == 0)
        assert (g.ver.accepted_len[greedy] == L).all() and (g.ver.next_token >= 0).all()


def test_ties_everywhere_and_degenerate_rows():
    B, L, V = 3, 2, 20000
    base = wl.tiny_random(B, L, V, dtype=torch.bfloat16, seed=5)
    d = base["draft"]
    d[0] = 1.5                                            # uniform rows: every token ties
    d[1, 0] = torch.arange(V, dtype=torch.float32).mul(1e-3).to(torch.bfloat16)   # ascending, many ties
    d[1, 1] = torch.arange(V, 0, -1, dtype=torch.float32).mul(1e-3).to(torch.bfloat16)
    d[2] = torch.round(d[2].float()).to(torch.bfloat16)   # few distinct values
    base["target"] = (d.float() + 0.25 * torch.round(base["target"].float())).to(torch.bfloat16)
    inp = _to(base)
    p = dict(K=16, W=8, tau=0.0, lam=0.5)
    g = gpu_step(inp, **p)
    check_step(g, inp, **p)
    assert g.lat.cand_id[0, 0].tolist() == list(range(16))


def test_masked_logits_and_nonfinite_flags():
    B, L, V = 4, 3, 9000
    base = wl.tiny_random(B, L, V, dtype=torch.float32, seed=6)
    ninf = -float("inf")
    base["draft"][0, :, 100:] = ninf                      # 100 allowed tokens
    base["target"][0, :, 100:] = ninf
    base["draft"][1, 1, 5:] = ninf                        # fewer finite logits than K
    base["draft"][2, 0, 77] = float("nan")
    base["target"][3, 2, 5] = float("inf")
    inp = _to(base)
    p = dict(K=8, W=4, lam=0.5)
    g = gpu_step(inp, **p)
    check_step(g, inp, **p)
    st = g.lat.row_status
    assert st[2] & dsp.ROW_NONFINITE_INPUT and st[3] & dsp.ROW_NONFINITE_INPUT
    assert not (st[0] & dsp.ROW_NONFINITE_INPUT) and not (st[1] & dsp.ROW_NONFINITE_INPUT)
    assert g.lat.cand_count[1, 1].item() == 5


def test_strided_and_offset_views():
    B, L, V = 3, 4, 10000
    base = wl.tiny_random(B, L, V + 24, dtype=torch.bfloat16, seed=8)
    inp = _to(base)
    full_d, full_t = inp["draft"], inp["target"]
    for off in (0, 3, 8):                                 # 3: rows start 6 bytes off a 16-byte boundary
        view_d, view_t = full_d[:, :, off:off + V], full_t[:, :, off:off + V]
        assert not view_d.is_contiguous()
        inp2 = dict(inp, draft=view_d.contiguous(), target=view_t.contiguous())
        p = dict(K=8, W=8, lam=0.5)
        g = gpu_step(inp, draft=view_d, target=view_t, **p)
        check_step(g, inp2, **p)


def test_run_to_run_determinism():
    w = wl.CONFIGS[3].scaled(B=4, L=4, V=152064)
    inp = wl.make_inputs(w, device=DEV)
    a, b = gpu_step(inp, **_params(w)), gpu_step(inp, **_params(w))
    for s in ("lat", "cps", "ver"):
        for k, v in vars(getattr(a, s)).items():
            assert torch.equal(v.view(torch.uint8), getattr(getattr(b, s), k).view(torch.uint8)), (s, k)


def test_adl_closed_loop_matches_oracle():
    """Configuration 2's loop: the draft length of each step comes from the controller."""
    import oracle
    w = wl.CONFIGS[2].scaled(V=20000, eos_id=19999)
    st, prm = dsp.dsp_adl_init(**wl.ADL_C2)
    ref = oracle.Adl(**wl.ADL_C2)
    walk = wl.eos_walk(12)
    seen = set()
    for t, c in enumerate(walk):
        L = st.k
        assert L == ref.k and L in (8, 16, 24, 32)
        seen.add(L)
        ws = w.scaled(L=L, eos_from=c if c < L else -1)
        inp = wl.make_inputs(ws, step=t, device=DEV)
        g = gpu_step(inp, **_params(ws))
        check_step(g, inp, **_params(ws))
        nxt = dsp.dsp_adl_update(st, prm, g.ver.accepted_len, g.lat.gen_len)
        assert nxt == ref.update(g.ver.accepted_len, g.lat.gen_len)
        assert abs(st.ema_gen - ref.ema_gen) < 1e-12 and abs(st.ema_acc - ref.ema_acc) < 1e-12
    assert len(seen) >= 2


@pytest.mark.parametrize("B", [1, 4])
def test_paper_default_settings(B):
    """The settings of the paper's experiments (Sec. 4, implementation details): draft block 30, at most 15
    candidates per position, beam 3, tau = 0.8, lambda = 0.5, EOS kept, and the controller with
    k in [20, 30], delta = 10, rho = 0.5; greedy verification for batch 1 (the paper's runs), odd rows
    stochastic in the batch of 4."""
    w = wl.CONFIGS[2].scaled(B=B, L=30, K=15, W=3, tau=0.8, lam=0.5, eos_from=23,
                             verify="greedy" if B == 1 else "mixed")
    adl = dict(k_min=20, k_max=30, delta=10.0, rho=0.5, granularity=1)
    st, prm = dsp.dsp_adl_init(**adl)
    ref = oracle.Adl(**adl)
    assert st.k == ref.k == 30                               # Algorithm 1: the first block has k_max tokens
    p = _params(w)
    for step, fused in ((0, False), (1, True)):
        inp = wl.make_inputs(w, step=step, device=DEV)
        g = gpu_step(inp, fused=fused, **p)
        rep = check_step(g, inp, **p)
        assert rep["near_accept"] + rep["near_token"] + rep["near_tau"] <= 1
        assert (g.lat.gen_len == 23).all()                   # EOS is the drafter's top-1 from position 23 on
        assert (g.lat.cand_count <= 16).all() and (g.lat.cand_count >= 1).all()
        nxt = dsp.dsp_adl_update(st, prm, g.ver.accepted_len, g.lat.gen_len)
        assert nxt == ref.update(g.ver.accepted_len, g.lat.gen_len) and 20 <= nxt <= 30
        assert abs(st.ema_gen - ref.ema_gen) < 1e-12 and abs(st.ema_acc - ref.ema_acc) < 1e-12


def test_breadth_closed_loop_matches_oracle():
    """Every step's candidate cap and beam width come from the breadth controller fed with the step before."""
    w0 = wl.CONFIGS[4].scaled(B=4, L=8, V=40000)
    prm_kw = dict(K_min=2, K_max=16, W_min=2, W_max=12, rho=0.5)
    st, prm = dsp.dsp_breadth_init(**prm_kw)
    ref = oracle.Breadth(**prm_kw)
    seen = set()
    for t in range(6):
        K, W = st.K, st.W
        assert (K, W) == (ref.K, ref.W)
        seen.add((K, W))
        w = w0.scaled(K=K, W=W)
        inp = wl.make_inputs(w, step=t, device=DEV)
        g = gpu_step(inp, fused=bool(t & 1), **_params(w))
        check_step(g, inp, **_params(w))
        nxt = dsp.dsp_breadth_update(st, prm, g.lat.entropy, g.ver.accepted_len, g.lat.gen_len)
        assert nxt == ref.update(g.lat.entropy, g.ver.accepted_len, g.lat.gen_len)
        assert st.ema_entropy == ref.ema_entropy and st.ema_shortfall == ref.ema_shortfall
    assert len(seen) >= 2


# ---- the path search alone, on lattices made by hand (sizes and ties the scans rarely give) ----
def _hand_lattice(B, L, KC, V, seed, *, flat=False, counts=None):
    g = torch.Generator().manual_seed(seed)
    cand_id = torch.stack([torch.stack([torch.randperm(V, generator=g)[:KC] for _ in range(L)]) for _ in range(B)])
    if flat:
        logit = torch.zeros(B, L, KC)
    else:
        logit = torch.sort(torch.randn(B, L, KC, generator=g) * 2.0, dim=2, descending=True).values
        logit = torch.round(logit * 4) / 4                 # quarter steps: many equal sums
    cnt = torch.randint(1, KC + 1, (B, L), generator=g) if counts is None else counts
    lse64 = torch.logsumexp(logit.double(), dim=2) + 0.5
    return SimpleNamespace(cand_id=cand_id.int(), cand_logit=logit.float(), lse64=lse64, cand_count=cnt.int())


@pytest.mark.parametrize("kind", [0, 2, 3])             # hashed bigram, tensor of scores, hashed trigram
@pytest.mark.parametrize("B,L,K,W,eos,lam,flat,case", [
    (3, 128, 32, 32, True, 0.5, False, "max"),     # largest K and W with the EOS slot: 1056 expansions, several windows
    (4, 40, 16, 16, True, 0.0, True, "flat"),      # equal logits and a constant proxy: every expansion ties
    (4, 24, 8, 8, False, 1.0, False, "holes"),     # positions without candidates end the lattice
    (6, 32, 16, 16, True, 0.5, False, "eos"),      # the best beam meets EOS and stops
    (5, 33, 5, 7, False, 0.3, False, "odd"),       # W > K, odd sizes
    (2, 1024, 3, 32, True, 0.5, False, "long"),    # the longest draft the library takes
    (4, 40, 8, 8, True, 0.0, True, "flat"),        # small beams (one warp walks the depths): all ties,
    (6, 32, 8, 8, True, 0.5, False, "eos"),        # the early stop,
    (2, 1024, 2, 8, True, 0.5, False, "long"),     # several windows
    (3, 20, 1, 1, False, 0.5, False, "odd"),       # and a single candidate and beam
])
def test_path_search_on_hand_made_lattices(B, L, K, W, eos, lam, flat, case, kind):
    V = 5000
    KC = K + (1 if eos else 0)
    eos_id = 17 if eos else -1
    lat = _hand_lattice(B, L, KC, V, seed=L * 7 + K, flat=flat)
    if case == "holes":
        lat.cand_count[0, 5] = 0
        lat.cand_count[1, 0] = 0
        lat.cand_count[2, L - 1] = 0
    if case == "eos":
        lat.cand_id[0, 3, 0] = eos_id
        lat.cand_id[1, 0, 0] = eos_id
        lat.cand_count[1, 0] = 1                           # the only candidate: the search must stop at once
        lat.cand_id[2, L - 1, 0] = eos_id
        lat.cand_count[2, L - 1] = 1
        lat.cand_id[3, 9, 1] = eos_id                      # not the best candidate: may or may not stop
    g = torch.Generator().manual_seed(99)
    tshape = (B, L, KC, KC) if kind == 2 else (1 << 12,)
    table = torch.zeros(tshape) if flat else torch.round(torch.randn(tshape, generator=g) * 8) / 8 - 3.0
    prev = torch.randint(0, V, (B, 2) if kind == 3 else (B,), generator=g).int()
    kw = dict(W=W, lam=lam, eos_id=eos_id, table_log2=12, hash_seed=5, V=V, proxy_kind=kind)
    o = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, **kw)
    dlat = SimpleNamespace(**{k: v.to(DEV) for k, v in vars(lat).items()})
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    for _ in range(2):                                     # twice: the kernel's state starts clean each time
        c = dsp.dsp_cps_search(dlat, prev.to(DEV), table.to(DEV), row_status=status, **kw)
        torch.cuda.synchronize()
        for name in ("path", "path_slot", "path_len", "beam_ids", "beam_cum"):
            assert torch.equal(getattr(c, name).cpu(), getattr(o, name)), f"{case}: {name} differs"
        assert torch.allclose(c.beam_score.cpu(), o.beam_score, atol=1e-3, rtol=1e-5, equal_nan=True)
    assert torch.equal((status.cpu() & dsp.ROW_EOS_STOPPED) != 0, (o.row_status & oracle.EOS_STOPPED) != 0)
    if case == "holes":
        assert o.path_len[:3].tolist() == [5, 0, L - 1]
    if case == "eos":
        assert o.path_len[1] == 1 and o.path_len[2] == L and (o.row_status[1:3] & oracle.EOS_STOPPED).all()


@pytest.mark.parametrize("kind", [0, 2, 3])
@pytest.mark.parametrize("B,L,K,W,eos,lam,mu", [
    (3, 128, 32, 32, True, 0.5, 0.75),      # largest K and W, several windows
    (5, 33, 5, 7, False, 0.3, -1.25),       # odd sizes, a negative weight
    (4, 24, 8, 8, True, 0.5, 0.0),          # weight 0 with a tensor given
])
def test_path_search_with_a_verifier_side_term(B, L, K, W, eos, lam, mu, kind):
    V = 5000
    KC = K + (1 if eos else 0)
    eos_id = 17 if eos else -1
    lat = _hand_lattice(B, L, KC, V, seed=L * 11 + K)
    g = torch.Generator().manual_seed(123)
    tshape = (B, L, KC, KC) if kind == 2 else (1 << 12,)
    table = torch.round(torch.randn(tshape, generator=g) * 8) / 8 - 3.0
    ver = torch.round(torch.randn((B, L, KC), generator=g) * 8) / 8 - 2.0     # eighths: many equal sums
    prev = torch.randint(0, V, (B, 2) if kind == 3 else (B,), generator=g).int()
    kw = dict(W=W, lam=lam, eos_id=eos_id, table_log2=12, hash_seed=5, V=V, proxy_kind=kind)
    o = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, ver_score=ver, mu=mu, **kw)
    plain = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, **kw)
    if mu != 0.0:
        assert not torch.equal(o.path, plain.path)         # the case does exercise the term
    dlat = SimpleNamespace(**{k: v.to(DEV) for k, v in vars(lat).items()})
    status = torch.zeros(B, dtype=torch.int32, device=DEV)
    c = dsp.dsp_cps_search_biased(dlat, prev.to(DEV), table.to(DEV), ver_score=ver.to(DEV), mu=mu,
                                  row_status=status, **kw)
    torch.cuda.synchronize()
    for name in ("path", "path_slot", "path_len", "beam_ids", "beam_cum"):
        assert torch.equal(getattr(c, name).cpu(), getattr(o, name)), f"{name} differs"
    assert torch.allclose(c.beam_score.cpu(), o.beam_score, atol=1e-3, rtol=1e-5, equal_nan=True)
    assert torch.allclose(c.path_score.cpu(), o.path_score, atol=1e-3, rtol=1e-5)
    assert torch.equal((status.cpu() & dsp.ROW_EOS_STOPPED) != 0, (o.row_status & oracle.EOS_STOPPED) != 0)
    # no tensor: the plain search bit for bit, whatever the weight
    n = dsp.dsp_cps_search_biased(dlat, prev.to(DEV), table.to(DEV), ver_score=None, mu=3.0, **kw)
    q = dsp.dsp_cps_search(dlat, prev.to(DEV), table.to(DEV), **kw)
    torch.cuda.synchronize()
    for name in ("path", "path_slot", "path_len", "path_score", "beam_ids", "beam_cum", "beam_score"):
        assert torch.equal(getattr(n, name), getattr(q, name)), f"no tensor: {name} differs"
    assert torch.equal(q.path.cpu(), plain.path)


def test_verifier_side_term_rejects_a_non_finite_weight():
    lat = _hand_lattice(1, 4, 3, 100, seed=1)
    dlat = SimpleNamespace(**{k: v.to(DEV) for k, v in vars(lat).items()})
    prev = torch.zeros(1, dtype=torch.int32, device=DEV)
    table = torch.zeros(1 << 4, device=DEV)
    ver = torch.zeros((1, 4, 3), device=DEV)
    for bad in (float("nan"), float("inf")):
        with pytest.raises(dsp.DspError):
            dsp.dsp_cps_search_biased(dlat, prev, table, ver_score=ver, mu=bad, W=2, lam=0.5, table_log2=4, V=100)


@pytest.mark.parametrize("seed", range(8))
def test_path_search_on_random_shapes(seed):
    """Seeded random shapes across both forms of the walk (one warp for small beams, the whole CTA for
    large ones), with quantised scores (ties), ragged counts, EOS among the candidates and all proxies."""
    rng = np.random.default_rng(1000 + seed)
    for case in range(6):
        B = int(rng.integers(1, 5))
        L = int(rng.integers(1, 70))
        K = int(rng.choice([1, 2, 3, 5, 8, 11, 16, 32]))
        W = int(rng.choice([1, 2, 3, 4, 8, 12, 16, 32]))
        eos = bool(rng.integers(0, 2))
        kind = int(rng.choice([0, 1, 2, 3]))
        lam = float(rng.choice([0.0, 0.25, 0.5, 1.0]))
        V = 300 if kind == 1 else 5000
        KC = K + (1 if eos else 0)
        eos_id = 17 if eos else -1
        lat = _hand_lattice(B, L, KC, V, seed=seed * 100 + case)
        if eos and L > 2:                                  # EOS somewhere among the candidates of one row
            lat.cand_id[0, int(rng.integers(0, L)), int(rng.integers(0, KC))] = eos_id
        if case % 3 == 2 and L > 3:
            lat.cand_count[B - 1, int(rng.integers(1, L))] = 0     # a hole ends that lattice
        g = torch.Generator().manual_seed(seed * 7 + case)
        tshape = {0: (1 << 10,), 1: (V, V), 2: (B, L, KC, KC), 3: (1 << 10,)}[kind]
        table = torch.round(torch.randn(tshape, generator=g) * 4) / 4 - 3.0
        prev = torch.randint(0, V, (B, 2) if kind == 3 else (B,), generator=g).int()
        ver = torch.round(torch.randn((B, L, KC), generator=g) * 4) / 4 if case % 2 else None
        kw = dict(W=W, lam=lam, eos_id=eos_id, table_log2=10, hash_seed=seed, V=V, proxy_kind=kind)
        o = oracle.cps_search(lat.cand_id, lat.cand_logit, lat.lse64, lat.cand_count, prev, table, ver_score=ver, mu=0.75, **kw)
        dlat = SimpleNamespace(**{k: v.to(DEV) for k, v in vars(lat).items()})
        status = torch.zeros(B, dtype=torch.int32, device=DEV)
        c = dsp.dsp_cps_search_biased(dlat, prev.to(DEV), table.to(DEV), ver_score=None if ver is None else ver.to(DEV),
                                      mu=0.75, row_status=status, **kw)
        torch.cuda.synchronize()
        what = f"seed {seed} case {case}: B={B} L={L} K={K} W={W} eos={eos} kind={kind} lam={lam}"
        for name in ("path", "path_slot", "path_len", "beam_ids", "beam_cum"):
            assert torch.equal(getattr(c, name).cpu(), getattr(o, name)), f"{what}: {name} differs"
        assert torch.allclose(c.beam_score.cpu(), o.beam_score, atol=1e-3, rtol=1e-5, equal_nan=True), what
        assert torch.equal((status.cpu() & dsp.ROW_EOS_STOPPED) != 0, (o.row_status & oracle.EOS_STOPPED) != 0), what


# ---- the step recorded as a CUDA graph ----
def _same_outputs(a, b, w=None):
    for s in ("lat", "cps", "ver"):
        for k, v in vars(getattr(a, s)).items():
            if v is None or (w is not None and all_greedy_unused(w, s, k)):
                continue
            assert torch.equal(v.cpu().view(torch.uint8), getattr(getattr(b, s), k).cpu().view(torch.uint8)), (s, k)


def _graph_kwargs(inp, p):
    kw = dict(K_max=p["K"], W=p["W"], lam=p["lam"], tau=p["tau"], eos_id=p["eos_id"],
              table_log2=inp["table_log2"], hash_seed=inp["hash_seed"], all_greedy=p["all_greedy"])
    if not p["all_greedy"]:
        kw.update(mode=inp["mode"], u=inp["u"])
    return kw


@pytest.mark.parametrize("cid", [1, 2, 3, 4])
def test_step_graph_replays_the_step(cid):
    w = wl.CONFIGS[cid].scaled(**SMALL[cid])
    if cid == 4:
        w = w.scaled(V=50048)
    p = _params(w)
    inp = wl.make_inputs(w, step=3, device=DEV)
    other = wl.make_inputs(w, step=4, device=DEV)
    graph = dsp.dsp_step_graph_create(inp["draft"], inp["target"], inp["prev_token"], inp["table"],
                                      **_graph_kwargs(inp, p))
    for rep in range(3):
        if rep == 1:                                       # new logits in place: the graph reads the same addresses
            for k in ("draft", "target", "prev_token", "u"):
                inp[k].copy_(other[k])
        graph.launch()
        torch.cuda.synchronize()
        ns = SimpleNamespace(lat=graph.lat, cps=graph.cps, ver=graph.ver)
        _same_outputs(gpu_step(inp, fused=True, **p), ns, w)
    cpu = lambda x: SimpleNamespace(**{k: (v.cpu() if v is not None else None) for k, v in vars(x).items()})
    check_step(SimpleNamespace(lat=cpu(graph.lat), cps=cpu(graph.cps), ver=cpu(graph.ver)), inp, **p)
    graph.destroy()
    graph.destroy()                                        # a second destroy is harmless


def test_step_graphs_per_draft_length_share_buffers():
    """One graph per draft length (the controller's buckets) over the same logits buffers and workspaces."""
    B, Lmax, V, K, W = 3, 16, 16384, 8, 4
    inp = _to(wl.tiny_random(B, Lmax, V, dtype=torch.bfloat16, seed=21))
    p = dict(K=K, W=W, tau=0.0, lam=0.5, eos_id=-1, all_greedy=False)
    dt = dsp.DSP_BF16
    ws_l = dsp.alloc_workspace(dsp.dsp_lattice_workspace_bytes(B, Lmax, V, dt, K), DEV)
    ws_v = dsp.alloc_workspace(dsp.dsp_verify_workspace_bytes(B, Lmax, Lmax, V, dt), DEV)
    graphs = {}
    for L in (4, 8, 16):
        view = dict(inp, draft=inp["draft"][:, :L], target=inp["target"][:, :L], u=inp["u"][:, :L + 1].contiguous())
        graphs[L] = (view, dsp.dsp_step_graph_create(view["draft"], view["target"], view["prev_token"], view["table"],
                                                     lattice_workspace=ws_l, verify_workspace=ws_v,
                                                     **_graph_kwargs(view, p)))
    for L in (8, 16, 4, 16):
        view, graph = graphs[L]
        graph.launch()
        torch.cuda.synchronize()
        _same_outputs(gpu_step(view, fused=True, **p), SimpleNamespace(lat=graph.lat, cps=graph.cps, ver=graph.ver))
    with pytest.raises(dsp.DspError):                      # argument errors surface at creation, nothing is left captured
        dsp.dsp_step_graph_create(inp["draft"], inp["target"], inp["prev_token"], inp["table"], K_max=K, W=999,
                                  lam=0.5, table_log2=10, mode=inp["mode"], u=inp["u"])
    g = gpu_step(inp, fused=True, **p)                     # the library still works after the refused capture
    check_step(g, inp, **p)


@pytest.mark.parametrize("kind", [2, 3])
def test_whole_step_with_tensor_and_trigram_proxies(kind):
    w = wl.CONFIGS[3].scaled(**SMALL[3])
    inp = wl.make_inputs(w, step=5, device=DEV)
    p = _params(w)
    g = torch.Generator().manual_seed(kind)
    if kind == 2:
        KC = w.K + (1 if w.eos_id >= 0 else 0)
        inp["table"] = (-6.0 * torch.rand((w.B, w.L, KC, KC), generator=g)).to(DEV)
    else:
        inp["prev_token"] = torch.randint(0, w.V, (w.B, 2), generator=g, dtype=torch.int32).to(DEV)
    for fused in (False, True):
        check_step(gpu_step(inp, proxy_kind=kind, fused=fused, **p), inp, proxy_kind=kind, **p)


# ---- the lattice from vocabulary slices (tensor-parallel drafter head) ----
def _sharded_lattice(x, cuts, K, tau, eos_id):
    """Slice records one after the other on this GPU, stacked slice-major (the all-gather's layout), merged."""
    recs = []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        recs.append(dsp.dsp_lattice_shard(x[:, :, lo:hi], lo, K, eos_id))
    stack = lambda name: torch.stack([getattr(r, name) for r in recs], dim=0).contiguous()
    return dsp.dsp_lattice_merge(stack("sums"), stack("keys"), stack("status"), x.shape[2], K, tau, eos_id)


@pytest.mark.parametrize("B,L,V,dtype,K,cuts", [
    (3, 5, 152064, torch.bfloat16, 16, [0, 38016, 76032, 114048, 152064]),      # four equal, aligned slices
    (2, 4, 152064, torch.bfloat16, 32, [0, 19008 * 3, 19008 * 4, 152064]),      # unequal slices
    (2, 3, 50021, torch.bfloat16, 8, [0, 16384, 16391, 50021]),                 # unaligned slices: element-wise path
    (2, 6, 12288, torch.float32, 4, [0, 12288]),                                # one slice
    (1, 2, 4096, torch.float32, 32, [0, 8, 16, 24, 4096]),                      # slices shorter than K_max
])
def test_lattice_from_vocabulary_slices_equals_the_whole_row_build(B, L, V, dtype, K, cuts):
    g = torch.Generator().manual_seed(V + K)
    x = (2.5 * torch.randn((B, L, V), generator=g)).to(dtype)
    x[0, 0, 100:200] = float("-inf")                       # masked tokens
    if B > 1:
        x[1, 1, :cuts[1]] = float("-inf")                  # a slice without a finite logit
    eos = V - 3
    x[0, L - 1, eos] = 30.0                                # EOS on top at the last position: gen_len = L - 1
    x = x.to(DEV)
    for tau, eos_id in ((0.0, -1), (0.8, eos)):
        whole = dsp.dsp_lattice_build(x, K, tau, eos_id)
        parts = _sharded_lattice(x, cuts, K, tau, eos_id)
        torch.cuda.synchronize()
        for name in ("cand_id", "cand_logit", "cand_count", "gen_len", "row_status"):
            assert torch.equal(getattr(parts, name), getattr(whole, name)), name
        assert torch.allclose(parts.lse64, whole.lse64, atol=1e-6, rtol=0, equal_nan=True)
        assert torch.allclose(parts.entropy, whole.entropy, atol=1e-5, rtol=0, equal_nan=True)
        assert torch.allclose(parts.cand_logp, whole.cand_logp, atol=1e-5, rtol=0, equal_nan=True)
        o = oracle.lattice_build(x.cpu(), K, tau=tau, eos_id=eos_id)
        good = (o.row_status & oracle.NONFINITE_INPUT) == 0     # a row without a finite logit flags its batch row
        assert torch.equal(parts.row_status.cpu() != 0, ~good)
        assert torch.equal(parts.cand_id.cpu()[good], o.cand_id[good])
        assert torch.equal(parts.cand_count.cpu()[good], o.cand_count[good])
        assert torch.equal(parts.gen_len.cpu()[good], o.gen_len[good])
        assert torch.allclose(parts.lse64.cpu()[good], o.lse64[good], atol=1e-5, rtol=0)
        assert torch.allclose(parts.entropy.cpu()[good], o.entropy[good], atol=1e-3, rtol=0)
        fin = torch.isfinite(o.cand_logp) & good.view(-1, 1, 1)
        assert (parts.cand_logp.cpu()[fin] - o.cand_logp[fin]).abs().max() <= 1e-3


def test_lattice_from_slices_flags_nonfinite_rows():
    B, L, V, K = 2, 3, 16384, 4
    x = torch.randn((B, L, V)).to(torch.bfloat16)
    x[1, 2, 9000] = float("nan")
    x = x.to(DEV)
    out = _sharded_lattice(x, [0, 8192, 16384], K, 0.0, -1)
    torch.cuda.synchronize()
    assert out.row_status.cpu().tolist() == [0, dsp.ROW_NONFINITE_INPUT]


def _sharded_verify(inp, lat, cps, cuts, eos_id, all_greedy):
    """dsp_verify from vocabulary slices of the target: records per slice, merge, gathered rows, draw."""
    target, draft = inp["target"], inp["draft"]
    B, Lt, V = target.shape
    L = draft.shape[1]
    recs = [dsp.dsp_target_shard(target[:, :, lo:hi], lo, cps) for lo, hi in zip(cuts[:-1], cuts[1:])]
    stack = lambda name: torch.stack([getattr(r, name) for r in recs], dim=0).contiguous()
    ver = dsp.dsp_verify_merge(stack("sums"), stack("keys"), stack("status"), cps, None if all_greedy else lat,
                               mode=None if all_greedy else inp["mode"], u=None if all_greedy else inp["u"],
                               eos_id=eos_id, all_greedy=all_greedy)
    if not all_greedy:
        # what the all-gather of the named rows' slices leaves on every GPU: the whole rows, one per batch row
        trow = ver.job_trow.long().clamp(min=0)
        drow = ver.job_drow.long().clamp(min=0)
        target_rows = torch.cat([target[:, :, lo:hi].reshape(B * Lt, hi - lo)[trow] for lo, hi in zip(cuts[:-1], cuts[1:])], dim=1)
        draft_rows = torch.cat([draft[:, :, lo:hi].reshape(B * L, hi - lo)[drow] for lo, hi in zip(cuts[:-1], cuts[1:])], dim=1)
        dsp.dsp_residual_sample(target_rows.contiguous(), draft_rows.contiguous(), ver, lat, inp["u"], L)
    torch.cuda.synchronize()
    return ver


@pytest.mark.parametrize("cid,cuts", [(3, [0, 38016, 76032, 114048, 152064]), (4, [0, 16384, 50048]),
                                      (1, [0, 8000, 16000, 24000, 32000]), (5, [0, 128000, 256000])])
def test_verification_from_vocabulary_slices_of_the_target(cid, cuts):
    w = wl.CONFIGS[cid].scaled(**SMALL[cid])
    if cid == 4:
        w = w.scaled(V=50048)
    p = _params(w)
    inp = wl.make_inputs(w, step=6, device=DEV)
    whole = gpu_step(inp, **p)                             # the three unsharded calls, CPU copies
    lat = dsp.dsp_lattice_build(inp["draft"], w.K, w.tau, w.eos_id)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=w.W, lam=w.lam, eos_id=w.eos_id,
                             table_log2=inp["table_log2"], hash_seed=inp["hash_seed"], V=w.V)
    ver = _sharded_verify(inp, lat, cps, cuts, w.eos_id, p["all_greedy"])
    assert torch.equal(ver.accepted_len.cpu(), whole.ver.accepted_len)
    assert torch.equal(ver.tgt_argmax.cpu(), whole.ver.tgt_argmax)
    assert torch.equal(ver.next_token.cpu(), whole.ver.next_token)
    if not p["all_greedy"]:
        stoch = inp["mode"].cpu() != 0
        assert torch.allclose(ver.tgt_lse.cpu()[stoch], whole.ver.tgt_lse[stoch], atol=1e-5, rtol=0)
        assert torch.allclose(ver.ratio.cpu(), whole.ver.ratio, atol=1e-5, rtol=1e-4)
    # and against the oracle: the sharded verification in place of the unsharded one
    cpu = lambda x: SimpleNamespace(**{k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in vars(x).items()})
    g = SimpleNamespace(lat=whole.lat, cps=whole.cps, ver=cpu(ver))
    g.lat.row_status = whole.lat.row_status | ver.row_status.cpu()
    if not p["all_greedy"]:
        greedy = inp["mode"].cpu() == 0
        g.ver.tgt_lse[greedy] = float("nan")               # dsp_verify leaves these unset
    check_step(g, inp, **p)


def test_sharded_verification_with_a_bonus_row():
    """Lt = L + 1 and a target that accepts everything: the draw comes from the extra row (no draft row)."""
    B, L, V = 4, 5, 4096
    inp = _to(wl.tiny_random(B, L, V, dtype=torch.bfloat16, seed=3))
    extra = (inp["target"][:, :1].float() * 0.5).to(torch.bfloat16)
    inp["target"] = torch.cat([inp["target"], extra], dim=1).contiguous()
    inp["target"][:, :L] = inp["draft"]
    p = dict(K=4, W=4, lam=1.0)
    whole = gpu_step(inp, **p)
    lat = dsp.dsp_lattice_build(inp["draft"], 4)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=4, lam=1.0, table_log2=inp["table_log2"],
                             hash_seed=inp["hash_seed"], V=V)
    ver = _sharded_verify(inp, lat, cps, [0, 1024, 1032, 4096], -1, False)
    stoch = inp["mode"].cpu() != 0
    assert (ver.job_drow.cpu()[stoch] == -1).all() and (ver.job_trow.cpu()[~stoch] == -1).all()
    assert torch.equal(ver.accepted_len.cpu(), whole.ver.accepted_len)
    assert torch.equal(ver.next_token.cpu(), whole.ver.next_token) and (ver.next_token >= 0).all()


# ---- several paths in one target pass: the beams as a token tree, verified greedily ----
@pytest.mark.parametrize("B,L,V,K,W,dtype", [
    (3, 6, 32000, 4, 8, torch.float32),
    (2, 8, 152064, 8, 16, torch.bfloat16),
    (4, 5, 50021, 3, 4, torch.bfloat16),     # rows that are not 16-byte aligned
    (2, 12, 4096, 2, 1, torch.float32),      # one beam: a chain
])
def test_beam_tree_and_its_greedy_verification(B, L, V, K, W, dtype):
    inp = _to(wl.tiny_random(B, L, V, dtype=dtype, seed=L + W))
    lat = dsp.dsp_lattice_build(inp["draft"], K)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=W, lam=0.5, table_log2=inp["table_log2"],
                             hash_seed=inp["hash_seed"], V=V)
    tree = dsp.dsp_beam_tree(cps)
    torch.cuda.synchronize()
    ot = oracle.beam_tree(cps.beam_ids.cpu(), cps.path_len.cpu())
    for name in ("node_token", "node_parent", "node_depth", "beam_node", "n_nodes"):
        assert torch.equal(getattr(tree, name).cpu(), getattr(ot, name)), name
    assert int(ot.n_nodes.max()) > L or W == 1              # the beams do branch
    # target rows: noise plus a push towards one child's token at every existing context, so walks go deep
    N = W * L
    g = torch.Generator().manual_seed(5)
    target = torch.randn((B, 1 + N, V), generator=g)
    for b in range(B):
        for n in range(int(ot.n_nodes[b])):
            if (n * 7 + b) % 3:                              # two contexts in three favour a child
                target[b, 1 + int(ot.node_parent[b, n]), int(ot.node_token[b, n])] += 9.0
        target[b, 1 + int(ot.n_nodes[b]):] = float("nan")    # rows of unused slots must not matter
    target = target.to(dtype)
    out = dsp.dsp_verify_tree(target.to(DEV), tree, L)
    torch.cuda.synchronize()
    o = oracle.verify_tree(target, ot, L)
    assert (o.row_status == 0).all() and (out.row_status.cpu() == 0).all()
    for name in ("accepted_len", "accepted_node", "next_token"):
        assert torch.equal(getattr(out, name).cpu(), getattr(o, name)), name
    assert int(o.accepted_len.max()) >= 2
    target[0, 1, 5] = float("nan")                           # an existing row goes bad: the batch row is flagged
    out = dsp.dsp_verify_tree(target.to(DEV), tree, L)
    o = oracle.verify_tree(target, ot, L)
    torch.cuda.synchronize()
    assert (out.row_status.cpu() != 0).tolist() == (o.row_status != 0).tolist() == [True] + [False] * (B - 1)


@pytest.mark.parametrize("B,L,V,K,W,dtype,sigma", [
    (4, 5, 3000, 4, 6, torch.float32, 0.7),
    (3, 6, 20000, 4, 8, torch.bfloat16, 0.3),     # target close to the draft: deep walks
    (3, 4, 5003, 3, 4, torch.bfloat16, 1.5),      # rows that are not 16-byte aligned; many rejections
    (2, 8, 1000, 2, 1, torch.float32, 0.5),       # one beam: the single-path rule
    (2, 3, 300000, 3, 2, torch.bfloat16, 1.0),    # more chunks than threads: several chunks per thread in the draw
    (2, 4, 152064, 4, 4, torch.bfloat16, 2.5),    # a target far from the draft: chains of rejections
    (3, 5, 40001, 3, 3, torch.float32, 0.1),      # fp32 rows that are not 16-byte aligned; long accepted walks
    (2, 16, 20000, 4, 4, torch.bfloat16, 0.4),    # few draft rows beside many target rows: the draft rows' statistics
                                                  # cut their rows into more slices than the target rows' (workspace sizing)
])
def test_stochastic_tree_verification_matches_oracle(B, L, V, K, W, dtype, sigma):
    inp = _to(wl.tiny_random(B, L, V, dtype=dtype, seed=L * 3 + W))
    lat = dsp.dsp_lattice_build(inp["draft"], K)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=W, lam=0.5, table_log2=inp["table_log2"],
                             hash_seed=inp["hash_seed"], V=V)
    tree = dsp.dsp_beam_tree(cps)
    torch.cuda.synchronize()
    ot = oracle.beam_tree(cps.beam_ids.cpu(), cps.path_len.cpu())
    N = W * L
    g = torch.Generator().manual_seed(B + W)
    draft = inp["draft"].cpu()
    # a causal target: the row after a node is the draft row of the next depth plus noise (row 0: depth 0)
    target = torch.zeros((B, 1 + N, V))
    for b in range(B):
        for r in range(1 + int(ot.n_nodes[b])):
            depth = 0 if r == 0 else int(ot.node_depth[b, r - 1]) + 1
            base = draft[b, min(depth, L - 1)].float()
            target[b, r] = base + sigma * torch.randn(V, generator=g)
        target[b, 1 + int(ot.n_nodes[b]):] = float("nan")    # rows of unused slots must not matter
    target = target.to(dtype)
    u = torch.rand((B, N + 1), generator=g)
    o = oracle.verify_tree_stochastic(target, draft, ot, u)
    out = dsp.dsp_verify_tree_stochastic(target.to(DEV), inp["draft"], tree, u.to(DEV))
    torch.cuda.synchronize()
    assert (o.row_status == 0).all() and (out.row_status.cpu() == 0).all()
    # The walk's row sums are fp32 terms added up in double, the oracle's are double throughout: a batch
    # row may differ only if its closest decision (acceptance ratio against u, or the emitted token's step
    # of the cumulative sum against u) was within 1e-5 of going the other way, and that is rare.
    near = 0
    for b in range(B):
        same = all(torch.equal(getattr(out, name).cpu()[b], getattr(o, name)[b])
                   for name in ("accepted_len", "accepted_node", "next_token"))
        assert same or o.margin[b] < 1e-5, f"batch row {b} differs with margin {o.margin[b]:.3g}"
        near += 0 if same else 1
    assert near <= 1
    assert (out.next_token >= 0).all()
    if W > 1:                                                # one path alone would have done no better
        single = oracle.verify_tree_stochastic(target, draft, SimpleNamespace(
            node_token=ot.node_token, node_parent=ot.node_parent, n_nodes=cps.path_len.cpu()), u)
        assert (o.accepted_len >= single.accepted_len).all()
    bad = target.clone()
    bad[0, 1, 3] = float("nan")                              # an existing row goes bad: the batch row is flagged
    out = dsp.dsp_verify_tree_stochastic(bad.to(DEV), inp["draft"], tree, u.to(DEV))
    torch.cuda.synchronize()
    ob = oracle.verify_tree_stochastic(bad, draft, ot, u)
    assert ((out.row_status.cpu() & dsp.ROW_NONFINITE_INPUT) != 0).tolist() == ((ob.row_status & oracle.NONFINITE_INPUT) != 0).tolist()


# ---- the drafter's refinement step (Eq. 5) ----
def _check_unmask(x, tokens, masked, n, ws=None):
    """One step on both sides from the same state; returns the new state (the GPU's)."""
    t_gpu, m_gpu = tokens.to(DEV), masked.to(DEV)
    g = dsp.dsp_unmask_step(x, t_gpu, m_gpu, n, workspace=ws)
    torch.cuda.synchronize()
    o = oracle.unmask_step(x.cpu(), tokens, masked, n)
    good = (o.row_status & oracle.NONFINITE_INPUT) == 0
    assert torch.equal((g.row_status.cpu() & dsp.ROW_NONFINITE_INPUT) != 0, ~good)
    was = masked.bool()
    assert torch.equal(g.argmax.cpu()[good], o.argmax[good])
    conf = g.confidence.cpu()
    assert torch.equal(torch.isinf(conf), torch.isinf(o.confidence))
    fin = torch.isfinite(o.confidence) & good.view(-1, 1)
    assert (conf[fin] - o.confidence[fin]).abs().max().item() <= 1e-3 if fin.any() else True
    assert (g.argmax.cpu()[~was] == -1).all()
    assert torch.equal(g.n_left.cpu()[good], o.n_left[good])
    for b in torch.nonzero(good).flatten().tolist():
        if torch.equal(m_gpu[b].cpu(), o.masked[b]):
            assert torch.equal(t_gpu[b].cpu(), o.tokens[b])
            continue
        # a different choice is only right where the two confidences are a rounding apart
        diff = torch.nonzero(m_gpu[b].cpu() != o.masked[b]).flatten().tolist()
        cs = o.confidence[b, diff]
        assert len(diff) == 2 and (cs.max() - cs.min()).item() <= 2e-5, (b, diff, cs)
    return t_gpu.cpu(), m_gpu.cpu()


@pytest.mark.parametrize("B,L,V,dtype,S", [
    (3, 6, 152064, torch.bfloat16, 3),       # the drafter's vocabulary: several tiles, ragged tail, slices
    (2, 5, 12288, torch.float32, 2),         # fp32 rows of exactly three tiles
    (4, 7, 50021, torch.bfloat16, 4),        # odd V: rows are not 16-byte aligned -> element-wise path
    (2, 40, 37, torch.float32, 1),           # S = 1: everything at once
    (1, 1, 1, torch.float32, 1),             # one position, one token
])
def test_unmask_step_matches_oracle_over_a_whole_refinement(B, L, V, dtype, S):
    g = torch.Generator().manual_seed(B * 1000 + L)
    x = (3.0 * torch.randn((B, L, V), generator=g)).to(dtype).to(DEV)
    tokens = torch.full((B, L), -7, dtype=torch.int32)
    masked = torch.ones((B, L), dtype=torch.uint8)
    if B > 1:
        masked[1, ::2] = 0                                # a batch row that starts half revealed
    n = -(-L // S)
    ws = dsp.alloc_workspace(dsp.dsp_unmask_workspace_bytes(B, L, V, dsp.DSP_BF16 if dtype == torch.bfloat16 else dsp.DSP_F32), DEV)
    for s in range(S):
        tokens, masked = _check_unmask(x, tokens, masked, n, ws)
    assert masked.sum() == 0
    am = x.float().argmax(dim=-1).cpu().int()
    keep = tokens != -7
    assert torch.equal(tokens[keep], am[keep])


def test_unmask_step_ties_masked_logits_and_flags():
    B, L, V = 4, 5, 16384
    g = torch.Generator().manual_seed(8)
    x = (2.0 * torch.randn((B, L, V), generator=g)).to(torch.bfloat16)
    x[0] = 0.5                                            # every position ties: lower positions first, argmax 0
    x[1, :, 100:] = float("-inf")                         # masked vocabulary
    x[2, 3, 77] = float("nan")                            # flagged only while position 3 is masked
    x[3, 1, :] = float("-inf")                            # no finite logit
    x = x.to(DEV)
    tokens = torch.zeros((B, L), dtype=torch.int32)
    masked = torch.ones((B, L), dtype=torch.uint8)
    masked[2, 3] = 0
    t1, m1 = _check_unmask(x, tokens, masked, 2)
    assert m1[0].tolist() == [0, 0, 1, 1, 1] and t1[0].tolist() == [0, 0, 0, 0, 0]
    masked[2, 3] = 1
    _check_unmask(x, tokens, masked, 2)
    with pytest.raises(dsp.DspError):
        dsp.dsp_unmask_step(x, tokens.to(DEV), masked.to(DEV), 0)


def test_longest_draft_through_the_whole_step_and_the_refinement():
    """L = DSP_MAX_L with a small vocabulary: every kernel's per-batch-row bookkeeping at its largest."""
    B, L, V = 2, dsp.DSP_MAX_L, 2048
    inp = _to(wl.tiny_random(B, L, V, dtype=torch.bfloat16, seed=31))
    p = dict(K=4, W=4, tau=0.0, lam=0.5, eos_id=-1)
    check_step(gpu_step(inp, fused=True, **p), inp, **p)
    tokens = torch.zeros((B, L), dtype=torch.int32)
    masked = torch.ones((B, L), dtype=torch.uint8)
    for _ in range(2):
        tokens, masked = _check_unmask(inp["draft"], tokens, masked, L // 2)
    assert masked.sum() == 0
    with pytest.raises(dsp.DspError):
        dsp.dsp_lattice_build(torch.zeros((1, L + 1, 64), device=DEV), 4)


def test_many_batch_rows():
    """Thousands of short rows: grids, tickets and per-batch-row state far beyond the benchmark's batch sizes."""
    B, L, V = 6000, 2, 256
    inp = _to(wl.tiny_random(B, L, V, dtype=torch.float32, seed=41))
    p = dict(K=4, W=2, tau=0.7, lam=0.5, eos_id=5)
    rep = check_step(gpu_step(inp, fused=True, **p), inp, **p)
    assert rep["near_accept"] + rep["near_token"] + rep["near_tau"] <= 6
    tokens = torch.zeros((B, L), dtype=torch.int32)
    masked = torch.ones((B, L), dtype=torch.uint8)
    _check_unmask(inp["draft"], tokens, masked, 1)


def test_profile_events_bracket_the_scan_kernels():
    w = wl.CONFIGS[3].scaled(B=2, L=4, V=152064)
    inp = wl.make_inputs(w, device=DEV)
    pairs = []
    for point in (dsp.PROFILE_LATTICE_SCAN, dsp.PROFILE_TARGET_SCAN):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); b.record()
        dsp.dsp_profile_events(point, a, b)
        pairs.append((a, b))
    try:
        g = gpu_step(inp, **_params(w))
    finally:
        for point in (dsp.PROFILE_LATTICE_SCAN, dsp.PROFILE_TARGET_SCAN):
            dsp.dsp_profile_events(point, None, None)
    check_step(g, inp, **_params(w))
    for a, b in pairs:
        assert 0.0 < a.elapsed_time(b) < 50.0          # milliseconds
    with pytest.raises(dsp.DspError):
        dsp.dsp_profile_events(7, None, None)


@pytest.mark.parametrize("cid", [1, 2, 3, 4, 5])
def test_single_call_step_equals_the_three_calls(cid):
    w = wl.CONFIGS[cid].scaled(**SMALL[cid])
    if cid == 4:
        w = w.scaled(V=50048)                              # an aligned layout: the streaming kernels
    inp = wl.make_inputs(w, step=2, device=DEV)
    for rep in range(2):                                  # twice: the second stream is reused
        a = gpu_step(inp, **_params(w))
        b = gpu_step(inp, fused=True, **_params(w))
        for s in ("lat", "cps", "ver"):
            for k, v in vars(getattr(a, s)).items():
                if v is None:
                    continue
                o = getattr(getattr(b, s), k)
                if all_greedy_unused(w, s, k):
                    continue
                assert torch.equal(v.view(torch.uint8), o.view(torch.uint8)), (s, k)
    check_step(b, inp, **_params(w))


@pytest.mark.parametrize("B,L", [(64, 32), (96, 24)])
def test_single_call_step_on_long_passes_equals_the_three_calls(B, L):
    """Logits tensors of 400 MB and more take the other stream arrangement of the single call (the
    lattice's finish and the search on the library's high-priority stream); up to 74 batch rows
    the search also keeps its SMs to itself, with more it shares them.  Same bytes either way."""
    w = wl.CONFIGS[4].scaled(B=B, L=L)
    assert w.logits_bytes >= 400 << 20
    inp = wl.make_inputs(w, step=5, device=DEV)
    a = gpu_step(inp, **_params(w))
    for rep in range(2):
        b = gpu_step(inp, fused=True, **_params(w))
        for s in ("lat", "cps", "ver"):
            for k, v in vars(getattr(a, s)).items():
                if v is not None:
                    assert torch.equal(v.view(torch.uint8), getattr(getattr(b, s), k).view(torch.uint8)), (s, k)
    check_step(b, inp, rows=[0, 1, B // 2, B - 1], **_params(w))
    del inp
    torch.cuda.empty_cache()


def test_read_probe_runs_and_rejects_bad_arguments():
    x = torch.zeros(1 << 22, dtype=torch.bfloat16, device=DEV)
    sink = torch.zeros(1, dtype=torch.int32, device=DEV)
    for _ in range(3):
        dsp.dsp_read_probe(x, sink)
    dsp.dsp_read_probe(x[: 8 * 1000 + 8], sink)           # a ragged last piece
    torch.cuda.synchronize()
    assert int(sink[0]) == 0                              # zeros never fold to the stored value
    with pytest.raises(dsp.DspError):
        dsp.dsp_read_probe(x[1:9], sink)                  # not 16-byte aligned
    with pytest.raises(dsp.DspError):
        dsp.dsp_read_probe(x[:4], sink)                   # fewer than 16 bytes


def all_greedy_unused(w, s, k):
    """Outputs that a greedy-only verification does not write."""
    return w.verify == "greedy" and s == "ver" and k in ("ratio", "tgt_lse")
