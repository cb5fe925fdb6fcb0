"""GPU-vs-oracle comparison of one whole draft-and-verify step (helper, not a test file).

``gpu_step`` runs the CUDA path through the binding; ``check_step`` runs the
oracle on the same bytes and compares field by field:

* integers (candidate ids and counts, generation length, paths, slots, path
  lengths, beams, accepted lengths, greedy tokens, target argmax) and the
  candidate logits must be identical;
* log-probabilities, log-sum-exps and entropies within 1e-3 absolute; path and
  beam scores within 1e-3 + 1e-5*|S|; acceptance ratios within 1e-5 + 1e-4*ratio;
  the fp32 ranking quantity of the beams bit for bit;
* every oracle stage is also run on the GPU's upstream outputs (stage-isolated),
  so a tolerated upstream difference cannot hide a downstream error;
* the only tolerated integer differences are near-ties of a floating-point
  comparison, each counted and returned: Eq. 7's cumulative mass within 1e-6 of
  tau, an acceptance draw with |u - p/q| < 1e-6, and a sampled token whose
  oracle CDF interval, widened by 1e-6, contains the draw.
"""
from __future__ import annotations

from types import SimpleNamespace

import torch

import oracle
from paper_2510_02358_b200 import binding as dsp

TOL_LOGP = 1e-3
NEAR = 1e-6


def gpu_step(inp: dict, *, K: int, W: int, tau: float = 0.0, lam: float = 0.5, eos_id: int = -1,
             all_greedy: bool = False, proxy_kind: int = 0, target=None, draft=None,
             fused: bool = False) -> SimpleNamespace:
    """One step on the GPU; ``inp`` holds CUDA tensors. Returns CPU copies of every output.
    ``fused`` takes the single-call entry point instead of the three calls."""
    draft = inp["draft"] if draft is None else draft
    target = inp["target"] if target is None else target
    V = draft.shape[2]
    cpu = lambda ns: SimpleNamespace(**{k: (v.cpu() if v is not None else None) for k, v in vars(ns).items()})
    if fused:
        lat, cps, ver = dsp.dsp_draft_verify_step(
            draft, target, inp["prev_token"], inp["table"], K_max=K, W=W, lam=lam, tau=tau, eos_id=eos_id,
            proxy_kind=proxy_kind, table_log2=inp.get("table_log2", 0), hash_seed=inp.get("hash_seed", 0),
            mode=None if all_greedy else inp["mode"], u=None if all_greedy else inp["u"], all_greedy=all_greedy)
        torch.cuda.synchronize()
        return SimpleNamespace(lat=cpu(lat), cps=cpu(cps), ver=cpu(ver))
    lat = dsp.dsp_lattice_build(draft, K, tau, eos_id)
    cps = dsp.dsp_cps_search(lat, inp["prev_token"], inp["table"], W=W, lam=lam, eos_id=eos_id,
                             proxy_kind=proxy_kind, table_log2=inp.get("table_log2", 0),
                             hash_seed=inp.get("hash_seed", 0), V=V, row_status=lat.row_status)
    if all_greedy:
        ver = dsp.dsp_verify(target, None, cps, None, eos_id=eos_id, all_greedy=True,
                             row_status=lat.row_status)
    else:
        ver = dsp.dsp_verify(target, draft, cps, lat, mode=inp["mode"], u=inp["u"], eos_id=eos_id,
                             row_status=lat.row_status)
    torch.cuda.synchronize()
    return SimpleNamespace(lat=cpu(lat), cps=cpu(cps), ver=cpu(ver))


def _close(a, b, atol, rtol=0.0):
    a, b = a.double(), b.double()
    both_inf = torch.isinf(a) & torch.isinf(b) & (a.sign() == b.sign())
    ok = both_inf | ((a - b).abs() <= atol + rtol * b.abs())
    return ok


def check_step(g: SimpleNamespace, inp: dict, *, K: int, W: int, tau: float = 0.0, lam: float = 0.5,
               eos_id: int = -1, all_greedy: bool = False, proxy_kind: int = 0,
               rows=None) -> dict:
    """Compare GPU outputs ``g`` with the oracle on CPU copies of the same inputs.

    ``rows``: optional list of batch rows to check (the oracle then runs on those only).
    Raises AssertionError on any difference that is not a counted near-tie.
    """
    sel = slice(None) if rows is None else torch.as_tensor(rows, dtype=torch.long)
    pick = lambda t: None if t is None else t.cpu()[sel].contiguous()
    draft, target = pick(inp["draft"]), pick(inp["target"])
    prev, table = pick(inp["prev_token"]), inp["table"].cpu()
    mode = None if all_greedy else pick(inp["mode"])
    u = None if all_greedy else pick(inp["u"])
    G = SimpleNamespace(**{s: SimpleNamespace(**{k: pick(v) for k, v in vars(getattr(g, s)).items()})
                           for s in ("lat", "cps", "ver")})
    B, L, V = draft.shape
    Lt = target.shape[1]
    rep = dict(rows=B, near_tau=0, near_accept=0, near_token=0, max_err={})

    def err(name, a, b):
        m = torch.isfinite(a.double()) & torch.isfinite(b.double())
        e = (a.double() - b.double()).abs()[m].max().item() if m.any() else 0.0
        rep["max_err"][name] = max(rep["max_err"].get(name, 0.0), e)

    # ---- stage 1: lattice ----
    O = oracle.lattice_build(draft, K, tau=tau, eos_id=eos_id)
    Ofull = oracle.lattice_build(draft, K, tau=0.0, eos_id=-1) if (0.0 < tau <= 1.0) else None
    bad_row = (O.row_status & oracle.NONFINITE_INPUT) != 0
    good = ~bad_row
    excused = torch.zeros(B, dtype=torch.bool)
    for b in range(B):
        if bad_row[b]:
            continue
        for l in range(L):
            cg, co = int(G.lat.cand_count[b, l]), int(O.cand_count[b, l])
            if cg != co or not torch.equal(G.lat.cand_id[b, l], O.cand_id[b, l]):
                # only Eq. 7's comparison against tau may differ, and only at a near-tie
                assert Ofull is not None, f"lattice ids differ at ({b},{l})"
                cum = torch.exp(Ofull.cand_logit[b, l].double() - O.lse64[b, l]).cumsum(0)
                assert ((cum - tau).abs() < NEAR).any(), f"candidate count differs away from tau at ({b},{l})"
                excused[b] = True
                rep["near_tau"] += 1
                # the candidates both sides kept must still be the same tokens in the same order
                n = max(0, min(cg, co) - (1 if eos_id >= 0 else 0))
                assert torch.equal(G.lat.cand_id[b, l, :n], O.cand_id[b, l, :n])
    ok = good & ~excused
    assert torch.equal(G.lat.cand_id[ok], O.cand_id[ok])
    assert torch.equal(G.lat.cand_count[ok], O.cand_count[ok])
    assert torch.equal(G.lat.cand_logit[ok], O.cand_logit[ok]), "candidate logits must be exact"
    assert torch.equal(G.lat.gen_len[good], O.gen_len[good])
    for name in ("lse", "cand_logp", "entropy"):
        a, o = getattr(G.lat, name)[ok], getattr(O, name)[ok]
        err(name, a, o)
        assert _close(a, o, TOL_LOGP).all(), f"{name} off by {rep['max_err'][name]}"
    err("lse64", G.lat.lse64[good], O.lse64[good])
    assert _close(G.lat.lse64[good], O.lse64[good], 1e-4).all()

    # ---- stage 2: path search, oracle on the GPU's lattice (stage-isolated) ----
    kw = dict(W=W, lam=lam, eos_id=eos_id, proxy_kind=proxy_kind, table_log2=inp.get("table_log2", 0),
              hash_seed=inp.get("hash_seed", 0), V=V)
    Oc = oracle.cps_search(G.lat.cand_id, G.lat.cand_logit, G.lat.lse64, G.lat.cand_count, prev, table, **kw)
    for name in ("path", "path_slot", "path_len", "beam_ids"):
        assert torch.equal(getattr(G.cps, name)[good], getattr(Oc, name)[good]), f"{name} differs"
    assert torch.equal(G.cps.beam_cum[good], Oc.beam_cum[good]), "ranking quantity must be bit-exact"
    for name in ("path_score", "beam_score"):
        a, o = getattr(G.cps, name)[good], getattr(Oc, name)[good]
        err(name, a, o)
        assert _close(a, o, 1e-3, 1e-5).all(), f"{name} off by {rep['max_err'][name]}"
    stopped_g = (G.lat.row_status & dsp.ROW_EOS_STOPPED) != 0
    assert torch.equal(stopped_g[good], ((Oc.row_status & oracle.EOS_STOPPED) != 0)[good])
    # end to end: the oracle's own lattice gives the same path wherever nothing was excused
    Oe = oracle.cps_search(O.cand_id, O.cand_logit, O.lse64, O.cand_count, prev, table, **kw)
    assert torch.equal(G.cps.path[ok], Oe.path[ok]) and torch.equal(G.cps.path_len[ok], Oe.path_len[ok])

    # ---- stage 3: verification, oracle on the GPU's path ----
    Ov = oracle.verify(target, None if all_greedy else draft, G.cps.path, G.cps.path_len, mode, u, eos_id=eos_id)
    bad_any = bad_row | ((Ov.row_status & oracle.NONFINITE_INPUT) != 0)
    assert torch.equal((G.lat.row_status & dsp.ROW_NONFINITE_INPUT) != 0, bad_any), "nonfinite flags differ"
    good = ~bad_any
    assert torch.equal(G.ver.tgt_argmax[good], Ov.tgt_argmax[good]), "target argmax differs"
    stoch = torch.zeros(B, dtype=torch.bool) if all_greedy else (mode != 0)
    if not all_greedy:
        a, o = G.ver.tgt_lse[stoch & good], Ov.tgt_lse[stoch & good]
        err("tgt_lse", a, o)
        assert _close(a, o, TOL_LOGP).all()
        a, o = G.ver.ratio[good], Ov.ratio[good]
        err("ratio", a, o)
        assert _close(a, o, 1e-5, 1e-4).all(), f"ratio off by {rep['max_err']['ratio']}"
    assert not (G.lat.row_status & dsp.ROW_TIMEOUT).any(), "a bounded wait inside a kernel ran out"
    flags = dsp.ROW_NO_BONUS_ROW | dsp.ROW_EOS_ACCEPTED | dsp.ROW_ZERO_RESIDUAL
    for b in range(B):
        if bad_any[b]:
            continue
        ag, ao = int(G.ver.accepted_len[b]), int(Ov.accepted_len[b])
        tg, to = int(G.ver.next_token[b]), int(Ov.next_token[b])
        m = int(G.cps.path_len[b])
        assert 0 <= ag <= m <= L
        if ag != ao:
            assert stoch[b], f"greedy accepted length differs in row {b}"
            i = min(ag, ao)
            assert abs(float(u[b, i]) - float(Ov.ratio[b, i])) < NEAR, \
                f"row {b}: accept decision differs away from a tie (u={float(u[b, i])}, ratio={float(Ov.ratio[b, i])})"
            rep["near_accept"] += 1
            continue
        if tg != to:
            assert stoch[b], f"greedy next token differs in row {b}: {tg} vs {to}"
            at = ag if ag < m else m
            trow = target[b, at]
            drow = draft[b, at] if ag < m else None
            _, lo, hi, r = oracle.residual_probe(trow, drow, float(u[b, L]), probe=tg)
            uu = float(u[b, L])
            assert r > 0 and lo - NEAR <= uu <= hi + NEAR, \
                f"row {b}: sampled token {tg} outside the oracle's CDF band [{lo},{hi}] for u={uu} (oracle {to})"
            rep["near_token"] += 1
            continue
        sg = int(G.lat.row_status[b]) & flags
        so = int(Ov.row_status[b]) & flags
        assert sg == so, f"row {b}: status flags {sg} vs {so}"
    return rep
