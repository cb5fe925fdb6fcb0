"""Pins for the oracle's lattice stage (row statistics, top-K, Eq. 7 pruning, EOS, Eq. 9).

Each test checks the oracle against something other than itself: a library
routine on a special case, a closed form, an invariant or a hand-built row.
"""
import math

import numpy as np
import pytest
import torch

import oracle


def _rand(B, L, V, seed, scale=3.0):
    g = torch.Generator().manual_seed(seed)
    return scale * torch.randn((B, L, V), generator=g)


def test_logsoftmax_topk_match_library_routines():
    x = _rand(2, 3, 1000, 1)
    K = 8
    o = oracle.lattice_build(x, K)
    ref = torch.log_softmax(x.double(), dim=-1)
    tv, ti = torch.topk(x.double(), K, dim=-1)          # no ties in continuous draws
    assert torch.equal(o.cand_id.long(), ti)
    assert torch.equal(o.cand_logit, tv.float())
    assert torch.allclose(o.cand_logp.double(), torch.gather(ref, -1, ti), atol=1e-6)
    lse = torch.logsumexp(x.double(), dim=-1)
    assert torch.allclose(o.lse64, lse, atol=1e-12)
    assert torch.allclose(o.lse.double(), lse, atol=1e-6)
    H = -(ref.exp() * ref).sum(-1)
    assert torch.allclose(o.entropy.double(), H, atol=1e-6)
    assert (o.cand_count == K).all() and (o.gen_len == 3).all() and (o.row_status == 0).all()


def test_probabilities_sum_to_one():
    V = 64
    x = _rand(1, 2, V, 2)
    o = oracle.lattice_build(x, V)                        # K = V: every token is a candidate
    tot = torch.exp(o.cand_logit.double() - o.lse64[..., None]).sum(-1)
    assert torch.allclose(tot, torch.ones_like(tot), atol=1e-12)


def test_uniform_onehot_and_two_point_closed_forms():
    V = 257
    x = torch.full((1, 1, V), 1.25)
    o = oracle.lattice_build(x, 4)
    assert abs(o.lse64.item() - (1.25 + math.log(V))) < 1e-12
    assert abs(o.entropy.item() - math.log(V)) < 1e-6
    assert o.cand_id[0, 0].tolist() == [0, 1, 2, 3]       # all tied: lowest ids first

    x = torch.full((1, 1, V), -float("inf"))
    x[0, 0, 100] = 3.5
    o = oracle.lattice_build(x, 4)
    assert abs(o.lse64.item() - 3.5) < 1e-12 and abs(o.entropy.item()) < 1e-12
    assert o.cand_count.item() == 1 and o.cand_id[0, 0].tolist() == [100, -1, -1, -1]
    assert o.row_status.item() == 0

    a, b = 2.0, -1.0                                      # two-point distribution
    x = torch.tensor([[[a, b]]])
    o = oracle.lattice_build(x, 2)
    d = a - b
    H = math.log1p(math.exp(-d)) + d * math.exp(-d) / (1 + math.exp(-d))
    assert abs(o.entropy.item() - H) < 1e-6
    assert abs(o.lse64.item() - (a + math.log1p(math.exp(-d)))) < 1e-12


def test_shift_invariance():
    x = _rand(1, 2, 500, 3)
    o1 = oracle.lattice_build(x, 5)
    o2 = oracle.lattice_build(x + 16.0, 5)                # fp32 rounding of x+16 moves lse by < 1e-5
    assert torch.equal(o1.cand_id, o2.cand_id)
    assert torch.allclose(o2.lse64 - o1.lse64, torch.full_like(o1.lse64, 16.0), atol=1e-5)
    assert torch.allclose(o1.entropy, o2.entropy, atol=1e-5)


def test_tie_break_hand_built_rows():
    # values: 1 5 5 2 5 0 2 2  -> order (value desc, id asc): 1,2,4 then 3,6,7 then 0 then 5
    x = torch.tensor([[[1.0, 5.0, 5.0, 2.0, 5.0, 0.0, 2.0, 2.0]]])
    o = oracle.lattice_build(x, 7)
    assert o.cand_id[0, 0].tolist() == [1, 2, 4, 3, 6, 7, 0]
    o = oracle.lattice_build(x, 2)
    assert o.cand_id[0, 0].tolist() == [1, 2]
    o = oracle.lattice_build(x, 12)                       # K > V: K_eff = V, rest padded
    assert o.cand_id[0, 0].tolist() == [1, 2, 4, 3, 6, 7, 0, 5, -1, -1, -1, -1]
    assert o.cand_count.item() == 8
    assert torch.isinf(o.cand_logit[0, 0, 8:]).all()


def test_bf16_rows_equal_their_fp32_upcast():
    x = _rand(2, 2, 777, 4).to(torch.bfloat16)
    o16 = oracle.lattice_build(x, 6)
    o32 = oracle.lattice_build(x.float(), 6)
    for k in ("cand_id", "cand_logit", "cand_logp", "cand_count", "lse64", "entropy"):
        assert torch.equal(getattr(o16, k), getattr(o32, k)), k


@pytest.mark.parametrize("r,tau", [(0.5, 0.8), (0.7, 0.8), (0.9, 0.5), (0.6, 0.999)])
def test_eq7_geometric_closed_form(r, tau):
    # p_k = (1-r) r^(k-1), k = 1..V (V large: truncated mass < 1e-30)
    V, K = 400, 30
    logits = torch.arange(V, dtype=torch.float64) * math.log(r)
    o = oracle.lattice_build(logits.float().view(1, 1, V), K, tau=tau)
    M = math.ceil(math.log(1 - tau) / math.log(r) - 1e-9)
    assert o.cand_count.item() == min(M, K)


def test_eq7_limits():
    x = _rand(1, 4, 300, 5)
    assert (oracle.lattice_build(x, 9, tau=1e-9).cand_count == 1).all()       # tau -> 0: one candidate
    flat = torch.zeros((1, 1, 1000))
    assert oracle.lattice_build(flat, 9, tau=0.5).cand_count.item() == 9       # unreachable: K
    assert oracle.lattice_build(x, 9, tau=0.0).cand_count.eq(9).all()          # disabled
    assert oracle.lattice_build(x, 9, tau=1.5).cand_count.eq(9).all()          # disabled
    # counts never decrease as tau grows
    c = [oracle.lattice_build(x, 9, tau=t).cand_count for t in (0.1, 0.3, 0.6, 0.9)]
    assert all((c[i] <= c[i + 1]).all() for i in range(3))


def test_eq7_mass_is_full_vocabulary_not_renormalised():
    # top-2 hold 0.4 + 0.3 of the mass; renormalised over top-3 they would hold more
    p = torch.tensor([0.4, 0.3, 0.1] + [0.2 / 50] * 50, dtype=torch.float64)
    o = oracle.lattice_build(p.log().float().view(1, 1, -1), 3, tau=0.75)
    assert o.cand_count.item() == 3
    o = oracle.lattice_build(p.log().float().view(1, 1, -1), 3, tau=0.65)
    assert o.cand_count.item() == 2


def test_eos_retention_and_gen_len():
    V, L, K, eos = 50, 6, 3, 49
    x = _rand(1, L, V, 6)
    x[0, :, eos] = -20.0                                   # EOS far from the top everywhere
    x[0, 3, eos] = 30.0                                    # ... except top-1 at position 3
    x[0, 5, eos] = 30.0
    o = oracle.lattice_build(x, K, eos_id=eos)
    assert o.cand_id.shape == (1, L, K + 1)
    assert o.gen_len.item() == 3                           # Eq. 9: positions before the first EOS
    for l in range(L):
        ids = o.cand_id[0, l].tolist()
        cnt = o.cand_count[0, l].item()
        if l in (3, 5):
            assert ids[0] == eos and cnt == K and ids[K] == -1
        else:
            assert ids[K] == eos and cnt == K + 1          # extra slot after the kept ones
            assert abs(o.cand_logit[0, l, K].item() + 20.0) < 1e-6
            assert abs(o.cand_logp[0, l, K].item() - (-20.0 - o.lse64[0, l].item())) < 1e-5
    # the EOS slot is not counted in Eq. 7
    o2 = oracle.lattice_build(x, K, tau=1e-9, eos_id=eos)
    assert o2.cand_count[0, 0].item() == 2 and o2.cand_id[0, 0, 1].item() == eos
    # a masked EOS is not appended
    x[0, 0, eos] = -float("inf")
    assert oracle.lattice_build(x, K, eos_id=eos).cand_count[0, 0].item() == K
    # no EOS anywhere on top: gen_len = L
    assert oracle.lattice_build(_rand(2, 4, 30, 7), 2, eos_id=0).gen_len.tolist() in ([4, 4],)


def test_masked_and_nonfinite_rows():
    x = _rand(2, 1, 40, 8)
    x[0, 0, 5:] = -float("inf")                            # five finite logits, K = 8
    x[1, 0, 3] = float("nan")
    o = oracle.lattice_build(x, 8)
    assert o.cand_count[0, 0].item() == 5 and (o.cand_id[0, 0, 5:] == -1).all()
    assert o.row_status.tolist() == [0, oracle.NONFINITE_INPUT]
    ref = torch.logsumexp(x[0, 0, :5].double(), 0)
    assert abs(o.lse64[0, 0].item() - ref.item()) < 1e-12


def test_row_stats_argmax_lowest_id():
    row = torch.tensor([0.0, 3.0, 3.0, -1.0, 3.0])
    lse, H, am, bad = oracle.row_stats(row)
    assert am == 1 and bad == 0
    assert abs(lse - torch.logsumexp(row.double(), 0).item()) < 1e-12
