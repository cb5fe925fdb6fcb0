"""Pins for the oracle's verification stage (Eq. 1, residual resampling, Eq. 2, greedy rule, bonus).

Closed forms on hand-built two- and three-token distributions, the
unbiasedness property of speculative sampling, and invariants.
"""
import math

import numpy as np
import pytest
import torch

import oracle


def _logits(p):
    return torch.tensor(p, dtype=torch.float64).log().float()


def _one(p, q, y, u_acc, u_res, Lt_extra=False, mode=1, eos=-1):
    """One row, one position: target p, draft q, drafted token y."""
    tgt = _logits(p).view(1, 1, -1)
    if Lt_extra:
        tgt = torch.cat([tgt, _logits(Lt_extra).view(1, 1, -1)], dim=1)
    out = oracle.verify(tgt, _logits(q).view(1, 1, -1), torch.tensor([[y]], dtype=torch.int32),
                        torch.tensor([1], dtype=torch.int32), torch.tensor([mode], dtype=torch.uint8),
                        torch.tensor([[u_acc, u_res]]), eos_id=eos)
    return out


def test_two_token_acceptance_closed_form():
    a, b = 0.3, 0.6                                        # p = (a, 1-a), q = (b, 1-b), token 0 drafted
    for u in (0.0, 0.25, 0.49, 0.499999):
        o = _one([a, 1 - a], [b, 1 - b], 0, u, 0.5)
        assert o.accepted_len.item() == 1 and o.next_token.item() == -1
        assert o.row_status.item() == oracle.NO_BONUS_ROW
        assert abs(o.ratio.item() - a / b) < 1e-6
    for u in (0.5000001, 0.75, 0.999):
        o = _one([a, 1 - a], [b, 1 - b], 0, u, 0.5)
        assert o.accepted_len.item() == 0
        assert o.next_token.item() == 1                    # residual [p-q]_+ is all on token 1
    # ratio >= 1: always accepted
    o = _one([b, 1 - b], [a, 1 - a], 0, 0.999999, 0.5)
    assert o.accepted_len.item() == 1 and abs(o.ratio.item() - b / a) < 1e-6


def test_three_token_residual_by_hand():
    p, q = [0.5, 0.3, 0.2], [0.2, 0.7, 0.1]               # token 1 drafted, ratio 3/7
    # [p-q]_+ = (0.3, 0, 0.1): token 0 w.p. 0.75, token 2 w.p. 0.25
    assert _one(p, q, 1, 0.9, 0.00, False).next_token.item() == 0
    assert _one(p, q, 1, 0.9, 0.74, False).next_token.item() == 0
    assert _one(p, q, 1, 0.9, 0.76, False).next_token.item() == 2
    assert _one(p, q, 1, 0.9, 0.999999, False).next_token.item() == 2
    assert _one(p, q, 1, 0.42, 0.1, False).accepted_len.item() == 1          # 0.42 < 3/7
    assert _one(p, q, 1, 0.43, 0.1, False).accepted_len.item() == 0          # 0.43 > 3/7


def test_residual_cdf_edges_skip_zero_mass_tokens():
    p, q = [0.1, 0.4, 0.1, 0.4], [0.4, 0.1, 0.4, 0.1]     # residual only on tokens 1 and 3
    t = _logits(p)
    d = _logits(q)
    assert oracle.residual_probe(t, d, 0.0)[0] == 1        # u = 0: first token with positive mass
    assert oracle.residual_probe(t, d, 0.4999)[0] == 1
    assert oracle.residual_probe(t, d, 0.5001)[0] == 3
    assert oracle.residual_probe(t, d, 0.9999999)[0] == 3  # u -> 1: last token with positive mass
    tok, lo, hi, r = oracle.residual_probe(t, d, 0.2, probe=3)
    assert tok == 1 and abs(lo - 0.5) < 1e-9 and abs(hi - 1.0) < 1e-9 and abs(r - 0.3) < 1e-7
    # draw from p itself (bonus token): exact rational masses
    assert oracle.residual_probe(_logits([0.25, 0.25, 0.5]), None, 0.49)[0] == 1
    assert oracle.residual_probe(_logits([0.25, 0.25, 0.5]), None, 0.51)[0] == 2


def test_identical_distributions_always_accept_and_zero_residual_flag():
    g = torch.Generator().manual_seed(0)
    x = torch.randn((4, 5, 30), generator=g)
    path = x.argmax(-1).int()
    u = torch.rand((4, 6), generator=g)
    u[:, :5] = 0.999999
    o = oracle.verify(x, x, path, torch.full((4,), 5, dtype=torch.int32),
                      torch.ones(4, dtype=torch.uint8), u)
    assert (o.accepted_len == 5).all() and torch.allclose(o.ratio, torch.ones(4, 5))
    assert (o.next_token == -1).all() and (o.row_status == oracle.NO_BONUS_ROW).all()


@pytest.mark.parametrize("p,q", [([0.6, 0.3, 0.1], [0.2, 0.5, 0.3]), ([0.05, 0.9, 0.05], [0.4, 0.2, 0.4])])
def test_unbiasedness_emitted_token_follows_target(p, q):
    """Drafting y ~ q then accepting / resampling emits a token distributed as p (Sec. 2)."""
    N = 40000
    g = torch.Generator().manual_seed(123)
    y = torch.multinomial(torch.tensor(q), N, replacement=True, generator=g).int().view(N, 1)
    u = torch.rand((N, 2), generator=g)
    tgt = _logits(p).view(1, 1, -1).expand(N, 1, 3).contiguous()
    drf = _logits(q).view(1, 1, -1).expand(N, 1, 3).contiguous()
    o = oracle.verify(tgt, drf, y, torch.ones(N, dtype=torch.int32), torch.ones(N, dtype=torch.uint8), u)
    emitted = torch.where(o.accepted_len == 1, y.view(-1), o.next_token)
    freq = torch.bincount(emitted.long(), minlength=3).double() / N
    for v in range(3):
        sd = math.sqrt(p[v] * (1 - p[v]) / N)
        assert abs(freq[v].item() - p[v]) < 4 * sd
    # acceptance frequency = sum_v min(p_v, q_v)
    acc = sum(min(a, b) for a, b in zip(p, q))
    assert abs((o.accepted_len == 1).double().mean().item() - acc) < 4 * math.sqrt(acc * (1 - acc) / N)


def test_greedy_rule_is_longest_prefix_of_argmax_matches():
    g = torch.Generator().manual_seed(5)
    B, L, V = 64, 12, 9
    tgt = torch.randn((B, L + 1, V), generator=g)
    am = tgt.argmax(-1)
    path = am[:, :L].clone().int()
    flip = torch.rand((B, L), generator=g) < 0.2           # break some matches
    path[flip] = (path[flip] + 1) % V
    plen = torch.randint(1, L + 1, (B,), generator=g, dtype=torch.int32)
    o = oracle.verify(tgt, None, path, plen, torch.zeros(B, dtype=torch.uint8), None)
    for b in range(B):
        m = int(plen[b])
        match = (path[b, :m].long() == am[b, :m]).tolist()
        want = match.index(False) if False in match else m           # independent one-liner
        assert o.accepted_len[b].item() == want <= m <= L
        assert o.next_token[b].item() == int(am[b, want])            # correction, or bonus from row m
        assert o.row_status[b].item() == 0
    assert torch.equal(o.tgt_argmax.long(), am)
    assert torch.allclose(o.tgt_lse.double(), torch.logsumexp(tgt.double(), -1), atol=1e-6)
    assert (o.ratio == -1).all()


def test_greedy_ties_take_lowest_id_and_target_equal_draft_accepts_all():
    tgt = torch.tensor([[[1.0, 3.0, 3.0], [2.0, 2.0, 0.0]]])
    o = oracle.verify(tgt, None, torch.tensor([[1, 0]], dtype=torch.int32), torch.tensor([2], dtype=torch.int32))
    assert o.accepted_len.item() == 2 and o.tgt_argmax[0].tolist() == [1, 0]
    o = oracle.verify(tgt, None, torch.tensor([[2, 0]], dtype=torch.int32), torch.tensor([2], dtype=torch.int32))
    assert o.accepted_len.item() == 0 and o.next_token.item() == 1


def test_bonus_token_and_eos_flag():
    p, q, nxt = [0.5, 0.5], [0.5, 0.5], [0.2, 0.8]
    o = _one(p, q, 1, 0.3, 0.1, Lt_extra=nxt)              # accepted; bonus drawn from row m = 1
    assert o.accepted_len.item() == 1 and o.next_token.item() == 0 and o.row_status.item() == 0
    o = _one(p, q, 1, 0.3, 0.25, Lt_extra=nxt)
    assert o.next_token.item() == 1
    o = _one(p, q, 1, 0.3, 0.25, Lt_extra=nxt, mode=0)     # greedy: 1 != argmax 0 (tie -> id 0)
    assert o.accepted_len.item() == 0 and o.next_token.item() == 0
    o = _one(p, q, 1, 0.3, 0.25, Lt_extra=nxt, eos=1)      # an accepted EOS counts and is flagged
    assert o.accepted_len.item() == 1 and o.row_status.item() & oracle.EOS_ACCEPTED


def test_zero_draft_probability_and_zero_target_probability():
    ninf = -float("inf")
    tgt = torch.tensor([[[0.0, 0.0, ninf]]])
    drf = torch.tensor([[[0.0, ninf, 0.0]]])
    one = torch.tensor([1], dtype=torch.int32)
    st = torch.ones(1, dtype=torch.uint8)
    u = torch.tensor([[0.999, 0.3]])
    # q(y) = 0 < p(y): accepted for every u
    assert oracle.verify(tgt, drf, torch.tensor([[1]], dtype=torch.int32), one, st, u).accepted_len.item() == 1
    # p(y) = 0: rejected for every u; residual = (0, 0.5, 0) -> token 1
    o = oracle.verify(tgt, drf, torch.tensor([[2]], dtype=torch.int32), one, st, torch.tensor([[0.0, 0.3]]))
    assert o.accepted_len.item() == 0 and o.next_token.item() == 1


def test_rejection_discards_the_rest():
    g = torch.Generator().manual_seed(9)
    B, L, V = 32, 8, 6
    drf = torch.randn((B, L, V), generator=g)
    tgt = drf + torch.randn((B, L, V), generator=g)
    path = torch.randint(0, V, (B, L), generator=g, dtype=torch.int32)
    u = torch.rand((B, L + 1), generator=g)
    o = oracle.verify(tgt, drf, path, torch.full((B,), L, dtype=torch.int32), torch.ones(B, dtype=torch.uint8), u)
    lp = torch.log_softmax(tgt.double(), -1).gather(-1, path.long()[..., None])[..., 0]
    lq = torch.log_softmax(drf.double(), -1).gather(-1, path.long()[..., None])[..., 0]
    ratio = (lp - lq).exp()
    assert torch.allclose(o.ratio.double(), ratio, rtol=1e-5)
    ok = u[:, :L].double() < ratio
    for b in range(B):
        row = ok[b].tolist()
        want = row.index(False) if False in row else L    # Eq. 2
        assert o.accepted_len[b].item() == want
        if want < L:                                       # the replacement has positive residual mass
            t = o.next_token[b].item()
            pr = torch.softmax(tgt[b, want].double(), 0) - torch.softmax(drf[b, want].double(), 0)
            assert pr[t] > 0


def _flag_case(poison_target=None, poison_draft=None, mode=1, path_tok=(0, 1), u=None):
    """Two batch rows, two positions, V = 4; batch row 1 stays clean as the control."""
    tgt = torch.tensor([[[2.0, 1.0, 0.0, -1.0], [0.0, 3.0, 1.0, 0.5]]]).repeat(2, 1, 1)
    drf = torch.tensor([[[1.5, 1.0, 0.5, -1.0], [0.5, 2.0, 1.0, 0.0]]]).repeat(2, 1, 1)
    if poison_target is not None:
        i, v, val = poison_target
        tgt[0, i, v] = val
    if poison_draft is not None:
        i, v, val = poison_draft
        drf[0, i, v] = val
    path = torch.tensor([list(path_tok)] * 2, dtype=torch.int32)
    if u is None:
        u = torch.tensor([[0.0, 0.0, 0.5]] * 2)
    return oracle.verify(tgt, drf, path, torch.tensor([2, 2], dtype=torch.int32),
                         torch.full((2,), mode, dtype=torch.uint8), u)


@pytest.mark.parametrize("val", [float("nan"), float("inf")])
def test_nonfinite_target_logit_flags_only_its_batch_row(val):
    # written by hand: NaN or +inf anywhere in a target row flags the batch row, in either mode,
    # also in a row the scan never reaches (position 1 after a rejection at position 0)
    for mode in (0, 1):
        for pos in (0, 1):
            o = _flag_case(poison_target=(pos, 3, val), mode=mode)
            assert o.row_status[0].item() & oracle.NONFINITE_INPUT
            assert o.row_status[1].item() & oracle.NONFINITE_INPUT == 0
    o = _flag_case(poison_target=(1, 3, val), mode=0, path_tok=(3, 1))   # greedy: rejected at 0, row 1 unread
    assert o.accepted_len.tolist() == [0, 0] and o.row_status[0].item() & oracle.NONFINITE_INPUT
    assert o.next_token.tolist() == [0, 0] and o.row_status[1].item() == 0


@pytest.mark.parametrize("val", [float("nan"), float("inf")])
def test_nonfinite_draft_logit_flags_a_stochastic_row_and_is_not_read_by_a_greedy_one(val):
    o = _flag_case(poison_draft=(0, 2, val), mode=1)
    assert o.row_status[0].item() & oracle.NONFINITE_INPUT and o.row_status[1].item() & oracle.NONFINITE_INPUT == 0
    o = _flag_case(poison_draft=(0, 2, val), mode=0)                      # greedy never looks at the draft logits
    assert o.row_status[0].item() & oracle.NONFINITE_INPUT == 0
    assert o.accepted_len.tolist() == [2, 2]                              # path (0, 1) is the target argmax twice


def test_minus_inf_is_masking_not_an_error():
    o = _flag_case(poison_target=(0, 3, -float("inf")), poison_draft=(1, 3, -float("inf")), mode=1)
    assert o.row_status[0].item() & oracle.NONFINITE_INPUT == 0


def test_zero_residual_needs_a_poisoned_row():
    """In double [p - q]_+ has positive mass whenever a token was rejected (p(y) < q(y) and both sum
    to one), and a bonus draw is from p itself: the flag is reachable only when the sums are not
    numbers.  Then the token is the target argmax of that row (written by hand) and both flags are up."""
    u = torch.tensor([[0.999999, 0.0, 0.5]] * 2)                          # reject position 0 on both rows
    o = _flag_case(poison_target=(0, 3, float("nan")), mode=1, path_tok=(1, 1), u=u)
    assert o.accepted_len.tolist() == [0, 0]
    assert o.row_status[0].item() & oracle.ZERO_RESIDUAL and o.row_status[0].item() & oracle.NONFINITE_INPUT
    assert o.next_token[0].item() == 0                                    # argmax of (2, 1, 0, NaN): NaN never wins
    assert o.row_status[1].item() == 0 and o.next_token[1].item() == 0   # clean row: residual is all on token 0
    # clean rows over many seeds never raise it
    g = torch.Generator().manual_seed(3)
    B, L, V = 64, 4, 5
    drf = torch.randn((B, L, V), generator=g) * 3
    tgt = drf + torch.randn((B, L, V), generator=g)
    path = torch.randint(0, V, (B, L), generator=g, dtype=torch.int32)
    o = oracle.verify(tgt, drf, path, torch.full((B,), L, dtype=torch.int32), torch.ones(B, dtype=torch.uint8),
                      torch.rand((B, L + 1), generator=g))
    assert (o.row_status & oracle.ZERO_RESIDUAL == 0).all()
