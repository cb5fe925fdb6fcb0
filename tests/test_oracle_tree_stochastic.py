"""Pins for the oracle's stochastic verification of a token tree (multi-branch form of Eq. 1 with residual
resampling): hand-computed three-token cases, the unbiasedness of the emitted token when the siblings are
drawn from the drafter's distribution, and the one-path tree against the single-path verification."""
import math
from types import SimpleNamespace

import pytest
import torch

import oracle


def _logits(p):
    return torch.tensor(p, dtype=torch.float64).log().float()


def _tree(tokens, parents, N):
    B = len(tokens)
    tok = torch.full((B, N), -1, dtype=torch.int32)
    par = torch.full((B, N), -1, dtype=torch.int32)
    for b in range(B):
        tok[b, :len(tokens[b])] = torch.tensor(tokens[b], dtype=torch.int32)
        par[b, :len(parents[b])] = torch.tensor(parents[b], dtype=torch.int32)
    return SimpleNamespace(node_token=tok, node_parent=par, n_nodes=torch.tensor([len(t) for t in tokens], dtype=torch.int32))


def _two_siblings(p, q, toks, u0, u1, ures, after=(0.25, 0.25, 0.5)):
    """One batch row, depth 1, two children of the root with tokens `toks`."""
    tgt = torch.stack([_logits(p), _logits(after), _logits(after)]).view(1, 3, -1)
    return oracle.verify_tree_stochastic(tgt, _logits(q).view(1, 1, -1), _tree([toks], [[-1, -1]], 2),
                                         torch.tensor([[u0, u1, ures]]))


def test_three_token_cases_by_hand():
    p, q = [0.5, 0.3, 0.2], [0.2, 0.7, 0.1]
    # first child token 1: ratio 3/7.  Accepted below it: the walk stands on node 0; the emitted token is then
    # the bonus draw from node 0's row (0.25, 0.25, 0.5)
    o = _two_siblings(p, q, [1, 0], 0.42, 0.0, 0.6)
    assert o.accepted_len.item() == 1 and o.accepted_node.tolist() == [[0]] and o.next_token.item() == 2
    # rejected (0.43 > 3/7): residual (0.3, 0, 0.1) / 0.4 = (0.75, 0, 0.25); second child token 0: 0.75 / 0.2 > 1
    o = _two_siblings(p, q, [1, 0], 0.43, 0.999, 0.1)
    assert o.accepted_len.item() == 1 and o.accepted_node.tolist() == [[1]]
    # second child token 2: 0.25 / 0.1 > 1: accepted as well
    assert _two_siblings(p, q, [1, 2], 0.9, 0.999, 0.1).accepted_node.tolist() == [[1]]
    # the same token twice: its residual mass is 0, rejected again; residual of the residual:
    # [(0.75, 0, 0.25) - (0.2, 0.7, 0.1)]_+ = (0.55, 0, 0.15) / 0.7: token 0 up to u = 0.7857, then token 2
    o = _two_siblings(p, q, [1, 1], 0.9, 0.0, 0.78)
    assert o.accepted_len.item() == 0 and o.next_token.item() == 0
    assert _two_siblings(p, q, [1, 1], 0.9, 0.0, 0.79).next_token.item() == 2
    # no child at all: the emitted token is a draw from p itself (0.5 | 0.8 | 1)
    tgt = _logits(p).view(1, 1, -1).repeat(1, 3, 1)
    for ures, want in ((0.49, 0), (0.51, 1), (0.81, 2)):
        o = oracle.verify_tree_stochastic(tgt, _logits(q).view(1, 1, -1), _tree([[]], [[]], 2), torch.tensor([[0.0, 0.0, ures]]))
        assert o.accepted_len.item() == 0 and o.next_token.item() == want and o.row_status.item() == 0


@pytest.mark.parametrize("p,q", [([0.6, 0.3, 0.1], [0.2, 0.5, 0.3]), ([0.05, 0.9, 0.05], [0.4, 0.2, 0.4])])
def test_emitted_token_follows_the_target_with_two_sampled_siblings(p, q):
    """Siblings drawn independently from q (the same token may come twice), tried in turn with residual
    updates: the first emitted token is distributed as p (the multi-branch form keeps Sec. 2's unbiasedness),
    and two branches accept more often than one."""
    N = 40000
    g = torch.Generator().manual_seed(7)
    toks = torch.multinomial(torch.tensor(q), 2 * N, replacement=True, generator=g).int().view(N, 2)
    u = torch.rand((N, 3), generator=g)
    tgt = _logits(p).view(1, 1, 3).expand(N, 3, 3).contiguous()
    drf = _logits(q).view(1, 1, 3).expand(N, 1, 3).contiguous()
    tree = SimpleNamespace(node_token=toks, node_parent=torch.full((N, 2), -1, dtype=torch.int32),
                           n_nodes=torch.full((N,), 2, dtype=torch.int32))
    o = oracle.verify_tree_stochastic(tgt, drf, tree, u)
    first = o.accepted_node[:, 0].long()
    emitted = torch.where(o.accepted_len == 1, toks.gather(1, first.clamp(min=0).view(-1, 1)).view(-1), o.next_token)
    freq = torch.bincount(emitted.long(), minlength=3).double() / N
    for v in range(3):
        assert abs(freq[v].item() - p[v]) < 4 * math.sqrt(p[v] * (1 - p[v]) / N)
    one_branch = sum(min(a, b) for a, b in zip(p, q))
    assert (o.accepted_len == 1).double().mean().item() > one_branch + 0.02


def test_one_path_tree_equals_the_single_path_verification():
    g = torch.Generator().manual_seed(11)
    B, L, V = 48, 6, 7
    drf = torch.randn((B, L, V), generator=g) * 1.5
    tgt = torch.cat([drf + torch.randn((B, L, V), generator=g), torch.randn((B, 1, V), generator=g)], dim=1)   # [B, L+1, V]
    path = torch.randint(0, V, (B, L), generator=g, dtype=torch.int32)
    m = torch.randint(1, L + 1, (B,), generator=g, dtype=torch.int32)
    u = torch.rand((B, L + 1), generator=g)
    tree = _tree([path[b, :int(m[b])].tolist() for b in range(B)], [list(range(-1, int(m[b]) - 1)) for b in range(B)], L)
    o = oracle.verify_tree_stochastic(tgt, drf, tree, u)          # node i sits at depth i: u[b,i], then u[b,L]
    for b in range(B):
        mm = int(m[b])
        rows = tgt[b:b + 1, :mm + 1]                               # a bonus row exists after the last node
        ref = oracle.verify(rows.contiguous(), drf[b:b + 1, :mm].contiguous(), path[b:b + 1, :mm], torch.tensor([mm], dtype=torch.int32),
                            torch.ones(1, dtype=torch.uint8), torch.cat([u[b:b + 1, :mm], u[b:b + 1, L:]], dim=1))
        assert o.accepted_len[b].item() == ref.accepted_len.item()
        assert o.next_token[b].item() == ref.next_token.item()
        acc = int(o.accepted_len[b])
        assert o.accepted_node[b, :acc].tolist() == list(range(acc)) and (o.accepted_node[b, acc:] == -1).all()


def test_flags_and_depth_limit():
    p, q = [0.5, 0.3, 0.2], [0.2, 0.7, 0.1]
    tgt = torch.stack([_logits(p)] * 4).view(1, 4, 3).clone()
    tree = _tree([[0, 1]], [[-1, 0]], 3)                          # a path of two nodes; slot 2 unused
    drf = _logits(q).view(1, 1, 3).repeat(1, 2, 1)
    u = torch.tensor([[0.0, 0.0, 0.0, 0.3]])
    o = oracle.verify_tree_stochastic(tgt, drf, tree, u)
    assert o.accepted_len.item() == 2 and o.row_status.item() == 0
    bad = tgt.clone(); bad[0, 3, 1] = float("nan")               # row of the unused slot: never read
    assert oracle.verify_tree_stochastic(bad, drf, tree, u).row_status.item() == 0
    bad = tgt.clone(); bad[0, 2, 1] = float("inf")               # row after node 1 exists
    assert oracle.verify_tree_stochastic(bad, drf, tree, u).row_status.item() & oracle.NONFINITE_INPUT
    o = oracle.verify_tree_stochastic(tgt, drf[:, :1], tree, u)   # L = 1: the walk stops after one node
    assert o.accepted_len.item() == 1 and o.accepted_node.tolist() == [[0]]


def test_margin_of_the_closest_decision_by_hand():
    p, q = [0.5, 0.3, 0.2], [0.2, 0.7, 0.1]
    # one acceptance test at ratio 3/7 with u = 0.42, then the bonus draw from (0.25, 0.25, 0.5) at u = 0.6:
    # token 2's step of the cumulative sum is (0.5, 1.0], so the draw is 0.1 from its lower end
    o = _two_siblings(p, q, [1, 0], 0.42, 0.0, 0.6)
    r = 3.0 / 7.0
    assert o.margin.item() == pytest.approx(min((r - 0.42) / r, 0.1), rel=1e-5)
    # rejected at 0.43 (margin (0.43 - 3/7) / 0.43), second child accepted far from its ratio (3.75 against
    # 0.999), bonus draw at 0.1 from (0.25, 0.25, 0.5): 0.1 from the lower end of token 0's step
    o = _two_siblings(p, q, [1, 0], 0.43, 0.999, 0.1)
    assert o.margin.item() == pytest.approx((0.43 - r) / 0.43, rel=1e-4)
