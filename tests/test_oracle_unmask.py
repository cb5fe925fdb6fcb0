"""Pins for the oracle's refinement step of the diffusion drafter (Sec. 3.1, Eq. 5, update set
"top-K by confidence").

Each test checks the oracle against something other than itself: library routines on random
inputs, closed forms, a hand-built block, or invariants of the iteration.
"""
import math

import torch

import oracle


def _case(B, L, V, seed, p_mask=0.7, dtype=torch.float32):
    g = torch.Generator().manual_seed(seed)
    x = (3.0 * torch.randn((B, L, V), generator=g)).to(dtype)
    masked = (torch.rand((B, L), generator=g) < p_mask).to(torch.uint8)
    tokens = torch.randint(0, V, (B, L), generator=g, dtype=torch.int32)
    return x, tokens, masked


def test_matches_softmax_argmax_and_topk_of_the_library():
    B, L, V, n = 4, 9, 200, 3
    x, tokens, masked = _case(B, L, V, 1)
    o = oracle.unmask_step(x, tokens, masked, n)
    p = torch.softmax(x.double(), dim=-1)
    conf, am = p.max(dim=-1)
    m = masked.bool()
    assert torch.equal(o.argmax[m].long(), am[m]) and (o.argmax[~m] == -1).all()
    assert torch.allclose(o.confidence[m].double(), conf[m].log(), atol=1e-6)
    assert torch.isinf(o.confidence[~m]).all() and (o.confidence[~m] < 0).all()
    for b in range(B):
        score = torch.where(m[b], conf[b], torch.full_like(conf[b], -1.0))   # probabilities are > 0
        k = min(n, int(m[b].sum()))
        chosen = set(torch.topk(score, k).indices.tolist())                  # no ties in continuous draws
        for i in range(L):
            if i in chosen:
                assert o.tokens[b, i] == am[b, i] and o.masked[b, i] == 0
            else:
                assert o.tokens[b, i] == tokens[b, i] and o.masked[b, i] == masked[b, i]
        assert o.n_left[b] == int(m[b].sum()) - k
    assert (o.row_status == 0).all()


def test_uniform_rows_closed_form_and_position_order_on_ties():
    B, L, V = 1, 6, 128
    x = torch.zeros((B, L, V))
    tokens = torch.full((B, L), 7, dtype=torch.int32)
    masked = torch.tensor([[1, 0, 1, 1, 0, 1]], dtype=torch.uint8)
    o = oracle.unmask_step(x, tokens, masked, 2)
    m = masked.bool()
    assert (o.argmax[m] == 0).all()                                  # lowest id wins a tie
    assert torch.allclose(o.confidence[m], torch.full((4,), -math.log(V)), atol=1e-6)
    assert o.masked.tolist() == [[0, 0, 0, 1, 0, 1]]                 # equal confidence: lower positions first
    assert o.tokens.tolist() == [[0, 7, 0, 7, 7, 7]] and o.n_left.tolist() == [2]


def test_hand_built_block():
    # four positions with top probabilities 0.5, 0.9, 0.6 and (unmasked) 0.99
    probs = torch.tensor([[0.5, 0.3, 0.2], [0.05, 0.9, 0.05], [0.1, 0.3, 0.6], [0.99, 0.005, 0.005]])
    x = probs.log().unsqueeze(0) + torch.tensor([1.0, -2.0, 0.5, 3.0]).view(1, 4, 1)   # shifts cancel
    tokens = torch.tensor([[10, 11, 12, 13]], dtype=torch.int32)
    masked = torch.tensor([[1, 1, 1, 0]], dtype=torch.uint8)
    o = oracle.unmask_step(x, tokens, masked, 2)
    assert o.argmax.tolist() == [[0, 1, 2, -1]]
    assert torch.allclose(o.confidence[0, :3], torch.tensor([0.5, 0.9, 0.6]).log(), atol=1e-6)
    assert o.tokens.tolist() == [[10, 1, 2, 13]]                     # 0.9 and 0.6 are revealed, 0.5 waits
    assert o.masked.tolist() == [[1, 0, 0, 0]] and o.n_left.tolist() == [1]
    o2 = oracle.unmask_step(x, o.tokens, o.masked, 2)                # the next step takes what is left
    assert o2.tokens.tolist() == [[0, 1, 2, 13]] and o2.masked.sum() == 0 and o2.n_left.tolist() == [0]


def test_iteration_empties_the_mask_in_S_steps_and_never_touches_revealed_tokens():
    B, L, V, S = 3, 10, 50, 4
    x, tokens, _ = _case(B, L, V, 3)
    masked = torch.ones((B, L), dtype=torch.uint8)
    n = -(-L // S)
    revealed_at = torch.full((B, L), -1)
    for s in range(S):
        o = oracle.unmask_step(x, tokens, masked, n)
        newly = (masked == 1) & (o.masked == 0)
        assert (newly.sum(dim=1) == torch.clamp(masked.sum(dim=1).long(), max=n)).all()
        kept = masked == 0
        assert torch.equal(o.tokens[kept], tokens[kept])             # y_i stays once revealed
        revealed_at[newly] = s
        tokens, masked = o.tokens, o.masked
    assert masked.sum() == 0 and (revealed_at >= 0).all()
    conf = torch.log_softmax(x.double(), -1).max(-1).values
    for b in range(B):                                               # with fixed logits: earlier = more confident
        order = torch.argsort(conf[b], descending=True)
        assert (revealed_at[b, order][1:] >= revealed_at[b, order][:-1]).all()


def test_bf16_logits_are_read_exactly_and_large_n_reveals_all():
    B, L, V = 2, 5, 300
    x, tokens, masked = _case(B, L, V, 4, dtype=torch.bfloat16)
    o = oracle.unmask_step(x, tokens, masked, 100)
    ref = oracle.unmask_step(x.float(), tokens, masked, 100)         # bf16 -> fp32 is exact
    for k in ("tokens", "masked", "argmax", "confidence", "n_left"):
        assert torch.equal(getattr(o, k), getattr(ref, k))
    assert o.masked.sum() == 0 and (o.n_left == 0).all()


def test_nonfinite_rows_are_flagged_only_when_masked():
    B, L, V = 2, 3, 40
    x, tokens, _ = _case(B, L, V, 5)
    x[0, 1, 3] = float("nan")
    x[1, 2, :] = float("-inf")
    masked = torch.tensor([[1, 0, 1], [1, 1, 1]], dtype=torch.uint8)
    o = oracle.unmask_step(x, tokens, masked, 1)
    assert o.row_status.tolist() == [0, oracle.NONFINITE_INPUT]      # row 0's NaN sits at a revealed position
    masked[0, 1] = 1
    o = oracle.unmask_step(x, tokens, masked, 1)
    assert o.row_status.tolist() == [oracle.NONFINITE_INPUT, oracle.NONFINITE_INPUT]
