"""Pins for the oracle's breadth controller (the reading of the paper's future work iii: the form of
Eq. 10 on the drafter's mean entropy and on the acceptance shortfall; K from the perplexity, W
from the shortfall).  Hand-computed steps, closed forms and guard rails."""
import math

import torch

import oracle


def test_hand_computed_steps():
    # rho = 0.5, K in [2, 16], W in [1, 9]; every value below worked out by hand from the rule
    c = oracle.Breadth(2, 16, 1, 9, 0.5)
    assert (c.K, c.W) == (16, 9) and c.ema_entropy == 0.0 and c.ema_shortfall == 0.0
    # step 1: one batch row, L = 4, gen_len 4, accepted 1: H = mean(2,2,2,2) = 2, s = 3/4
    #   ema_H = 1, ema_s = 0.375; K = ceil(e^1 = 2.718) = 3; W = ceil(1 + 8 * 0.375 = 4) = 4
    assert c.update(torch.full((1, 4), 2.0), [1], [4]) == (3, 4)
    assert c.ema_entropy == 1.0 and c.ema_shortfall == 0.375
    # step 2: gen_len 2: only positions 0, 1 count: H = (4 + 2) / 2 = 3; accepted 2 of 2: s = 0
    #   ema_H = 2, ema_s = 0.1875; K = ceil(e^2 = 7.389) = 8; W = ceil(1 + 1.5) = 3
    assert c.update(torch.tensor([[4.0, 2.0, 9.0, 9.0]]), [2], [2]) == (8, 3)
    assert c.ema_entropy == 2.0 and c.ema_shortfall == 0.1875
    # step 3: two batch rows: row 0 gen_len 0 counts position 0 alone (H 0.5), shortfall 0 / 1;
    #   row 1 gen_len 4 (H 1, 1, 1, 1.5), accepted 5 > gen: shortfall 0.  H = (0.5 + 4.5) / 5 = 1
    #   ema_H = 1.5, ema_s = 0.09375; K = ceil(e^1.5 = 4.48) = 5; W = ceil(1.75) = 2
    e = torch.tensor([[0.5, 7.0, 7.0, 7.0], [1.0, 1.0, 1.0, 1.5]])
    assert c.update(e, [0, 5], [0, 4]) == (5, 2)
    assert c.ema_entropy == 1.5 and c.ema_shortfall == 0.09375


def test_constant_signals_closed_form():
    H, rho = 2.2, 0.3
    c = oracle.Breadth(1, 1000, 1, 101, rho)
    for t in range(1, 25):
        K, W = c.update(torch.full((3, 5), H), [2, 2, 2], [5, 5, 5])       # shortfall 3/5 on every row
        f = 1 - (1 - rho) ** t
        assert abs(c.ema_entropy - H * f) < 1e-6 and abs(c.ema_shortfall - 0.6 * f) < 1e-12   # H is fp32 on the way in
        assert K == math.ceil(math.exp(c.ema_entropy)) and W == math.ceil(1 + 100 * c.ema_shortfall)


def test_uniform_drafter_asks_for_about_n_candidates_and_full_acceptance_for_the_narrowest_beam():
    n = 12
    c = oracle.Breadth(1, 32, 2, 16, 1.0)                                   # rho = 1: no memory
    K, W = c.update(torch.full((2, 3), math.log(n) - 1e-4), [3, 3], [3, 3])
    assert K == n and W == 2                                                # perplexity n, nothing cut short
    K, W = c.update(torch.full((2, 3), math.log(n) + 1e-4), [0, 0], [3, 3])
    assert K == n + 1 and W == 16                                           # everything rejected: the widest beam
    K, W = c.update(torch.full((2, 3), 0.0), [3, 3], [3, 3])
    assert K == 1                                                           # one-hot rows: one candidate


def test_guard_rails():
    g = torch.Generator().manual_seed(0)
    c = oracle.Breadth(3, 15, 2, 8, 0.5)
    for _ in range(200):
        B, L = int(torch.randint(1, 5, (1,), generator=g)), int(torch.randint(1, 9, (1,), generator=g))
        e = 12.0 * torch.rand((B, L), generator=g)
        K, W = c.update(e, torch.randint(0, L + 2, (B,), generator=g), torch.randint(0, L + 1, (B,), generator=g))
        assert 3 <= K <= 15 and 2 <= W <= 8
