"""Pins for the oracle's adaptive draft-length controller (Eq. 9-11, Algorithm 1 init)."""
import math
import os

import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "adl_trajectories.txt")


def golden_cases():
    cases = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        a, b, c = [s.split() for s in line.split("|")]
        cases.setdefault(a[0], []).append(
            (tuple(float(v) for v in a[1:]), (int(b[0]), int(b[1])), (float(c[0]), float(c[1]), int(c[2]))))
    return cases


@pytest.mark.parametrize("case", sorted(golden_cases()))
def test_hand_computed_trajectories(case):
    rows = golden_cases()[case]
    k_min, k_max, delta, rho, gran = rows[0][0]
    adl = oracle.Adl(int(k_min), int(k_max), delta, rho, int(gran))
    assert adl.k == int(k_max) and adl.ema_gen == 0.0 and adl.ema_acc == 0.0     # Algorithm 1 init
    for _, (gen, acc), (eg, ea, k) in rows:
        assert adl.update([acc], [gen]) == k
        assert adl.ema_gen == eg and adl.ema_acc == ea and adl.k == k


def test_constant_signal_closed_form():
    c, rho = 17, 0.3
    adl = oracle.Adl(1, 1000, 5.0, rho)
    for t in range(1, 30):
        k = adl.update([0], [c])                          # acceptance lags: no growth term
        ema = c * (1 - (1 - rho) ** t)                    # L~_t = c (1 - (1-rho)^t)
        assert abs(adl.ema_gen - ema) < 1e-12
        assert k == math.ceil(ema - 1e-12)


def test_rho_one_has_no_memory():
    adl = oracle.Adl(4, 64, 6.0, 1.0)
    assert adl.update([9], [9]) == 15                     # ceil(9 + 6)
    assert adl.update([3], [20]) == 20                    # acceptance lags: ceil(20)
    assert adl.update([40], [41]) == 41
    assert adl.update([60], [60]) == 64                   # clipped at k_max
    assert adl.update([0], [1]) == 4                      # clipped at k_min


def test_guardrails_and_batch_mean():
    adl = oracle.Adl(20, 30, 10.0, 0.5)
    import random
    rng = random.Random(0)
    for _ in range(200):
        B = rng.randint(1, 5)
        k = adl.update([rng.randint(0, 40) for _ in range(B)], [rng.randint(0, 40) for _ in range(B)])
        assert 20 <= k <= 30
    a = oracle.Adl(1, 100, 0.0, 1.0)
    assert a.update([0, 0, 0, 0], [3, 4, 4, 4]) == 4      # mean 3.75 -> ceil
    b = oracle.Adl(1, 100, 0.0, 1.0)
    assert b.update([0], [3]) == 3
