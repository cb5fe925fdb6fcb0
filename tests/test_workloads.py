"""The seeded generators: shapes, dtypes, determinism, and the structure each recipe promises."""
import torch

import oracle
from paper_2510_02358_b200 import workloads as wl


def test_shapes_dtypes_determinism():
    for cid, w in wl.CONFIGS.items():
        s = w.scaled(B=min(w.B, 2), L=min(w.L, 4), V=4096)
        a, b = wl.make_inputs(s, step=3), wl.make_inputs(s, step=3)
        assert a["draft"].shape == (s.B, s.L, s.V) and a["draft"].dtype == s.dtype
        assert a["target"].shape == (s.B, s.L, s.V) and a["u"].shape == (s.B, s.L + 1)
        for k in ("draft", "target", "prev_token", "table", "mode", "u"):
            assert torch.equal(a[k], b[k]), (cid, k)
        assert not torch.equal(a["draft"], wl.make_inputs(s, step=4)["draft"])
        assert a["table"].min() >= -8.0 and a["table"].max() <= 0.0 and a["table"].numel() == 1 << 20
        assert 0.0 <= a["u"].min() and a["u"].max() < 1.0
    assert wl.CONFIGS[4].logits_bytes == 622_854_144 and wl.CONFIGS[5].logits_bytes == 8_388_608_000


def test_chunking_does_not_change_the_bytes_layout():
    s = wl.CONFIGS[3].scaled(B=4, L=2, V=1024)
    a = wl.make_inputs(s, chunk_elems=1 << 30)
    assert a["mode"].tolist() == [1, 1, 1, 1]
    m = wl.make_inputs(wl.CONFIGS[4].scaled(B=4, L=2, V=1024))["mode"]
    assert m.tolist() == [0, 1, 0, 1]


def test_zipf_rows_are_permuted_power_laws():
    s = wl.CONFIGS[5].scaled(B=1, L=2, V=8192)
    x = wl.make_inputs(s)["draft"].float()
    top = x.sort(dim=-1, descending=True).values
    assert (top[..., 0] > -1.0).all() and (top[..., 99] < -3.5).all()        # -1.1 ln 100 = -5.07 +- noise


def test_planted_eos_makes_gen_len():
    s = wl.CONFIGS[2].scaled(L=16, V=4096, eos_id=4095, eos_from=5)
    x = wl.make_inputs(s)
    lat = oracle.lattice_build(x["draft"], s.K, eos_id=s.eos_id)
    assert lat.gen_len.item() == 5
    assert wl.eos_walk(50) == wl.eos_walk(50) and all(4 <= c <= 40 for c in wl.eos_walk(50))
