"""The C-ABI library without a GPU: it loads, exports what the header declares, rejects bad
arguments before touching CUDA, and its host-side controller matches the oracle."""
import ctypes as C
import os
import re

import pytest

import oracle
from paper_2510_02358_b200 import binding as dsp
from paper_2510_02358_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "dsp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(dsp_[a-z0-9_]+)\s*\(", text))
    assert declared == set(dsp.EXPORTS)
    lib = dsp.lib()
    for name in declared:
        assert hasattr(lib, name), name
    assert dsp.dsp_version() == 1
    assert lib.dsp_strerror(dsp.DSP_ERR_WORKSPACE) == b"workspace too small"


def test_workspace_queries_and_limits():
    n = dsp.dsp_lattice_workspace_bytes(64, 32, 152064, dsp.DSP_BF16, 16)
    assert 0 < n < (1 << 26) and n % 256 == 0
    assert dsp.dsp_verify_workspace_bytes(64, 32, 32, 152064, dsp.DSP_BF16) % 256 == 0
    for bad, code in (((1, 8, 1000, 7, 4), dsp.DSP_ERR_UNSUPPORTED),          # dtype
                      ((1, 8, 1000, 0, 33), dsp.DSP_ERR_UNSUPPORTED),         # K_max > 32
                      ((1, 2000, 1000, 0, 4), dsp.DSP_ERR_UNSUPPORTED),       # L > 1024
                      ((1, 0, 1000, 0, 4), dsp.DSP_ERR_INVALID_ARG),
                      ((-1, 8, 1000, 0, 4), dsp.DSP_ERR_INVALID_ARG)):
        with pytest.raises(dsp.DspError) as e:
            dsp.dsp_lattice_workspace_bytes(*bad)
        assert e.value.code == code
    with pytest.raises(dsp.DspError):
        dsp.dsp_verify_workspace_bytes(1, 8, 10, 1000, 0)                       # Lt > L + 1


def test_device_entry_points_reject_bad_arguments_on_the_host():
    lib = dsp.lib()
    z, one = C.c_void_p(0), C.c_void_p(256)
    # null pointers
    assert lib.dsp_lattice_build(z, 0, 1, 8, 100, C.c_int64(800), C.c_int64(100), 4, C.c_float(0), -1,
                                 z, z, z, z, z, z, z, z, z, z, C.c_size_t(0), z) == dsp.DSP_ERR_INVALID_ARG
    # stride shorter than the vocabulary
    assert lib.dsp_lattice_build(one, 0, 1, 8, 100, C.c_int64(800), C.c_int64(50), 4, C.c_float(0), -1,
                                 one, one, one, one, one, one, one, one, one, one, C.c_size_t(1 << 20), z) \
        == dsp.DSP_ERR_INVALID_ARG
    # workspace too small / misaligned
    assert lib.dsp_lattice_build(one, 0, 1, 8, 100, C.c_int64(800), C.c_int64(100), 4, C.c_float(0), -1,
                                 one, one, one, one, one, one, one, one, one, one, C.c_size_t(16), z) \
        == dsp.DSP_ERR_WORKSPACE
    assert lib.dsp_lattice_build(one, 0, 1, 8, 100, C.c_int64(800), C.c_int64(100), 4, C.c_float(0), -1,
                                 one, one, one, one, one, one, one, one, one, C.c_void_p(8),
                                 C.c_size_t(1 << 20), z) == dsp.DSP_ERR_INVALID_ARG
    # batch of zero rows is a no-op
    assert lib.dsp_lattice_build(z, 0, 0, 8, 100, C.c_int64(800), C.c_int64(100), 4, C.c_float(0), -1,
                                 z, z, z, z, z, z, z, z, z, z, C.c_size_t(0), z) == dsp.DSP_OK
    # read probe: null and misaligned pointers, too few bytes
    assert lib.dsp_read_probe(z, C.c_size_t(1024), one, z) == dsp.DSP_ERR_INVALID_ARG
    assert lib.dsp_read_probe(one, C.c_size_t(1024), z, z) == dsp.DSP_ERR_INVALID_ARG
    assert lib.dsp_read_probe(C.c_void_p(264), C.c_size_t(1024), one, z) == dsp.DSP_ERR_INVALID_ARG
    assert lib.dsp_read_probe(one, C.c_size_t(8), one, z) == dsp.DSP_ERR_INVALID_ARG
    # path search: beam too wide, bad table size, bad lambda
    def cps(W=4, log2=10, lam=0.5, kind=0):
        return lib.dsp_cps_search(one, one, one, one, 1, 8, 5, one, kind, one, log2, C.c_uint32(0), 100,
                                  W, C.c_float(lam), -1, one, one, one, one, z, z, z, z, z)
    assert cps(W=33) == dsp.DSP_ERR_UNSUPPORTED and cps(log2=0) == dsp.DSP_ERR_INVALID_ARG
    assert cps(lam=1.5) == dsp.DSP_ERR_INVALID_ARG and cps(kind=4) == dsp.DSP_ERR_UNSUPPORTED
    # verify: stochastic rows need the draft side
    assert lib.dsp_verify(one, 0, 1, 8, 8, 100, C.c_int64(800), C.c_int64(100), z, C.c_int64(0), C.c_int64(0),
                          one, one, one, z, z, 5, 0, z, z, -1, one, one, z, z, z, one, one,
                          C.c_size_t(1 << 20), z) == dsp.DSP_ERR_INVALID_ARG


def test_adl_host_entry_points_follow_the_golden_trajectories():
    from test_oracle_adl import golden_cases
    for case, rows in golden_cases().items():
        k_min, k_max, delta, rho, gran = rows[0][0]
        st, p = dsp.dsp_adl_init(k_min, k_max, delta, rho, gran)
        ref = oracle.Adl(int(k_min), int(k_max), delta, rho, int(gran))
        assert st.k == int(k_max) and st.ema_gen == 0.0
        for _, (gen, acc), (eg, ea, k) in rows:
            assert dsp.dsp_adl_update(st, p, [acc], [gen]) == k == ref.update([acc], [gen])
            assert st.ema_gen == eg and st.ema_acc == ea
    with pytest.raises(dsp.DspError):
        dsp.dsp_adl_init(k_min=10, k_max=5)
    with pytest.raises(dsp.DspError):
        dsp.dsp_adl_init(rho=0.0)


def test_breadth_host_entry_points_follow_the_hand_computed_steps_and_the_oracle():
    import torch
    import oracle
    st, prm = dsp.dsp_breadth_init(2, 16, 1, 9, 0.5)
    assert (st.K, st.W) == (16, 9)
    # the hand-computed steps of tests/test_oracle_breadth.py
    assert dsp.dsp_breadth_update(st, prm, torch.full((1, 4), 2.0), [1], [4]) == (3, 4)
    assert dsp.dsp_breadth_update(st, prm, torch.tensor([[4.0, 2.0, 9.0, 9.0]]), [2], [2]) == (8, 3)
    assert dsp.dsp_breadth_update(st, prm, torch.tensor([[0.5, 7.0, 7.0, 7.0], [1.0, 1.0, 1.0, 1.5]]), [0, 5], [0, 4]) == (5, 2)
    assert st.ema_entropy == 1.5 and st.ema_shortfall == 0.09375 and st.steps == 3
    # a random trajectory against the oracle, state for state
    g = torch.Generator().manual_seed(1)
    st, prm = dsp.dsp_breadth_init(3, 15, 2, 8, 0.3)
    ref = oracle.Breadth(3, 15, 2, 8, 0.3)
    for _ in range(100):
        B, L = int(torch.randint(1, 5, (1,), generator=g)), int(torch.randint(1, 9, (1,), generator=g))
        e = 6.0 * torch.rand((B, L), generator=g)
        acc, gen = torch.randint(0, L + 2, (B,), generator=g), torch.randint(0, L + 1, (B,), generator=g)
        assert dsp.dsp_breadth_update(st, prm, e, acc, gen) == ref.update(e, acc, gen)
        assert st.ema_entropy == ref.ema_entropy and st.ema_shortfall == ref.ema_shortfall
    # argument errors
    import ctypes as C
    bad = dsp.BreadthParams(4, 2, 1, 8, 0.5)
    assert dsp.lib().dsp_breadth_init(C.byref(dsp.BreadthState()), C.byref(bad)) == dsp.DSP_ERR_INVALID_ARG
    bad = dsp.BreadthParams(1, 64, 1, 8, 0.5)                      # beyond DSP_MAX_K
    assert dsp.lib().dsp_breadth_init(C.byref(dsp.BreadthState()), C.byref(bad)) == dsp.DSP_ERR_INVALID_ARG
