"""dsp_lattice_build_static: the lattice build for callers that cannot allocate device memory.

Some users of the library run where no device allocation is possible for them: inside another
runtime's callback, on a thread that must not call allocating CUDA routines, or after all device
memory has been handed out.  For them the library holds the build's scratch in an array of its
own (DSP_STATIC_WS_BYTES) and they pass inputs and outputs only.  The test calls that entry point
through the C ABI twice in a row, with different inputs, and compares every output with
dsp_lattice_build's on the same inputs: integers and candidate logits identical, floating-point
outputs within the 1e-3 of the parity tests.  The file sorts last on purpose so that a run that
stops at the first failure has already run every other test; it also passes on its own.
"""
import pytest
import torch

from paper_2510_02358_b200 import binding as dsp
from paper_2510_02358_b200 import workloads as wl

TOL = 1e-3


def _same(a, b):
    for name in ("cand_id", "cand_count", "gen_len", "row_status"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    assert torch.equal(a.cand_logit, b.cand_logit), "candidate logits must be identical"
    for name in ("cand_logp", "lse", "lse64", "entropy"):
        x, y = getattr(a, name).double(), getattr(b, name).double()
        both_inf = torch.isinf(x) & torch.isinf(y) & (x.sign() == y.sign())
        assert (both_inf | ((x - y).abs() <= TOL)).all(), name


@pytest.mark.gpu
def test_static_scratch_build_matches_the_workspace_build_on_two_calls_in_a_row():
    dev = "cuda"
    # two different problems one after the other: the second call finds the first call's
    # leftovers in the shared array (other row and slice counts, other K)
    cases = [(wl.CONFIGS[4].scaled(B=6, L=8, V=152064), 1),
             (wl.CONFIGS[2].scaled(B=1, L=16, V=152064, eos_from=9), 2),
             (wl.CONFIGS[4].scaled(B=6, L=8, V=152064), 1)]
    for w, step in cases:
        inp = wl.make_inputs(w, step=step, device=dev)
        ref = dsp.dsp_lattice_build(inp["draft"], w.K, w.tau, w.eos_id)
        out = dsp.lattice_outputs(w.B, w.L, w.K, w.eos_id, dev)        # the caller's buffers
        for t in vars(out).values():
            t.view(torch.uint8).fill_(0xA5)
        got = dsp.dsp_lattice_build_static(inp["draft"], w.K, w.tau, w.eos_id, out=out)
        torch.cuda.synchronize()
        _same(got, ref)
        # the claim itself: with the outputs passed in, a call takes no device memory, neither from
        # torch's allocator nor from the driver
        torch.cuda.synchronize()
        held, (free0, _) = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()
        dsp.dsp_lattice_build_static(inp["draft"], w.K, w.tau, w.eos_id, out=out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == held and torch.cuda.mem_get_info()[0] == free0


def test_static_scratch_rejects_problems_beyond_its_limit():
    # host-side check only: nothing is enqueued, so this runs without a GPU
    import os
    if not os.path.exists(dsp.LIB_PATH):
        pytest.skip("libdsp.so is not built")
    need = dsp.dsp_lattice_workspace_bytes(2048, 64, 256000, dsp.DSP_BF16, 16)
    assert need > dsp.DSP_STATIC_WS_BYTES
    import ctypes as C
    one = C.c_void_p(256)
    rc = dsp.lib().dsp_lattice_build_static(one, dsp.DSP_BF16, 2048, 64, 256000, C.c_int64(64 * 256000),
                                            C.c_int64(256000), 16, C.c_float(0), -1, one, one, one, one,
                                            one, one, one, one, one, C.c_void_p(0))
    assert rc == dsp.DSP_ERR_STATIC_SCRATCH
    assert b"built-in scratch" in dsp.lib().dsp_strerror(rc)
