"""B200-native draft-and-verify core of DiffuSpec (lattice build, CPS, verify, ADL).

``paper_2510_02358_b200.binding`` is the thin ctypes layer over the C-ABI CUDA
library (``libdsp.so``, built in-tree by ``paper_2510_02358_b200.build``);
``paper_2510_02358_b200.workloads`` draws the seeded synthetic inputs.
Nothing here falls back to a CPU implementation: without the CUDA library the
binding raises.
"""
__all__ = ["binding", "build", "workloads"]
