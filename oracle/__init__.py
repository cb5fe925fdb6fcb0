"""CPU oracle for the draft-and-verify step: TEST INFRASTRUCTURE, not product code.

Thin ctypes wrapper over ``dsp_oracle.c`` (plain scalar C, double precision).
Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg import
this package; it imports nothing from the CUDA package and the CUDA package
never imports it.  Inputs are torch CPU tensors (fp32 or bf16 logits); outputs
are torch CPU tensors.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from types import SimpleNamespace

import numpy as np
import torch

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "dsp_oracle.c")
_LIB = os.path.join(_DIR, "liboracle.so")
_lock = threading.Lock()
_lib = None

NONFINITE_INPUT = 1
ZERO_RESIDUAL = 2
NO_BONUS_ROW = 4
EOS_ACCEPTED = 8
EOS_STOPPED = 16


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-Wall",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _AdlState(C.Structure):
    _fields_ = [("ema_gen", C.c_double), ("ema_acc", C.c_double), ("k", C.c_int32),
                ("steps", C.c_int32)]


def lib():
    global _lib
    with _lock:
        if _lib is None:
            _lib = C.CDLL(build())
            _lib.orc_residual_probe.restype = C.c_int64
            _lib.orc_proxy_score.restype = C.c_float
            _lib.orc_trigram_score.restype = C.c_float
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle uses (batch rows are split over them)."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return 0
    if t.dtype == torch.bfloat16:
        return 1
    raise TypeError("logits must be fp32 or bf16")


def _logits_ptr(t: torch.Tensor):
    """Pointer to the raw words of a contiguous CPU logits tensor (kept alive by the caller)."""
    assert t.device.type == "cpu" and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _np(t, dtype):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        t = t.detach().cpu().contiguous().numpy()
    return np.ascontiguousarray(t, dtype=dtype)


def row_stats(row: torch.Tensor):
    """(lse, entropy, argmax, bad) of one vocabulary row, all in double."""
    row = row.contiguous()
    lse, H, am = C.c_double(), C.c_double(), C.c_int64()
    bad = lib().orc_row_stats(_logits_ptr(row), _dtype_code(row), C.c_int64(row.numel()),
                              C.byref(lse), C.byref(H), C.byref(am))
    return lse.value, H.value, am.value, bad


def lattice_build(draft: torch.Tensor, K_max: int, tau: float = 0.0, eos_id: int = -1):
    draft = draft.contiguous()
    B, L, V = draft.shape
    KC = K_max + (1 if eos_id >= 0 else 0)
    o = SimpleNamespace(
        cand_id=np.empty((B, L, KC), np.int32), cand_logit=np.empty((B, L, KC), np.float32),
        cand_logp=np.empty((B, L, KC), np.float32), cand_count=np.empty((B, L), np.int32),
        lse=np.empty((B, L), np.float32), lse64=np.empty((B, L), np.float64),
        entropy=np.empty((B, L), np.float32), gen_len=np.empty((B,), np.int32),
        row_status=np.zeros((B,), np.uint32))
    rc = lib().orc_lattice_build(
        _logits_ptr(draft), _dtype_code(draft), B, L, C.c_int64(V), K_max, C.c_double(float(np.float32(tau))),
        eos_id, _p(o.cand_id), _p(o.cand_logit), _p(o.cand_logp), _p(o.cand_count), _p(o.lse),
        _p(o.lse64), _p(o.entropy), _p(o.gen_len), _p(o.row_status))
    if rc != 0:
        raise ValueError("orc_lattice_build: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def cps_search(cand_id, cand_logit, lse64, cand_count, prev_token, table, *, W: int, lam: float,
               eos_id: int = -1, proxy_kind: int = 0, table_log2: int = 0, hash_seed: int = 0,
               V: int = 0, ver_score=None, mu: float = 0.0):
    cand_id = _np(cand_id, np.int32)
    cand_logit = _np(cand_logit, np.float32)
    lse64 = _np(lse64, np.float64)
    cand_count = _np(cand_count, np.int32)
    prev_token = _np(prev_token, np.int32)
    table = _np(table, np.float32)
    B, L, KC = cand_id.shape
    o = SimpleNamespace(
        path=np.empty((B, L), np.int32), path_slot=np.empty((B, L), np.int32),
        path_len=np.empty((B,), np.int32), path_score=np.empty((B,), np.float32),
        beam_ids=np.empty((B, W, L), np.int32), beam_score=np.empty((B, W), np.float32),
        beam_cum=np.empty((B, W), np.float32), row_status=np.zeros((B,), np.uint32))
    ver = _np(ver_score, np.float32)
    assert ver is None or ver.shape == (B, L, KC)
    rc = lib().orc_cps_search_biased(
        _p(cand_id), _p(cand_logit), _p(lse64), _p(cand_count), B, L, KC, _p(prev_token),
        proxy_kind, _p(table), table_log2, C.c_uint32(hash_seed & 0xFFFFFFFF), C.c_int64(V), W,
        C.c_float(lam), eos_id, _p(ver) if ver is not None else None, C.c_float(mu), _p(o.path), _p(o.path_slot), _p(o.path_len), _p(o.path_score),
        _p(o.beam_ids), _p(o.beam_score), _p(o.beam_cum), _p(o.row_status))
    if rc != 0:
        raise ValueError("orc_cps_search: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def proxy_score(table, prev: int, cur: int, *, proxy_kind=0, table_log2=0, hash_seed=0, V=0) -> float:
    table = _np(table, np.float32)
    return float(lib().orc_proxy_score(proxy_kind, _p(table), table_log2,
                                       C.c_uint32(hash_seed & 0xFFFFFFFF), C.c_int64(V), prev, cur))


def beam_tree(beam_ids, path_len):
    """Token tree of the beams [B,W,L]: node_token / node_parent / node_depth [B,W*L], beam_node [B,W,L], n_nodes [B]."""
    beam_ids = _np(beam_ids, np.int32)
    path_len = _np(path_len, np.int32)
    B, W, L = beam_ids.shape
    N = W * L
    o = SimpleNamespace(node_token=np.empty((B, N), np.int32), node_parent=np.empty((B, N), np.int32),
                        node_depth=np.empty((B, N), np.int32), beam_node=np.empty((B, W, L), np.int32),
                        n_nodes=np.empty((B,), np.int32))
    rc = lib().orc_beam_tree(_p(beam_ids), _p(path_len), B, W, L, _p(o.node_token), _p(o.node_parent),
                             _p(o.node_depth), _p(o.beam_node), _p(o.n_nodes))
    if rc != 0:
        raise ValueError("orc_beam_tree: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def verify_tree(target: torch.Tensor, tree: SimpleNamespace, L: int):
    """Greedy verification of the tree; target is [B, 1 + N, V] (row 0: after the prefix, row 1+n: after node n)."""
    target = target.contiguous()
    B, N1, V = target.shape
    N = N1 - 1
    o = SimpleNamespace(accepted_len=np.empty((B,), np.int32), accepted_node=np.empty((B, L), np.int32),
                        next_token=np.empty((B,), np.int32), row_status=np.zeros((B,), np.uint32))
    rc = lib().orc_verify_tree(_logits_ptr(target), _dtype_code(target), B, N, C.c_int64(V),
                               _p(_np(tree.node_token, np.int32)), _p(_np(tree.node_parent, np.int32)),
                               _p(_np(tree.n_nodes, np.int32)), L, _p(o.accepted_len), _p(o.accepted_node),
                               _p(o.next_token), _p(o.row_status))
    if rc != 0:
        raise ValueError("orc_verify_tree: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def unmask_step(logits: torch.Tensor, tokens, masked, n_update: int):
    """One refinement step (Eq. 5, top-K by confidence); returns new tokens / masked and the per-position
    argmax, confidence (log-probability of the argmax, fp32), n_left and row_status."""
    logits = logits.contiguous()
    B, L, V = logits.shape
    o = SimpleNamespace(
        tokens=_np(tokens, np.int32).copy(), masked=_np(masked, np.uint8).copy(),
        argmax=np.empty((B, L), np.int32), confidence=np.empty((B, L), np.float32),
        n_left=np.empty((B,), np.int32), row_status=np.zeros((B,), np.uint32))
    rc = lib().orc_unmask_step(_logits_ptr(logits), _dtype_code(logits), B, L, C.c_int64(V), int(n_update),
                               _p(o.tokens), _p(o.masked), _p(o.argmax), _p(o.confidence), _p(o.n_left),
                               _p(o.row_status))
    if rc != 0:
        raise ValueError("orc_unmask_step: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def trigram_score(table, prev2: int, prev: int, cur: int, *, table_log2=0, hash_seed=0) -> float:
    table = _np(table, np.float32)
    return float(lib().orc_trigram_score(_p(table), table_log2, C.c_uint32(hash_seed & 0xFFFFFFFF),
                                         prev2, prev, cur))


def verify(target: torch.Tensor, draft, path, path_len, mode=None, u=None, eos_id: int = -1):
    target = target.contiguous()
    B, Lt, V = target.shape
    path = _np(path, np.int32)
    L = path.shape[1]
    path_len = _np(path_len, np.int32)
    mode_np = _np(mode, np.uint8)
    u_np = _np(u, np.float32)
    if draft is not None:
        draft = draft.contiguous()
        assert draft.dtype == target.dtype and tuple(draft.shape) == (B, L, V)
    if mode_np is not None and mode_np.any():
        assert draft is not None and u_np is not None and u_np.shape == (B, L + 1)
    o = SimpleNamespace(
        accepted_len=np.empty((B,), np.int32), next_token=np.empty((B,), np.int32),
        ratio=np.empty((B, L), np.float32), tgt_argmax=np.empty((B, Lt), np.int32),
        tgt_lse=np.empty((B, Lt), np.float32), row_status=np.zeros((B,), np.uint32))
    rc = lib().orc_verify(
        _logits_ptr(target), _logits_ptr(draft) if draft is not None else None, _dtype_code(target),
        B, L, Lt, C.c_int64(V), _p(path), _p(path_len),
        _p(mode_np) if mode_np is not None else None, _p(u_np) if u_np is not None else None, eos_id,
        _p(o.accepted_len), _p(o.next_token), _p(o.ratio), _p(o.tgt_argmax), _p(o.tgt_lse),
        _p(o.row_status))
    if rc != 0:
        raise ValueError("orc_verify: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})


def residual_probe(target_row: torch.Tensor, draft_row, u: float, probe: int = -1):
    """Oracle's inverse-CDF draw from [p-q]_+ (or from p if draft_row is None), and its
    normalised CDF just below / at token ``probe``: returns (token, F_lo, F_hi, r_probe)."""
    target_row = target_row.contiguous()
    if draft_row is not None:
        draft_row = draft_row.contiguous()
    F_lo, F_hi, r = C.c_double(float("nan")), C.c_double(float("nan")), C.c_double(float("nan"))
    tok = lib().orc_residual_probe(
        _logits_ptr(target_row), _logits_ptr(draft_row) if draft_row is not None else None,
        _dtype_code(target_row), C.c_int64(target_row.numel()), C.c_double(float(np.float32(u))),
        C.c_int64(probe), C.byref(F_lo), C.byref(F_hi), C.byref(r))
    return int(tok), F_lo.value, F_hi.value, r.value


class Adl:
    """ADL controller state (Eq. 9-11); ``k`` is the draft length for the next step."""

    def __init__(self, k_min=20, k_max=30, delta=10.0, rho=0.5, granularity=1):
        self.p = (int(k_min), int(k_max), float(delta), float(rho), int(granularity))
        self.st = _AdlState()
        lib().orc_adl_init(C.byref(self.st), int(k_max))

    @property
    def k(self) -> int:
        return int(self.st.k)

    @property
    def ema_gen(self) -> float:
        return float(self.st.ema_gen)

    @property
    def ema_acc(self) -> float:
        return float(self.st.ema_acc)

    def update(self, accepted_len, gen_len) -> int:
        a = _np(accepted_len, np.int32).reshape(-1)
        g = _np(gen_len, np.int32).reshape(-1)
        assert a.size == g.size and a.size > 0
        k_min, k_max, delta, rho, gran = self.p
        return int(lib().orc_adl_update(C.byref(self.st), _p(a), _p(g), int(a.size), k_min, k_max,
                                        C.c_double(delta), C.c_double(rho), gran))


class _BreadthState(C.Structure):
    _fields_ = [("ema_entropy", C.c_double), ("ema_shortfall", C.c_double), ("K", C.c_int32), ("W", C.c_int32),
                ("steps", C.c_int32)]


class Breadth:
    """Breadth controller state (the reading of the paper's future work iii): ``K`` / ``W`` for the next step."""

    def __init__(self, K_min=1, K_max=16, W_min=1, W_max=16, rho=0.5):
        self.p = (int(K_min), int(K_max), int(W_min), int(W_max), float(rho))
        self.st = _BreadthState()
        lib().orc_breadth_init(C.byref(self.st), int(K_max), int(W_max))

    K = property(lambda self: int(self.st.K))
    W = property(lambda self: int(self.st.W))
    ema_entropy = property(lambda self: float(self.st.ema_entropy))
    ema_shortfall = property(lambda self: float(self.st.ema_shortfall))

    def update(self, entropy, accepted_len, gen_len):
        e = _np(entropy, np.float32)
        a = _np(accepted_len, np.int32).reshape(-1)
        g = _np(gen_len, np.int32).reshape(-1)
        B, L = e.shape
        assert a.size == g.size == B
        K_min, K_max, W_min, W_max, rho = self.p
        rc = lib().orc_breadth_update(C.byref(self.st), _p(e), _p(a), _p(g), B, L, K_min, K_max, W_min, W_max,
                                      C.c_double(rho))
        if rc != 0:
            raise ValueError("orc_breadth_update: bad arguments")
        return self.K, self.W


def verify_tree_stochastic(target: torch.Tensor, draft: torch.Tensor, tree: SimpleNamespace, u):
    """Stochastic verification of the tree; target [B, 1 + N, V], draft [B, L, V], u [B, N + 1]."""
    target, draft = target.contiguous(), draft.contiguous()
    B, N1, V = target.shape
    N, L = N1 - 1, draft.shape[1]
    assert draft.dtype == target.dtype and draft.shape[0] == B and draft.shape[2] == V
    u_np = _np(u, np.float32)
    assert u_np.shape == (B, N + 1)
    o = SimpleNamespace(accepted_len=np.empty((B,), np.int32), accepted_node=np.empty((B, L), np.int32),
                        next_token=np.empty((B,), np.int32), row_status=np.zeros((B,), np.uint32),
                        margin=np.empty((B,), np.float64))
    rc = lib().orc_verify_tree_stochastic(
        _logits_ptr(target), _logits_ptr(draft), _dtype_code(target), B, N, L, C.c_int64(V),
        _p(_np(tree.node_token, np.int32)), _p(_np(tree.node_parent, np.int32)), _p(_np(tree.n_nodes, np.int32)),
        _p(u_np), _p(o.accepted_len), _p(o.accepted_node), _p(o.next_token), _p(o.row_status), _p(o.margin))
    if rc != 0:
        raise ValueError("orc_verify_tree_stochastic: bad arguments")
    return SimpleNamespace(**{k: torch.from_numpy(v) for k, v in vars(o).items()})
