"""Thin ctypes binding of the C ABI in ``include/dsp.h`` (argument marshalling only).

Functions carry the C entry points' names.  Tensors are torch CUDA tensors whose
``data_ptr()`` is handed to the library; outputs and the scratch workspace are
allocated here with torch (or passed in by the caller to reuse them) and the
call is enqueued on torch's current stream.  There is no CPU fallback: if the
CUDA library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from types import SimpleNamespace
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdsp.so")

DSP_OK, DSP_ERR_INVALID_ARG, DSP_ERR_UNSUPPORTED, DSP_ERR_WORKSPACE, DSP_ERR_CUDA = 0, -1, -2, -3, -4
DSP_ERR_STATIC_SCRATCH = -5
DSP_STATIC_WS_BYTES = 4 << 20
DSP_F32, DSP_BF16 = 0, 1
ROW_NONFINITE_INPUT, ROW_ZERO_RESIDUAL, ROW_NO_BONUS_ROW, ROW_EOS_ACCEPTED, ROW_EOS_STOPPED = 1, 2, 4, 8, 16
ROW_TIMEOUT = 32
DSP_MAX_K, DSP_MAX_W, DSP_MAX_L = 32, 32, 1024

EXPORTS = ["dsp_strerror", "dsp_last_cuda_error", "dsp_version", "dsp_profile_events", "dsp_read_probe", "dsp_lattice_workspace_bytes",
           "dsp_lattice_build", "dsp_lattice_build_static", "dsp_cps_search", "dsp_cps_search_biased", "dsp_verify_workspace_bytes", "dsp_verify", "dsp_draft_verify_step",
           "dsp_step_graph_create", "dsp_step_graph_launch", "dsp_step_graph_destroy",
           "dsp_unmask_workspace_bytes", "dsp_unmask_step",
           "dsp_shard_workspace_bytes", "dsp_lattice_shard", "dsp_merge_workspace_bytes", "dsp_lattice_merge",
           "dsp_target_shard", "dsp_verify_merge_workspace_bytes", "dsp_verify_merge",
           "dsp_residual_sample_workspace_bytes", "dsp_residual_sample",
           "dsp_beam_tree", "dsp_verify_tree_workspace_bytes", "dsp_verify_tree", "dsp_verify_tree_stochastic",
           "dsp_adl_init", "dsp_adl_update", "dsp_breadth_init", "dsp_breadth_update"]


class DspError(RuntimeError):
    def __init__(self, fn: str, code: int):
        msg = lib().dsp_strerror(code).decode()
        if code == DSP_ERR_CUDA:
            msg += " [cudaError %d]" % lib().dsp_last_cuda_error()
        super().__init__("%s: %s (%d)" % (fn, msg, code))
        self.code = code


class AdlParams(C.Structure):
    _fields_ = [("k_min", C.c_int32), ("k_max", C.c_int32), ("delta", C.c_double),
                ("rho", C.c_double), ("granularity", C.c_int32)]


class AdlState(C.Structure):
    _fields_ = [("ema_gen", C.c_double), ("ema_acc", C.c_double), ("k", C.c_int32),
                ("steps", C.c_int32)]


_lib = None


def lib():
    """Load ``libdsp.so`` (built in-tree by ``paper_2510_02358_b200.build``); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("CUDA library %s is not built; run paper_2510_02358_b200.build.build()"
                              % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        l.dsp_strerror.restype = C.c_char_p
        l.dsp_strerror.argtypes = [C.c_int32]
        for name in EXPORTS[1:]:
            getattr(l, name).restype = C.c_int32
        _lib = l
    return _lib


def _check(fn: str, code: int):
    if code != DSP_OK:
        raise DspError(fn, code)


def _ptr(t: Optional[torch.Tensor]):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DSP_F32
    if t.dtype == torch.bfloat16:
        return DSP_BF16
    raise DspError("dtype", DSP_ERR_UNSUPPORTED)


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _logits3(t: torch.Tensor, name: str):
    if t.dim() != 3 or not t.is_cuda or t.stride(2) != 1:
        raise ValueError("%s must be a CUDA tensor [B, L, V] with a contiguous vocabulary dimension" % name)
    return t.shape[0], t.shape[1], t.shape[2], t.stride(0), t.stride(1)


def dsp_version() -> int:
    return lib().dsp_version()


PROFILE_LATTICE_SCAN, PROFILE_TARGET_SCAN = 0, 1


def dsp_profile_events(point: int, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
    """Bracket the launches of one streaming kernel with two timing events (None, None = off).
    The events must have been recorded once before, so that torch has created them."""
    h = lambda e: C.c_void_p(0 if e is None else e.cuda_event)
    _check("dsp_profile_events", lib().dsp_profile_events(point, h(start), h(stop)))


def dsp_read_probe(buffer: torch.Tensor, sink: torch.Tensor) -> None:
    """Enqueue one read-only pass over ``buffer`` (contiguous CUDA tensor) on the current stream;
    ``sink`` is a CUDA tensor with at least 4 bytes that the kernel may write."""
    if not (buffer.is_cuda and buffer.is_contiguous() and sink.is_cuda and sink.numel() * sink.element_size() >= 4):
        raise ValueError("buffer must be a contiguous CUDA tensor and sink a CUDA tensor of at least 4 bytes")
    _check("dsp_read_probe", lib().dsp_read_probe(_ptr(buffer), C.c_size_t(buffer.numel() * buffer.element_size()),
                                                   _ptr(sink), _stream(None)))


def dsp_lattice_workspace_bytes(B: int, L: int, V: int, dtype: int, K_max: int) -> int:
    n = C.c_size_t(0)
    _check("dsp_lattice_workspace_bytes",
           lib().dsp_lattice_workspace_bytes(B, L, V, dtype, K_max, C.byref(n)))
    return n.value


def dsp_verify_workspace_bytes(B: int, L: int, Lt: int, V: int, dtype: int) -> int:
    n = C.c_size_t(0)
    _check("dsp_verify_workspace_bytes", lib().dsp_verify_workspace_bytes(B, L, Lt, V, dtype, C.byref(n)))
    return n.value


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=device)


def lattice_outputs(B: int, L: int, K_max: int, eos_id: int, device) -> SimpleNamespace:
    KC = K_max + (1 if eos_id >= 0 else 0)
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=device)
    return SimpleNamespace(
        cand_id=e((B, L, KC), torch.int32), cand_logit=e((B, L, KC), torch.float32),
        cand_logp=e((B, L, KC), torch.float32), cand_count=e((B, L), torch.int32),
        lse=e((B, L), torch.float32), lse64=e((B, L), torch.float64), entropy=e((B, L), torch.float32),
        gen_len=e((B,), torch.int32), row_status=e((B,), torch.int32))


def dsp_lattice_build(draft: torch.Tensor, K_max: int, tau: float = 0.0, eos_id: int = -1,
                      out: Optional[SimpleNamespace] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> SimpleNamespace:
    B, L, V, sb, sl = _logits3(draft, "draft")
    dt = _dtype(draft)
    if out is None:
        out = lattice_outputs(B, L, K_max, eos_id, draft.device)
    if workspace is None:
        workspace = alloc_workspace(dsp_lattice_workspace_bytes(B, L, V, dt, K_max), draft.device)
    _check("dsp_lattice_build", lib().dsp_lattice_build(
        _ptr(draft), dt, B, L, V, C.c_int64(sb), C.c_int64(sl), K_max, C.c_float(tau), eos_id,
        _ptr(out.cand_id), _ptr(out.cand_logit), _ptr(out.cand_logp), _ptr(out.cand_count),
        _ptr(out.lse), _ptr(out.lse64), _ptr(out.entropy), _ptr(out.gen_len), _ptr(out.row_status),
        _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def dsp_lattice_build_static(draft: torch.Tensor, K_max: int, tau: float = 0.0, eos_id: int = -1,
                             out: Optional[SimpleNamespace] = None, stream=None) -> SimpleNamespace:
    """``dsp_lattice_build`` with the scratch held inside the library: for callers that cannot
    allocate device memory.  Nothing is allocated by the C call; pass ``out`` to keep this wrapper
    from allocating the outputs.  Raises DspError(DSP_ERR_STATIC_SCRATCH) beyond the size limit."""
    B, L, V, sb, sl = _logits3(draft, "draft")
    dt = _dtype(draft)
    if out is None:
        out = lattice_outputs(B, L, K_max, eos_id, draft.device)
    _check("dsp_lattice_build_static", lib().dsp_lattice_build_static(
        _ptr(draft), dt, B, L, V, C.c_int64(sb), C.c_int64(sl), K_max, C.c_float(tau), eos_id,
        _ptr(out.cand_id), _ptr(out.cand_logit), _ptr(out.cand_logp), _ptr(out.cand_count),
        _ptr(out.lse), _ptr(out.lse64), _ptr(out.entropy), _ptr(out.gen_len), _ptr(out.row_status),
        _stream(stream)))
    return out


def cps_outputs(B: int, L: int, W: int, device, beams: bool = True) -> SimpleNamespace:
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=device)
    return SimpleNamespace(
        path=e((B, L), torch.int32), path_slot=e((B, L), torch.int32), path_len=e((B,), torch.int32),
        path_score=e((B,), torch.float32),
        beam_ids=e((B, W, L), torch.int32) if beams else None,
        beam_score=e((B, W), torch.float32) if beams else None,
        beam_cum=e((B, W), torch.float32) if beams else None)


def dsp_cps_search(lat: SimpleNamespace, prev_token: torch.Tensor, table: torch.Tensor, *, W: int,
                   lam: float, eos_id: int = -1, proxy_kind: int = 0, table_log2: int = 0,
                   hash_seed: int = 0, V: int = 1, out: Optional[SimpleNamespace] = None,
                   row_status: Optional[torch.Tensor] = None, beams: bool = True,
                   stream=None) -> SimpleNamespace:
    B, L, KC = lat.cand_id.shape
    if out is None:
        out = cps_outputs(B, L, W, lat.cand_id.device, beams)
    _check("dsp_cps_search", lib().dsp_cps_search(
        _ptr(lat.cand_id), _ptr(lat.cand_logit), _ptr(lat.lse64), _ptr(lat.cand_count), B, L, KC,
        _ptr(prev_token), proxy_kind, _ptr(table), table_log2, C.c_uint32(hash_seed & 0xFFFFFFFF), V,
        W, C.c_float(lam), eos_id, _ptr(out.path), _ptr(out.path_slot), _ptr(out.path_len),
        _ptr(out.path_score), _ptr(out.beam_ids), _ptr(out.beam_score), _ptr(out.beam_cum),
        _ptr(row_status), _stream(stream)))
    return out


def dsp_cps_search_biased(lat: SimpleNamespace, prev_token: torch.Tensor, table: torch.Tensor, *, W: int,
                          lam: float, ver_score: Optional[torch.Tensor], mu: float, eos_id: int = -1,
                          proxy_kind: int = 0, table_log2: int = 0, hash_seed: int = 0, V: int = 1,
                          out: Optional[SimpleNamespace] = None, row_status: Optional[torch.Tensor] = None,
                          beams: bool = True, stream=None) -> SimpleNamespace:
    B, L, KC = lat.cand_id.shape
    if ver_score is not None and (ver_score.dtype != torch.float32 or tuple(ver_score.shape) != (B, L, KC)
                                  or not ver_score.is_contiguous()):
        raise ValueError("ver_score must be a contiguous float32 [B, L, KC] tensor")
    if out is None:
        out = cps_outputs(B, L, W, lat.cand_id.device, beams)
    _check("dsp_cps_search_biased", lib().dsp_cps_search_biased(
        _ptr(lat.cand_id), _ptr(lat.cand_logit), _ptr(lat.lse64), _ptr(lat.cand_count), B, L, KC,
        _ptr(prev_token), proxy_kind, _ptr(table), table_log2, C.c_uint32(hash_seed & 0xFFFFFFFF), V,
        W, C.c_float(lam), eos_id, _ptr(ver_score), C.c_float(mu), _ptr(out.path), _ptr(out.path_slot),
        _ptr(out.path_len), _ptr(out.path_score), _ptr(out.beam_ids), _ptr(out.beam_score),
        _ptr(out.beam_cum), _ptr(row_status), _stream(stream)))
    return out


def verify_outputs(B: int, L: int, Lt: int, device) -> SimpleNamespace:
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=device)
    return SimpleNamespace(
        accepted_len=e((B,), torch.int32), next_token=e((B,), torch.int32),
        ratio=e((B, L), torch.float32), tgt_argmax=e((B, Lt), torch.int32),
        tgt_lse=e((B, Lt), torch.float32))


def dsp_verify(target: torch.Tensor, draft: Optional[torch.Tensor], cps: SimpleNamespace,
               lat: Optional[SimpleNamespace], *, mode: Optional[torch.Tensor] = None,
               u: Optional[torch.Tensor] = None, eos_id: int = -1, all_greedy: bool = False,
               row_status: torch.Tensor, out: Optional[SimpleNamespace] = None,
               workspace: Optional[torch.Tensor] = None, stream=None) -> SimpleNamespace:
    B, Lt, V, tsb, tsl = _logits3(target, "target")
    L = cps.path.shape[1]
    dt = _dtype(target)
    dsb = dsl = 0
    if draft is not None:
        Bd, Ld, Vd, dsb, dsl = _logits3(draft, "draft")
        if (Bd, Ld, Vd) != (B, L, V) or draft.dtype != target.dtype:
            raise ValueError("draft must be [B, L, V] with the target's dtype")
    if out is None:
        out = verify_outputs(B, L, Lt, target.device)
    if workspace is None:
        workspace = alloc_workspace(dsp_verify_workspace_bytes(B, L, Lt, V, dt), target.device)
    KC = lat.cand_logit.shape[2] if lat is not None else 1
    _check("dsp_verify", lib().dsp_verify(
        _ptr(target), dt, B, L, Lt, V, C.c_int64(tsb), C.c_int64(tsl),
        _ptr(draft), C.c_int64(dsb), C.c_int64(dsl),
        _ptr(cps.path), _ptr(cps.path_slot), _ptr(cps.path_len),
        _ptr(lat.cand_logit if lat is not None else None),
        _ptr(lat.lse64 if lat is not None else None), KC,
        1 if all_greedy else 0, _ptr(mode), _ptr(u), eos_id,
        _ptr(out.accepted_len), _ptr(out.next_token), _ptr(out.ratio), _ptr(out.tgt_argmax),
        _ptr(out.tgt_lse), _ptr(row_status), _ptr(workspace), C.c_size_t(workspace.numel()),
        _stream(stream)))
    return out


def _step_call(draft, target, prev_token, table, K_max, W, lam, tau, eos_id, proxy_kind, table_log2, hash_seed,
               mode, u, all_greedy, lat, cps, ver, lattice_workspace, verify_workspace):
    """Buffers (made where not given) and the argument list shared by the step and its graph."""
    B, L, V, dsb, dsl = _logits3(draft, "draft")
    Bt, Lt, Vt, tsb, tsl = _logits3(target, "target")
    if (Bt, Vt) != (B, V) or target.dtype != draft.dtype:
        raise ValueError("target must be [B, Lt, V] with the draft's dtype")
    dt = _dtype(draft)
    dev = draft.device
    lat = lattice_outputs(B, L, K_max, eos_id, dev) if lat is None else lat
    cps = cps_outputs(B, L, W, dev, True) if cps is None else cps
    ver = verify_outputs(B, L, Lt, dev) if ver is None else ver
    if lattice_workspace is None:
        lattice_workspace = alloc_workspace(dsp_lattice_workspace_bytes(B, L, V, dt, K_max), dev)
    if verify_workspace is None:
        verify_workspace = alloc_workspace(dsp_verify_workspace_bytes(B, L, Lt, V, dt), dev)
    args = (
        _ptr(draft), _ptr(target), dt, B, L, Lt, V, C.c_int64(dsb), C.c_int64(dsl), C.c_int64(tsb),
        C.c_int64(tsl), K_max, C.c_float(tau), eos_id, _ptr(prev_token), proxy_kind, _ptr(table), table_log2,
        C.c_uint32(hash_seed & 0xFFFFFFFF), W, C.c_float(lam), 1 if all_greedy else 0, _ptr(mode), _ptr(u),
        _ptr(lat.cand_id), _ptr(lat.cand_logit), _ptr(lat.cand_logp), _ptr(lat.cand_count), _ptr(lat.lse),
        _ptr(lat.lse64), _ptr(lat.entropy), _ptr(lat.gen_len),
        _ptr(cps.path), _ptr(cps.path_slot), _ptr(cps.path_len), _ptr(cps.path_score), _ptr(cps.beam_ids),
        _ptr(cps.beam_score), _ptr(cps.beam_cum),
        _ptr(ver.accepted_len), _ptr(ver.next_token), _ptr(ver.ratio), _ptr(ver.tgt_argmax), _ptr(ver.tgt_lse),
        _ptr(lat.row_status), _ptr(lattice_workspace), C.c_size_t(lattice_workspace.numel()),
        _ptr(verify_workspace), C.c_size_t(verify_workspace.numel()))
    keep = (draft, target, prev_token, table, mode, u, lattice_workspace, verify_workspace)
    return args, lat, cps, ver, keep


def dsp_draft_verify_step(draft: torch.Tensor, target: torch.Tensor, prev_token: torch.Tensor,
                          table: torch.Tensor, *, K_max: int, W: int, lam: float, tau: float = 0.0,
                          eos_id: int = -1, proxy_kind: int = 0, table_log2: int = 0, hash_seed: int = 0,
                          mode: Optional[torch.Tensor] = None, u: Optional[torch.Tensor] = None,
                          all_greedy: bool = False, lat: Optional[SimpleNamespace] = None,
                          cps: Optional[SimpleNamespace] = None, ver: Optional[SimpleNamespace] = None,
                          lattice_workspace: Optional[torch.Tensor] = None,
                          verify_workspace: Optional[torch.Tensor] = None, stream=None):
    """The three device calls of a step in one (same results); returns (lat, cps, ver)."""
    args, lat, cps, ver, _ = _step_call(draft, target, prev_token, table, K_max, W, lam, tau, eos_id, proxy_kind,
                                        table_log2, hash_seed, mode, u, all_greedy, lat, cps, ver,
                                        lattice_workspace, verify_workspace)
    _check("dsp_draft_verify_step", lib().dsp_draft_verify_step(*args, _stream(stream)))
    return lat, cps, ver


class StepGraph:
    """Handle of dsp_step_graph_create: ``launch()`` replays the recorded step; ``lat``, ``cps``,
    ``ver`` are its output buffers.  Holds references to every buffer the graph points at."""

    def __init__(self, handle, lat, cps, ver, keep):
        self._h, self.lat, self.cps, self.ver, self._keep = handle, lat, cps, ver, keep

    def launch(self, stream=None):
        _check("dsp_step_graph_launch", lib().dsp_step_graph_launch(self._h, _stream(stream)))

    def destroy(self):
        if self._h is not None:
            h, self._h = self._h, None
            _check("dsp_step_graph_destroy", lib().dsp_step_graph_destroy(h))

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def dsp_step_graph_create(draft: torch.Tensor, target: torch.Tensor, prev_token: torch.Tensor,
                          table: torch.Tensor, *, K_max: int, W: int, lam: float, tau: float = 0.0,
                          eos_id: int = -1, proxy_kind: int = 0, table_log2: int = 0, hash_seed: int = 0,
                          mode: Optional[torch.Tensor] = None, u: Optional[torch.Tensor] = None,
                          all_greedy: bool = False, lat: Optional[SimpleNamespace] = None,
                          cps: Optional[SimpleNamespace] = None, ver: Optional[SimpleNamespace] = None,
                          lattice_workspace: Optional[torch.Tensor] = None,
                          verify_workspace: Optional[torch.Tensor] = None) -> StepGraph:
    """Record dsp_draft_verify_step on these buffers as a CUDA graph (nothing runs yet)."""
    args, lat, cps, ver, keep = _step_call(draft, target, prev_token, table, K_max, W, lam, tau, eos_id,
                                           proxy_kind, table_log2, hash_seed, mode, u, all_greedy, lat, cps, ver,
                                           lattice_workspace, verify_workspace)
    h = C.c_void_p(0)
    _check("dsp_step_graph_create", lib().dsp_step_graph_create(C.byref(h), *args))
    return StepGraph(h, lat, cps, ver, keep)


SHARD_SUMS_BYTES = 24      # sizeof(dsp_shard_sums)


def dsp_shard_workspace_bytes(B: int, L: int, Vs: int, dtype: int, K_max: int) -> int:
    n = C.c_size_t(0)
    _check("dsp_shard_workspace_bytes", lib().dsp_shard_workspace_bytes(B, L, Vs, dtype, K_max, C.byref(n)))
    return n.value


def dsp_lattice_shard(logits: torch.Tensor, vocab_offset: int, K_max: int, eos_id: int = -1, *,
                      out: Optional[SimpleNamespace] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> SimpleNamespace:
    """Records of one vocabulary slice [B,L,Vs]: sums (uint8 [B,L,24], raw dsp_shard_sums), keys
    (int64 [B,L,K_max], raw 64-bit keys), status (int32 [B])."""
    B, L, Vs, sb, sl = _logits3(logits, "logits")
    dev = logits.device
    if out is None:
        out = SimpleNamespace(sums=torch.empty((B, L, SHARD_SUMS_BYTES), dtype=torch.uint8, device=dev),
                              keys=torch.empty((B, L, K_max), dtype=torch.int64, device=dev),
                              status=torch.empty((B,), dtype=torch.int32, device=dev))
    dt = _dtype(logits)
    if workspace is None:
        workspace = alloc_workspace(dsp_shard_workspace_bytes(B, L, Vs, dt, K_max), dev)
    _check("dsp_lattice_shard", lib().dsp_lattice_shard(
        _ptr(logits), dt, B, L, Vs, C.c_int64(sb), C.c_int64(sl), int(vocab_offset), K_max, eos_id,
        _ptr(out.sums), _ptr(out.keys), _ptr(out.status), _ptr(workspace), C.c_size_t(workspace.numel()),
        _stream(stream)))
    return out


def dsp_lattice_merge(sums: torch.Tensor, keys: torch.Tensor, status: torch.Tensor, V: int, K_max: int,
                      tau: float = 0.0, eos_id: int = -1, *, out: Optional[SimpleNamespace] = None,
                      workspace: Optional[torch.Tensor] = None, stream=None) -> SimpleNamespace:
    """Finish the lattice from the gathered records of all G slices: sums [G,B,L,24] uint8, keys
    [G,B,L,K_max] int64, status [G,B] int32 (slice-major, contiguous).  Same outputs as dsp_lattice_build."""
    G, B, L = sums.shape[0], sums.shape[1], sums.shape[2]
    dev = sums.device
    if (tuple(sums.shape) != (G, B, L, SHARD_SUMS_BYTES) or tuple(keys.shape) != (G, B, L, K_max)
            or tuple(status.shape) != (G, B) or not (sums.is_contiguous() and keys.is_contiguous()
                                                    and status.is_contiguous())):
        raise ValueError("records must be contiguous [G,B,L,24] / [G,B,L,K_max] / [G,B] tensors")
    if out is None:
        out = lattice_outputs(B, L, K_max, eos_id, dev)
    n = C.c_size_t(0)
    _check("dsp_merge_workspace_bytes", lib().dsp_merge_workspace_bytes(B, C.byref(n)))
    if workspace is None:
        workspace = alloc_workspace(n.value, dev)
    _check("dsp_lattice_merge", lib().dsp_lattice_merge(
        G, _ptr(sums), _ptr(keys), _ptr(status), B, L, int(V), K_max, C.c_float(tau), eos_id,
        _ptr(out.cand_id), _ptr(out.cand_logit), _ptr(out.cand_logp), _ptr(out.cand_count), _ptr(out.lse),
        _ptr(out.lse64), _ptr(out.entropy), _ptr(out.gen_len), _ptr(out.row_status), _ptr(workspace),
        C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def dsp_target_shard(logits: torch.Tensor, vocab_offset: int, cps: SimpleNamespace, *,
                     out: Optional[SimpleNamespace] = None, workspace: Optional[torch.Tensor] = None,
                     stream=None) -> SimpleNamespace:
    """Records of one vocabulary slice [B,Lt,Vs] of the target logits for the path in ``cps``."""
    B, Lt, Vs, sb, sl = _logits3(logits, "logits")
    L = cps.path.shape[1]
    dev = logits.device
    if out is None:
        out = SimpleNamespace(sums=torch.empty((B, Lt, SHARD_SUMS_BYTES), dtype=torch.uint8, device=dev),
                              keys=torch.empty((B, Lt, 1), dtype=torch.int64, device=dev),
                              status=torch.empty((B,), dtype=torch.int32, device=dev))
    dt = _dtype(logits)
    if workspace is None:
        workspace = alloc_workspace(dsp_shard_workspace_bytes(B, Lt, Vs, dt, 1), dev)
    _check("dsp_target_shard", lib().dsp_target_shard(
        _ptr(logits), dt, B, L, Lt, Vs, C.c_int64(sb), C.c_int64(sl), int(vocab_offset), _ptr(cps.path),
        _ptr(cps.path_len), _ptr(out.sums), _ptr(out.keys), _ptr(out.status), _ptr(workspace),
        C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def dsp_verify_merge(sums: torch.Tensor, keys: torch.Tensor, status: torch.Tensor, cps: SimpleNamespace,
                     lat: Optional[SimpleNamespace], *, mode: Optional[torch.Tensor] = None,
                     u: Optional[torch.Tensor] = None, eos_id: int = -1, all_greedy: bool = False,
                     row_status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                     stream=None) -> SimpleNamespace:
    """Verification from the gathered target records ([G,B,Lt,24] / [G,B,Lt,1] / [G,B]); returns
    dsp_verify's outputs plus tgt_lse64, job_trow, job_drow (see include/dsp.h)."""
    G, B, Lt = sums.shape[0], sums.shape[1], sums.shape[2]
    L = cps.path.shape[1]
    dev = sums.device
    out = verify_outputs(B, L, Lt, dev)
    e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
    out.tgt_lse64, out.job_trow, out.job_drow = e((B, Lt), torch.float64), e((B,), torch.int32), e((B,), torch.int32)
    out.row_status = torch.zeros((B,), dtype=torch.int32, device=dev) if row_status is None else row_status
    n = C.c_size_t(0)
    _check("dsp_verify_merge_workspace_bytes", lib().dsp_verify_merge_workspace_bytes(B, Lt, C.byref(n)))
    if workspace is None:
        workspace = alloc_workspace(n.value, dev)
    KC = 1 if lat is None else lat.cand_logit.shape[2]
    _check("dsp_verify_merge", lib().dsp_verify_merge(
        G, _ptr(sums.contiguous()), _ptr(keys.contiguous()), _ptr(status.contiguous()), B, L, Lt,
        _ptr(cps.path), _ptr(cps.path_slot), _ptr(cps.path_len),
        _ptr(None if lat is None else lat.cand_logit), _ptr(None if lat is None else lat.lse64), KC,
        1 if all_greedy else 0, _ptr(mode), _ptr(u), eos_id, _ptr(out.accepted_len), _ptr(out.next_token),
        _ptr(out.ratio), _ptr(out.tgt_argmax), _ptr(out.tgt_lse), _ptr(out.tgt_lse64), _ptr(out.job_trow),
        _ptr(out.job_drow), _ptr(out.row_status), _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def dsp_residual_sample(target_rows: torch.Tensor, draft_rows: torch.Tensor, ver: SimpleNamespace,
                        lat: SimpleNamespace, u: torch.Tensor, L: int, *,
                        workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """Draw the pending tokens of ``ver`` (from dsp_verify_merge) from the gathered whole rows
    [B,V]; ``ver.next_token`` and ``ver.row_status`` are updated in place."""
    B, V = target_rows.shape
    Lt = ver.tgt_argmax.shape[1]
    if target_rows.stride(1) != 1 or draft_rows.stride(1) != 1 or tuple(draft_rows.shape) != (B, V):
        raise ValueError("target_rows / draft_rows must be [B, V] with a contiguous vocabulary dimension")
    dt = _dtype(target_rows)
    n = C.c_size_t(0)
    _check("dsp_residual_sample_workspace_bytes", lib().dsp_residual_sample_workspace_bytes(B, V, dt, C.byref(n)))
    if workspace is None:
        workspace = alloc_workspace(n.value, target_rows.device)
    _check("dsp_residual_sample", lib().dsp_residual_sample(
        _ptr(target_rows), _ptr(draft_rows), dt, B, L, Lt, V, C.c_int64(target_rows.stride(0)),
        C.c_int64(draft_rows.stride(0)), _ptr(ver.job_trow), _ptr(ver.job_drow), _ptr(ver.tgt_lse64),
        _ptr(lat.lse64), _ptr(ver.tgt_argmax), _ptr(u), _ptr(ver.next_token), _ptr(ver.row_status),
        _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)))


def dsp_beam_tree(cps: SimpleNamespace, stream=None) -> SimpleNamespace:
    """Token tree of the beams in ``cps`` (beam_ids [B,W,L], path_len [B])."""
    B, W, L = cps.beam_ids.shape
    dev = cps.beam_ids.device
    e = lambda shape: torch.empty(shape, dtype=torch.int32, device=dev)
    out = SimpleNamespace(node_token=e((B, W * L)), node_parent=e((B, W * L)), node_depth=e((B, W * L)),
                          beam_node=e((B, W, L)), n_nodes=e((B,)))
    _check("dsp_beam_tree", lib().dsp_beam_tree(
        _ptr(cps.beam_ids), _ptr(cps.path_len), B, W, L, _ptr(out.node_token), _ptr(out.node_parent),
        _ptr(out.node_depth), _ptr(out.beam_node), _ptr(out.n_nodes), _stream(stream)))
    return out


def dsp_verify_tree(target: torch.Tensor, tree: SimpleNamespace, L: int, *,
                    workspace: Optional[torch.Tensor] = None, stream=None) -> SimpleNamespace:
    """Greedy verification of the token tree; ``target`` is [B, 1 + N, V]."""
    B, N1, V, sb, sl = _logits3(target, "target")
    N = N1 - 1
    if tuple(tree.node_token.shape) != (B, N):
        raise ValueError("target must have one row per node slot plus one")
    dev = target.device
    dt = _dtype(target)
    e = lambda shape: torch.empty(shape, dtype=torch.int32, device=dev)
    out = SimpleNamespace(accepted_len=e((B,)), accepted_node=e((B, L)), next_token=e((B,)),
                          tgt_argmax=e((B, N1)), row_status=e((B,)))
    n = C.c_size_t(0)
    _check("dsp_verify_tree_workspace_bytes", lib().dsp_verify_tree_workspace_bytes(B, N, V, dt, C.byref(n)))
    if workspace is None:
        workspace = alloc_workspace(n.value, dev)
    _check("dsp_verify_tree", lib().dsp_verify_tree(
        _ptr(target), dt, B, N, V, C.c_int64(sb), C.c_int64(sl), _ptr(tree.node_token), _ptr(tree.node_parent),
        _ptr(tree.n_nodes), L, _ptr(out.accepted_len), _ptr(out.accepted_node), _ptr(out.next_token),
        _ptr(out.tgt_argmax), _ptr(out.row_status), _ptr(workspace), C.c_size_t(workspace.numel()),
        _stream(stream)))
    return out


def dsp_verify_tree_stochastic(target: torch.Tensor, draft: torch.Tensor, tree: SimpleNamespace, u: torch.Tensor, *,
                               workspace: Optional[torch.Tensor] = None, stream=None) -> SimpleNamespace:
    """Stochastic verification of the token tree; ``target`` [B, 1 + N, V], ``draft`` [B, L, V], ``u`` fp32 [B, N + 1]."""
    B, N1, V, tsb, tsl = _logits3(target, "target")
    Bd, L, Vd, dsb, dsl = _logits3(draft, "draft")
    N = N1 - 1
    if tuple(tree.node_token.shape) != (B, N) or (Bd, Vd) != (B, V) or draft.dtype != target.dtype:
        raise ValueError("target must have one row per node slot plus one, draft the same batch, vocabulary and dtype")
    if u.dtype != torch.float32 or tuple(u.shape) != (B, N + 1) or not u.is_contiguous() or u.device != target.device:
        raise ValueError("u must be a contiguous fp32 [B, N + 1] tensor on the logits' device")
    dev = target.device
    dt = _dtype(target)
    e = lambda shape: torch.empty(shape, dtype=torch.int32, device=dev)
    out = SimpleNamespace(accepted_len=e((B,)), accepted_node=e((B, L)), next_token=e((B,)),
                          tgt_argmax=e((B, N1)), row_status=e((B,)))
    n = C.c_size_t(0)
    _check("dsp_verify_tree_workspace_bytes", lib().dsp_verify_tree_workspace_bytes(B, N, V, dt, C.byref(n)))
    if workspace is None:
        workspace = alloc_workspace(n.value, dev)
    _check("dsp_verify_tree_stochastic", lib().dsp_verify_tree_stochastic(
        _ptr(target), _ptr(draft), dt, B, N, L, V, C.c_int64(tsb), C.c_int64(tsl), C.c_int64(dsb), C.c_int64(dsl),
        _ptr(tree.node_token), _ptr(tree.node_parent), _ptr(tree.n_nodes), _ptr(u),
        _ptr(out.accepted_len), _ptr(out.accepted_node), _ptr(out.next_token), _ptr(out.tgt_argmax),
        _ptr(out.row_status), _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def gather_shard_records(rec: SimpleNamespace, group=None) -> SimpleNamespace:
    """All-gather one rank's slice records into the slice-major buffers dsp_lattice_merge reads
    (rank r holds slice r).  Plain torch.distributed collectives on the records' device."""
    import torch.distributed as dist
    G = dist.get_world_size(group)
    out = SimpleNamespace()
    for name in ("sums", "keys", "status"):
        t = getattr(rec, name).contiguous()
        parts = [torch.empty_like(t) for _ in range(G)]
        dist.all_gather(parts, t, group=group)
        setattr(out, name, torch.stack(parts, dim=0).contiguous())
    return out


def dsp_unmask_workspace_bytes(B: int, L: int, V: int, dtype: int) -> int:
    n = C.c_size_t(0)
    _check("dsp_unmask_workspace_bytes", lib().dsp_unmask_workspace_bytes(B, L, V, dtype, C.byref(n)))
    return n.value


def dsp_unmask_step(logits: torch.Tensor, tokens: torch.Tensor, masked: torch.Tensor, n_update: int, *,
                    out: Optional[SimpleNamespace] = None, workspace: Optional[torch.Tensor] = None,
                    stream=None) -> SimpleNamespace:
    """One refinement step of the drafter: ``tokens`` (int32 [B,L]) and ``masked`` (uint8 [B,L]) are
    updated in place; returns argmax, confidence, n_left, row_status."""
    B, L, V, sb, sl = _logits3(logits, "logits")
    dev = logits.device
    for t, dt in ((tokens, torch.int32), (masked, torch.uint8)):
        if t.dtype != dt or tuple(t.shape) != (B, L) or not t.is_contiguous() or t.device != dev:
            raise ValueError("tokens / masked must be contiguous [B, L] int32 / uint8 tensors on the logits' device")
    if out is None:
        e = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
        out = SimpleNamespace(argmax=e((B, L), torch.int32), confidence=e((B, L), torch.float32),
                              n_left=e((B,), torch.int32), row_status=e((B,), torch.int32))
    dt = _dtype(logits)
    if workspace is None:
        workspace = alloc_workspace(dsp_unmask_workspace_bytes(B, L, V, dt), dev)
    _check("dsp_unmask_step", lib().dsp_unmask_step(
        _ptr(logits), dt, B, L, V, C.c_int64(sb), C.c_int64(sl), int(n_update), _ptr(tokens), _ptr(masked),
        _ptr(out.argmax), _ptr(out.confidence), _ptr(out.n_left), _ptr(out.row_status), _ptr(workspace),
        C.c_size_t(workspace.numel()), _stream(stream)))
    return out


def dsp_adl_init(k_min=20, k_max=30, delta=10.0, rho=0.5, granularity=1):
    """Returns (state, params) for dsp_adl_update; the paper's defaults (Sec. 4)."""
    p = AdlParams(int(k_min), int(k_max), float(delta), float(rho), int(granularity))
    st = AdlState()
    _check("dsp_adl_init", lib().dsp_adl_init(C.byref(st), C.byref(p)))
    return st, p


def dsp_adl_update(state: AdlState, params: AdlParams, accepted_len, gen_len) -> int:
    """accepted_len / gen_len: host int32 tensors or sequences of equal length B."""
    a = torch.as_tensor(accepted_len, dtype=torch.int32, device="cpu").contiguous().view(-1)
    g = torch.as_tensor(gen_len, dtype=torch.int32, device="cpu").contiguous().view(-1)
    if a.numel() != g.numel():
        raise ValueError("accepted_len and gen_len must have the same length")
    nxt = C.c_int32(0)
    _check("dsp_adl_update", lib().dsp_adl_update(
        C.byref(state), C.byref(params), C.c_void_p(a.data_ptr()), C.c_void_p(g.data_ptr()),
        a.numel(), C.byref(nxt)))
    return nxt.value


class BreadthParams(C.Structure):
    _fields_ = [("K_min", C.c_int32), ("K_max", C.c_int32), ("W_min", C.c_int32), ("W_max", C.c_int32),
                ("rho", C.c_double)]


class BreadthState(C.Structure):
    _fields_ = [("ema_entropy", C.c_double), ("ema_shortfall", C.c_double), ("K", C.c_int32), ("W", C.c_int32),
                ("steps", C.c_int32)]


def dsp_breadth_init(K_min=1, K_max=16, W_min=1, W_max=16, rho=0.5):
    """Returns (state, params) for dsp_breadth_update."""
    p = BreadthParams(int(K_min), int(K_max), int(W_min), int(W_max), float(rho))
    st = BreadthState()
    _check("dsp_breadth_init", lib().dsp_breadth_init(C.byref(st), C.byref(p)))
    return st, p


def dsp_breadth_update(state: BreadthState, params: BreadthParams, entropy, accepted_len, gen_len):
    """entropy: host float32 [B,L]; accepted_len / gen_len: host int32 [B].  Returns (K, W) for the next step."""
    e = torch.as_tensor(entropy, dtype=torch.float32, device="cpu").contiguous()
    a = torch.as_tensor(accepted_len, dtype=torch.int32, device="cpu").contiguous().view(-1)
    g = torch.as_tensor(gen_len, dtype=torch.int32, device="cpu").contiguous().view(-1)
    if e.dim() != 2 or a.numel() != e.shape[0] or g.numel() != e.shape[0]:
        raise ValueError("entropy must be [B, L] and the two lengths [B]")
    K, W = C.c_int32(0), C.c_int32(0)
    _check("dsp_breadth_update", lib().dsp_breadth_update(
        C.byref(state), C.byref(params), C.c_void_p(e.data_ptr()), C.c_void_p(a.data_ptr()), C.c_void_p(g.data_ptr()),
        e.shape[0], e.shape[1], C.byref(K), C.byref(W)))
    return K.value, W.value
