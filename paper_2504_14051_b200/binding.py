"""ctypes binding of libcaote.so: argument marshalling only, every step runs in the CUDA kernels.

The functions mirror the C entry points one to one and take torch tensors (device memory) in place
of raw pointers. There is no CPU fallback: if the library is missing it is built with nvcc, and if
that fails the import raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

BF16, F32 = 0, 1
BASE_MODES = {"last_query": 0, "chunk_sum": 1, "accum": 2, "external": 3}
COMPACT_MODES = {"fill": 0, "stable": 1}

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_LENGTH, ERR_OVERFLOW = 0, -1, -2, -3, -4, -5, -6
ERR_TOO_LARGE = -7
STATIC_SCRATCH_BYTES = 16 << 20


class Params(ctypes.Structure):
    """Mirror of caote_params_t."""

    _fields_ = [
        ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("capacity", ctypes.c_int32),
        ("n_new", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("scale", ctypes.c_float),
        ("base_mode", ctypes.c_int32),
        ("flags", ctypes.c_int32),
    ]


class TraceEntry(ctypes.Structure):
    """Mirror of caote_trace_entry_t."""

    _fields_ = [("name", ctypes.c_char * 48), ("launches", ctypes.c_int64), ("total_ms", ctypes.c_double)]


class CaoteError(RuntimeError):
    def __init__(self, fn: str, code: int):
        msg = lib().caote_status_string(code).decode()
        detail = lib().caote_last_cuda_error().decode()
        super().__init__(f"{fn}: {msg} ({code})" + (f": {detail}" if code == ERR_CUDA and detail else ""))
        self.code = code


_lib = None


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Load (building first if needed) the CUDA library; raises if it cannot be had."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    if not os.path.exists(path):
        raise ImportError(f"CAOTE CUDA library not found at {path}")
    L = ctypes.CDLL(path)
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
    pp = ctypes.POINTER(Params)
    L.caote_workspace_bytes.restype = sz
    L.caote_workspace_bytes.argtypes = [pp]
    L.caote_append.restype = ctypes.c_int
    L.caote_append.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.caote_score.restype = ctypes.c_int
    L.caote_score.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.caote_score_static.restype = ctypes.c_int
    L.caote_score_static.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.caote_select_evict.restype = ctypes.c_int
    L.caote_select_evict.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp]
    L.caote_compact.restype = ctypes.c_int
    L.caote_compact.argtypes = [pp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, sz, vp]
    L.caote_step.restype = ctypes.c_int
    L.caote_step.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, sz, vp]
    L.caote_vsum.restype = ctypes.c_int
    L.caote_vsum.argtypes = [pp, vp, vp, vp, vp]
    L.caote_score_fast.restype = ctypes.c_int
    L.caote_score_fast.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.caote_step_fast.restype = ctypes.c_int
    L.caote_step_fast.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, i32, vp, sz, vp]
    L.caote_score_sum_errors.restype = ctypes.c_int
    L.caote_score_sum_errors.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.caote_post_evict_output.restype = ctypes.c_int
    L.caote_post_evict_output.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp]
    L.caote_post_evict_output_ws.restype = ctypes.c_int
    L.caote_post_evict_output_ws.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    L.caote_read_status.restype = ctypes.c_int
    L.caote_read_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
    L.caote_status_string.restype = ctypes.c_char_p
    L.caote_status_string.argtypes = [ctypes.c_int]
    L.caote_last_cuda_error.restype = ctypes.c_char_p
    L.caote_last_cuda_error.argtypes = []
    L.caote_trace_enable.restype = ctypes.c_int
    L.caote_trace_enable.argtypes = [ctypes.c_int]
    L.caote_trace_collect.restype = ctypes.c_int
    L.caote_trace_collect.argtypes = [ctypes.POINTER(TraceEntry), i32, ctypes.POINTER(ctypes.c_int32)]
    L.caote_select_evict_greedy.restype = ctypes.c_int
    L.caote_select_evict_greedy.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp]
    L.caote_launch_count.restype = ctypes.c_int64
    L.caote_launch_count.argtypes = []
    L.caote_set_option.restype = ctypes.c_int
    L.caote_set_option.argtypes = [ctypes.c_int32, ctypes.c_int64]
    _lib = L
    return L


def make_params(batch, n_q_heads, n_kv_heads, head_dim, capacity, n_new, dtype, scale, base_mode) -> Params:
    if isinstance(dtype, torch.dtype):
        dtype = {torch.bfloat16: BF16, torch.float32: F32}[dtype]
    if isinstance(base_mode, str):
        base_mode = BASE_MODES[base_mode]
    return Params(batch, n_q_heads, n_kv_heads, head_dim, capacity, n_new, dtype, float(scale), base_mode, 0)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(fn: str, rc: int):
    if rc != 0:
        raise CaoteError(fn, rc)


def caote_workspace_bytes(p: Params) -> int:
    return int(lib().caote_workspace_bytes(ctypes.byref(p)))


def alloc_workspace(p: Params, device) -> torch.Tensor:
    """A zeroed uint8 workspace of the size the library asks for."""
    n = caote_workspace_bytes(p)
    if n == 0:
        raise CaoteError("caote_workspace_bytes", ERR_INVALID_ARG)
    return torch.zeros(n, dtype=torch.uint8, device=device)


def caote_append(p, K, V, base, pos, lens, n_seen, k_new, v_new, workspace, stream=None):
    _check("caote_append", lib().caote_append(ctypes.byref(p), _p(K), _p(V), _p(base), _p(pos), _p(lens),
                                              _p(n_seen), _p(k_new), _p(v_new), _p(workspace),
                                              workspace.numel(), _stream(stream)))


def caote_score(p, q, K, V, lens, base, o, scores, workspace, stream=None):
    _check("caote_score", lib().caote_score(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(base), _p(o),
                                            _p(scores), _p(workspace), workspace.numel(), _stream(stream)))


def caote_score_static(p, q, K, V, lens, base, o, scores, status_out=None, stream=None):
    """caote_score on the library's built-in scratch array: for callers that may not allocate device
    memory (no workspace argument). ``status_out``: optional int32 device tensor of one element."""
    _check("caote_score_static",
           lib().caote_score_static(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(base), _p(o), _p(scores),
                                    _p(status_out), _stream(stream)))


def caote_select_evict(p, scores, lens, budget, pos, evict_idx, n_evict, workspace, stream=None):
    _check("caote_select_evict",
           lib().caote_select_evict(ctypes.byref(p), _p(scores), _p(lens), _p(budget), _p(pos), _p(evict_idx),
                                    evict_idx.shape[-1], _p(n_evict), _p(workspace), workspace.numel(),
                                    _stream(stream)))


def caote_select_evict_greedy(p, V, h, lens, budget, pos, evict_idx, order, n_evict, workspace, stream=None):
    _check("caote_select_evict_greedy", lib().caote_select_evict_greedy(
        ctypes.byref(p), _p(V), _p(h), _p(lens), _p(budget), _p(pos), _p(evict_idx), _p(order), evict_idx.shape[-1],
        _p(n_evict), _p(workspace), workspace.numel() * workspace.element_size(), _stream(stream)))


def caote_compact(p, K, V, base, pos, lens, evict_idx, n_evict, mode, workspace, stream=None):
    if isinstance(mode, str):
        mode = COMPACT_MODES[mode]
    _check("caote_compact",
           lib().caote_compact(ctypes.byref(p), _p(K), _p(V), _p(base), _p(pos), _p(lens), _p(evict_idx),
                               evict_idx.shape[-1], _p(n_evict), mode, _p(workspace), workspace.numel(),
                               _stream(stream)))


def caote_step(p, q, k_new, v_new, K, V, base, pos, lens, n_seen, budget, o, scores, evict_idx, n_evict, mode,
               workspace, stream=None):
    if isinstance(mode, str):
        mode = COMPACT_MODES[mode]
    _check("caote_step",
           lib().caote_step(ctypes.byref(p), _p(q), _p(k_new), _p(v_new), _p(K), _p(V), _p(base), _p(pos),
                            _p(lens), _p(n_seen), _p(budget), _p(o), _p(scores), _p(evict_idx),
                            evict_idx.shape[-1], _p(n_evict), mode, _p(workspace), workspace.numel(),
                            _stream(stream)))


def caote_vsum(p, V, lens, vsum, stream=None):
    """vsum[u, :] = sum of the unit's valid V rows (FastCAOTE, Sec. 3.3)."""
    _check("caote_vsum", lib().caote_vsum(ctypes.byref(p), _p(V), _p(lens), _p(vsum), _stream(stream)))


def caote_score_fast(p, q, K, V, lens, base, vsum, o, scores, workspace, stream=None):
    _check("caote_score_fast",
           lib().caote_score_fast(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(base), _p(vsum), _p(o),
                                  _p(scores), _p(workspace), workspace.numel(), _stream(stream)))


def caote_step_fast(p, q, k_new, v_new, K, V, base, pos, lens, n_seen, budget, vsum, o, scores, evict_idx, n_evict,
                    mode, workspace, stream=None):
    if isinstance(mode, str):
        mode = COMPACT_MODES[mode]
    _check("caote_step_fast",
           lib().caote_step_fast(ctypes.byref(p), _p(q), _p(k_new), _p(v_new), _p(K), _p(V), _p(base), _p(pos),
                                 _p(lens), _p(n_seen), _p(budget), _p(vsum), _p(o), _p(scores), _p(evict_idx),
                                 evict_idx.shape[-1], _p(n_evict), mode, _p(workspace), workspace.numel(),
                                 _stream(stream)))


def caote_score_sum_errors(p, q, K, V, lens, o, scores, workspace, stream=None):
    """Scores as the sum over the counted query rows of the exact single-query eviction errors."""
    _check("caote_score_sum_errors",
           lib().caote_score_sum_errors(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(o), _p(scores),
                                        _p(workspace), workspace.numel(), _stream(stream)))


def caote_post_evict_output(p, q, K, V, lens, evict_idx, n_evict, o, o_post, stream=None):
    """Attention output over the retained tokens (call between caote_select_evict and caote_compact)."""
    _check("caote_post_evict_output",
           lib().caote_post_evict_output(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(evict_idx),
                                         evict_idx.shape[-1], _p(n_evict), _p(o), _p(o_post), _stream(stream)))


def caote_post_evict_output_ws(p, q, K, V, lens, evict_idx, n_evict, o, o_post, workspace, stream=None):
    """The same from the softmax statistics the scoring call left in `workspace`, where it left any."""
    _check("caote_post_evict_output_ws",
           lib().caote_post_evict_output_ws(ctypes.byref(p), _p(q), _p(K), _p(V), _p(lens), _p(evict_idx),
                                            evict_idx.shape[-1], _p(n_evict), _p(o), _p(o_post), _p(workspace),
                                            workspace.numel(), _stream(stream)))


def caote_read_status(workspace, stream=None) -> int:
    out = ctypes.c_int32(0)
    _check("caote_read_status", lib().caote_read_status(_p(workspace), _stream(stream), ctypes.byref(out)))
    return int(out.value)


def caote_status_string(code: int) -> str:
    return lib().caote_status_string(code).decode()


def caote_trace_enable(on: bool) -> None:
    _check("caote_trace_enable", lib().caote_trace_enable(1 if on else 0))


def caote_trace_collect(max_entries: int = 32) -> dict:
    """{kernel name: (launches, total_ms)} since the last collect."""
    buf = (TraceEntry * max_entries)()
    n = ctypes.c_int32(0)
    _check("caote_trace_collect", lib().caote_trace_collect(buf, max_entries, ctypes.byref(n)))
    return {buf[i].name.decode(): (int(buf[i].launches), float(buf[i].total_ms)) for i in range(n.value)}


OPT_WAIT_CYCLES, OPT_DECODE_CLUSTER, OPT_SIDE_BY_SIDE = 1, 2, 3


def caote_set_option(option: int, value: int) -> None:
    _check("caote_set_option", lib().caote_set_option(int(option), int(value)))


def caote_launch_count() -> int:
    return int(lib().caote_launch_count())
