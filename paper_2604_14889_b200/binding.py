"""Thin ctypes binding of libmemosight.so: same names as the C ABI, argument
marshalling only.  Every step of the path runs in the CUDA kernels behind the
library; there is no CPU fallback -- if the library is missing or a call fails,
an exception is raised.

Tensor arguments may be torch tensors (their ``data_ptr()`` is passed; they must
be contiguous and on the current CUDA device), ``None`` for an optional pointer,
or plain integers that already are addresses.  Host-side arrays are numpy arrays
or Python lists.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

MS_OK = 0
MS_ERR_INVALID_ARG = -1
MS_ERR_UNSUPPORTED_SHAPE = -2
MS_ERR_WORKSPACE_TOO_SMALL = -3
MS_ERR_ALIGNMENT = -4
MS_ERR_CUDA = -5
MS_ERR_DEVICE_TIMEOUT = -6

MS_ATTN_PATH_AUTO = 0
MS_ATTN_PATH_MMA_SYNC = 1
MS_ATTN_PATH_TCGEN05 = 2
MS_ATTN_PATH_GENERAL = 3
MS_ATTN_PATH_TCGEN05_KEYS = 4
MS_ATTN_PATH_LARGE_BLOCK = 5

MS_KIND_PROMPT, MS_KIND_REASON, MS_KIND_FORESIGHT, MS_KIND_MEMORY, MS_KIND_OUTPUT = 0, 1, 2, 3, 4

MS_ROPE_NEOX = 0
MS_ROPE_INTERLEAVED = 1
MS_POS_HALF_UNITS = 2
MS_LAYOUT_MONOTONE = 4


class MemosightError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().memosight_status_string(status).decode()
        extra = ""
        if status == MS_ERR_CUDA:
            extra = f" (cudaError {lib().memosight_last_cuda_error()})"
        super().__init__(f"{what}: {msg}{extra} [{status}]")


class AttnParams(C.Structure):
    """Mirror of ``memosight_attn_params`` (include/memosight.h)."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("kv_head_stride", C.c_int64), ("n_slots", C.c_int64),
        ("kv_off", C.c_void_p), ("kv_len", C.c_void_p),
        ("max_kv_len", C.c_int32), ("max_nq", C.c_int32),
        ("q_off", C.c_void_p), ("n_cand", C.c_void_p), ("anchor", C.c_void_p),
        ("total_rows", C.c_int32), ("sm_scale", C.c_float),
        ("q", C.c_void_p), ("k_step", C.c_void_p), ("v_step", C.c_void_p),
        ("out", C.c_void_p), ("lse", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("tok_kind", C.c_void_p), ("tok_step", C.c_void_p),
    ]


class AttnLayers(C.Structure):
    """Mirror of ``memosight_attn_layers`` (include/memosight.h)."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("kv_layer_stride", C.c_int64),
        ("q_layer_stride", C.c_int64), ("kstep_layer_stride", C.c_int64), ("out_layer_stride", C.c_int64),
        ("lse_layer_stride", C.c_int64),
    ]


class StepHostParams(C.Structure):
    """Mirror of ``memosight_step_host_params`` (include/memosight.h)."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("attn", AttnParams),
        ("h_q", C.c_void_p), ("h_k_step", C.c_void_p), ("h_v_step", C.c_void_p),
        ("h_pos_id", C.c_void_p), ("d_pos_id", C.c_void_p),
        ("rope_base", C.c_double), ("rope_flags", C.c_uint32), ("vocab", C.c_int32),
        ("h_logits", C.c_void_p), ("ld_v", C.c_int64), ("d_logits", C.c_void_p),
        ("h_draft", C.c_void_p), ("d_draft", C.c_void_p),
        ("d_argmax", C.c_void_p), ("d_n_match", C.c_void_p), ("d_n_keep", C.c_void_p),
        ("accept_workspace", C.c_void_p), ("accept_workspace_bytes", C.c_size_t),
        ("d_seg_start", C.c_void_p), ("d_seg_len", C.c_void_p), ("max_tail", C.c_int32),
        ("d_kv_cap", C.c_void_p),
        ("h_out", C.c_void_p), ("h_argmax", C.c_void_p), ("h_n_match", C.c_void_p),
    ]


class DecodeState(C.Structure):
    """Mirror of ``memosight_decode_state`` (include/memosight.h)."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("batch", C.c_int32), ("d", C.c_int32), ("c", C.c_int32),
        ("max_out", C.c_int32), ("max_mem", C.c_int32),
        ("tok_foresight", C.c_int32), ("tok_memory", C.c_int32), ("tok_output", C.c_int32),
        ("tok_delim", C.c_int32), ("tok_eos", C.c_int32),
        ("kv_len", C.c_void_p), ("pos_next", C.c_void_p), ("seg_start", C.c_void_p), ("seg_n", C.c_void_p),
        ("seg_pid0", C.c_void_p), ("cand", C.c_void_p), ("n_cand", C.c_void_p), ("flags", C.c_void_p),
        ("out_tok", C.c_void_p), ("n_out", C.c_void_p),
    ]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads (building first if a source is newer) the CUDA library; raises if impossible."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path) or _build.is_stale():
            path = _build.build()
        L = C.CDLL(path)
        L.memosight_status_string.restype = C.c_char_p
        L.memosight_status_string.argtypes = [C.c_int32]
        L.memosight_version.restype = C.c_int32
        L.memosight_last_cuda_error.restype = C.c_int32
        L.memosight_ama.restype = C.c_int32
        L.memosight_ama.argtypes = [C.c_int32, C.c_int32]
        L.memosight_upl_pids.restype = C.c_int32
        L.memosight_upl_pids.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_uint32, C.c_void_p, C.c_int32]
        L.memosight_out_pid.restype = C.c_int32
        L.memosight_out_pid.argtypes = [C.c_int32, C.c_int32]
        L.memosight_step_pids.restype = C.c_int32
        L.memosight_step_pids.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.memosight_rope_qk.restype = C.c_int32
        L.memosight_rope_qk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_double, C.c_void_p, C.c_uint32, C.c_void_p]
        L.memosight_attn_workspace_bytes.restype = C.c_size_t
        L.memosight_attn_workspace_bytes.argtypes = [C.c_int32] * 6
        L.memosight_attn_step.restype = C.c_int32
        L.memosight_attn_step.argtypes = [C.POINTER(AttnParams), C.c_void_p]
        L.memosight_attn_step_layers.restype = C.c_int32
        L.memosight_attn_step_layers.argtypes = [C.POINTER(AttnParams), C.POINTER(AttnLayers), C.c_void_p]
        L.memosight_attn_debug_events.restype = C.c_int32
        L.memosight_attn_debug_events.argtypes = [C.c_void_p, C.c_void_p]
        L.memosight_debug_set_wait_limit_us.restype = C.c_uint32
        L.memosight_debug_set_wait_limit_us.argtypes = [C.c_uint32]
        L.memosight_debug_set_bank_limit.restype = C.c_int32
        L.memosight_debug_set_bank_limit.argtypes = [C.c_int32]
        L.memosight_debug_wait_timeout.restype = C.c_int32
        L.memosight_debug_wait_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.memosight_attn_set_path.restype = C.c_int32
        L.memosight_attn_set_path.argtypes = [C.c_int32]
        L.memosight_attn_status.restype = C.c_int32
        L.memosight_attn_status.argtypes = [C.c_void_p, C.c_void_p]
        L.memosight_kv_compact.restype = C.c_int32
        L.memosight_kv_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int64, C.c_int32,
                                           C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.memosight_budget_pids.restype = C.c_int32
        L.memosight_budget_pids.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32]
        L.memosight_kv_gather.restype = C.c_int32
        L.memosight_kv_gather.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int64, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_int32, C.c_void_p]
        L.memosight_decode_scratch_bytes.restype = C.c_size_t
        L.memosight_decode_scratch_bytes.argtypes = [C.c_int32]
        L.memosight_decode_plan.restype = C.c_int32
        L.memosight_decode_plan.argtypes = [C.POINTER(DecodeState)] + [C.c_void_p] * 8
        L.memosight_decode_commit.restype = C.c_int32
        L.memosight_decode_commit.argtypes = [C.POINTER(DecodeState)] + [C.c_void_p] * 5
        L.memosight_decode_plan_compress.restype = C.c_int32
        L.memosight_decode_plan_compress.argtypes = [C.POINTER(DecodeState)] + [C.c_void_p] * 10
        L.memosight_decode_commit_compress.restype = C.c_int32
        L.memosight_decode_commit_compress.argtypes = [C.POINTER(DecodeState)] + [C.c_void_p] * 3
        L.memosight_kv_append.restype = C.c_int32
        L.memosight_kv_append.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                          C.c_void_p]
        L.memosight_accept_workspace_bytes.restype = C.c_size_t
        L.memosight_accept_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
        L.memosight_accept.restype = C.c_int32
        L.memosight_accept.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int32, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                       C.c_void_p]
        L.memosight_accept_static.restype = C.c_int32
        L.memosight_accept_static.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int32, C.c_int32,
                                              C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.memosight_step_host.restype = C.c_int32
        L.memosight_step_host.argtypes = [C.POINTER(StepHostParams), C.c_void_p]
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    """Address behind a tensor-like argument (marshalling only)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        if not t.is_contiguous():
            raise ValueError("memosight: tensors must be contiguous")
        return t.data_ptr()
    raise TypeError(f"memosight: cannot take the address of {type(t)!r}")


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(rc: int, what: str) -> None:
    if rc != MS_OK:
        raise MemosightError(rc, what)


# ------------------------------------------------------------------ host helpers

def memosight_version() -> int:
    return int(lib().memosight_version())


def memosight_ama(n: int, c: int) -> int:
    r = int(lib().memosight_ama(n, c))
    if r < 0:
        raise MemosightError(r, "memosight_ama")
    return r


def memosight_upl_pids(rho_first: int, n: int, c: int, flags: int = 0) -> np.ndarray:
    out = np.empty(max(n, 1), dtype=np.int32)
    r = int(lib().memosight_upl_pids(rho_first, n, c, flags, out.ctypes.data, out.size))
    if r < 0:
        raise MemosightError(r, "memosight_upl_pids")
    return out[:r].copy()


def memosight_budget_pids(rho_first: int, n: int, l: int) -> np.ndarray:
    out = np.empty(max(l, 1), dtype=np.int32)
    r = int(lib().memosight_budget_pids(rho_first, n, l, out.ctypes.data, out.size))
    if r < 0:
        raise MemosightError(r, "memosight_budget_pids")
    return out[:r].copy()


def memosight_out_pid(rho_first: int, n: int) -> int:
    return int(lib().memosight_out_pid(rho_first, n))


def memosight_step_pids(p0: int, n_c: int, d: int, anchor: Optional[Sequence[int]] = None) -> np.ndarray:
    out = np.empty(max(n_c + d, 1), dtype=np.int32)
    a = None if anchor is None else np.ascontiguousarray(anchor, dtype=np.int32)
    _check(int(lib().memosight_step_pids(p0, n_c, d, None if a is None else a.ctypes.data, out.ctypes.data)),
           "memosight_step_pids")
    return out[:n_c + d].copy()


# ------------------------------------------------------------------ device calls

def memosight_rope_qk(q, k, pos_id, T: int, H_q: int, H_kv: int, D: int, rope_base: float,
                      inv_freq=None, flags: int = 0, stream=None) -> None:
    f = None if inv_freq is None else np.ascontiguousarray(inv_freq, dtype=np.float64)
    _check(int(lib().memosight_rope_qk(_ptr(q), _ptr(k), _ptr(pos_id), T, H_q, H_kv, D, float(rope_base),
                                       None if f is None else f.ctypes.data, flags, _stream(stream))),
           "memosight_rope_qk")


def memosight_attn_workspace_bytes(batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                                   max_kv_len: int, max_nq: int) -> int:
    return int(lib().memosight_attn_workspace_bytes(batch, n_q_heads, n_kv_heads, head_dim, max_kv_len, max_nq))


def attn_params(*, batch, n_q_heads, n_kv_heads, head_dim, k_cache, v_cache, kv_head_stride, n_slots,
                kv_off, kv_len, max_kv_len, max_nq, q_off, n_cand, anchor, total_rows, sm_scale,
                q, k_step, v_step, out, lse, workspace, workspace_bytes, tok_kind=None,
                tok_step=None) -> AttnParams:
    """Fills a memosight_attn_params structure (addresses only; nothing is copied)."""
    p = AttnParams()
    p.struct_size = C.sizeof(AttnParams)
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = batch, n_q_heads, n_kv_heads, head_dim
    p.k_cache, p.v_cache = _ptr(k_cache), _ptr(v_cache)
    p.kv_head_stride, p.n_slots = kv_head_stride, n_slots
    p.kv_off, p.kv_len = _ptr(kv_off), _ptr(kv_len)
    p.max_kv_len, p.max_nq = max_kv_len, max_nq
    p.q_off, p.n_cand, p.anchor = _ptr(q_off), _ptr(n_cand), _ptr(anchor)
    p.total_rows, p.sm_scale = total_rows, float(sm_scale)
    p.q, p.k_step, p.v_step = _ptr(q), _ptr(k_step), _ptr(v_step)
    p.out, p.lse = _ptr(out), _ptr(lse)
    p.workspace, p.workspace_bytes = _ptr(workspace), workspace_bytes
    p.tok_kind, p.tok_step = _ptr(tok_kind), _ptr(tok_step)
    return p


def memosight_attn_step(params: Optional[AttnParams] = None, stream=None, **fields) -> None:
    """memosight_attn_step(params) or memosight_attn_step(**fields of attn_params)."""
    p = params if params is not None else attn_params(**fields)
    _check(int(lib().memosight_attn_step(C.byref(p), _stream(stream))), "memosight_attn_step")


def memosight_attn_step_layers(params: AttnParams, n_layers: int, kv_layer_stride: int, q_layer_stride: int,
                               kstep_layer_stride: int, out_layer_stride: int, lse_layer_stride: int = 0,
                               stream=None) -> None:
    """The attention of n_layers stacked layers that share the step's metadata (strides in elements)."""
    ly = AttnLayers()
    ly.struct_size = C.sizeof(AttnLayers)
    ly.n_layers = n_layers
    ly.kv_layer_stride, ly.q_layer_stride = kv_layer_stride, q_layer_stride
    ly.kstep_layer_stride, ly.out_layer_stride, ly.lse_layer_stride = kstep_layer_stride, out_layer_stride, lse_layer_stride
    _check(int(lib().memosight_attn_step_layers(C.byref(params), C.byref(ly), _stream(stream))),
           "memosight_attn_step_layers")


def memosight_attn_debug_events(ev_split_begin=None, ev_split_end=None) -> None:
    """Timing events (cudaEvent_t addresses) the calling thread's attention calls record around the
    split-KV kernel; (None, None) switches it off."""
    _check(int(lib().memosight_attn_debug_events(_ptr(ev_split_begin), _ptr(ev_split_end))),
           "memosight_attn_debug_events")


def memosight_step_host(params: StepHostParams, stream=None) -> None:
    _check(int(lib().memosight_step_host(C.byref(params), _stream(stream))), "memosight_step_host")


def memosight_attn_set_path(path: int) -> int:
    """Selects the attention kernel (MS_ATTN_PATH_*); returns the previous setting."""
    rc = int(lib().memosight_attn_set_path(int(path)))
    if rc < 0:
        raise MemosightError(rc, "memosight_attn_set_path")
    return rc


def memosight_debug_set_wait_limit_us(limit_us: int) -> int:
    """Limit of one bounded device-side wait for later launches; returns the previous one (0 only queries)."""
    return int(lib().memosight_debug_set_wait_limit_us(int(limit_us)))


def memosight_debug_set_bank_limit(n_banks: int) -> int:
    """Caps the last-block-done counter banks handed out (0: every call takes its two-launch form);
    returns the previous cap; negative only queries."""
    return int(lib().memosight_debug_set_bank_limit(int(n_banks)))


def memosight_debug_wait_timeout(workspace, limit_us: int, stream=None) -> None:
    """Queues the one-warp kernel whose bounded wait runs out after limit_us microseconds."""
    _check(int(lib().memosight_debug_wait_timeout(_ptr(workspace), int(limit_us), _stream(stream))),
           "memosight_debug_wait_timeout")


def memosight_attn_status(workspace, stream=None) -> int:
    """Synchronises the stream; returns MS_OK or MS_ERR_DEVICE_TIMEOUT (raises on CUDA errors)."""
    rc = int(lib().memosight_attn_status(_ptr(workspace), _stream(stream)))
    if rc not in (MS_OK, MS_ERR_DEVICE_TIMEOUT):
        raise MemosightError(rc, "memosight_attn_status")
    return rc


def memosight_kv_compact(k_cache, v_cache, n_layers, layer_stride, kv_head_stride, batch, n_kv_heads, head_dim,
                         kv_off, kv_len, seg_start, seg_len, src_idx, idx_stride, max_tail, stream=None) -> None:
    _check(int(lib().memosight_kv_compact(_ptr(k_cache), _ptr(v_cache), n_layers, layer_stride, kv_head_stride,
                                          batch, n_kv_heads, head_dim, _ptr(kv_off), _ptr(kv_len),
                                          _ptr(seg_start), _ptr(seg_len), _ptr(src_idx), idx_stride, max_tail,
                                          _stream(stream))), "memosight_kv_compact")


def decode_state(batch, d, c, max_out, max_mem, tok_foresight, tok_memory, tok_output, tok_delim, tok_eos,
                 kv_len, pos_next, seg_start, seg_n, seg_pid0, cand, n_cand, flags, out_tok, n_out) -> DecodeState:
    """Fills a ``memosight_decode_state`` from tensors / addresses."""
    st = DecodeState()
    st.struct_size = C.sizeof(DecodeState)
    st.batch, st.d, st.c, st.max_out, st.max_mem = batch, d, c, max_out, max_mem
    st.tok_foresight, st.tok_memory, st.tok_output = tok_foresight, tok_memory, tok_output
    st.tok_delim, st.tok_eos = tok_delim, tok_eos
    for name, t in (("kv_len", kv_len), ("pos_next", pos_next), ("seg_start", seg_start), ("seg_n", seg_n),
                    ("seg_pid0", seg_pid0), ("cand", cand), ("n_cand", n_cand), ("flags", flags),
                    ("out_tok", out_tok), ("n_out", n_out)):
        setattr(st, name, _ptr(t))
    return st


def memosight_decode_scratch_bytes(batch: int) -> int:
    return int(lib().memosight_decode_scratch_bytes(batch))


def memosight_decode_plan(state, q_off, n_cand_blk, row_tok, pos_id, draft, summary, scratch, stream=None) -> None:
    _check(int(lib().memosight_decode_plan(C.byref(state), _ptr(q_off), _ptr(n_cand_blk), _ptr(row_tok),
                                           _ptr(pos_id), _ptr(draft), _ptr(summary), _ptr(scratch),
                                           _stream(stream))), "memosight_decode_plan")


def memosight_decode_commit(state, q_off, argmax, n_match, n_keep, stream=None) -> None:
    _check(int(lib().memosight_decode_commit(C.byref(state), _ptr(q_off), _ptr(argmax), _ptr(n_match),
                                             _ptr(n_keep), _stream(stream))), "memosight_decode_commit")


def memosight_decode_plan_compress(state, q_off, n_cand_blk, row_tok, pos_id, n_keep, seg_start, seg_len, summary,
                                   scratch, stream=None) -> None:
    _check(int(lib().memosight_decode_plan_compress(C.byref(state), _ptr(q_off), _ptr(n_cand_blk), _ptr(row_tok),
                                                    _ptr(pos_id), _ptr(n_keep), _ptr(seg_start), _ptr(seg_len),
                                                    _ptr(summary), _ptr(scratch), _stream(stream))),
           "memosight_decode_plan_compress")


def memosight_decode_commit_compress(state, q_off, argmax, stream=None) -> None:
    _check(int(lib().memosight_decode_commit_compress(C.byref(state), _ptr(q_off), _ptr(argmax),
                                                      _stream(stream))), "memosight_decode_commit_compress")


def memosight_kv_gather(k_cache, v_cache, n_layers, layer_stride, kv_head_stride, batch, n_kv_heads, head_dim,
                        kv_off, kv_len, keep_idx, idx_stride, n_keep, max_keep, stream=None) -> None:
    _check(int(lib().memosight_kv_gather(_ptr(k_cache), _ptr(v_cache), n_layers, layer_stride, kv_head_stride,
                                         batch, n_kv_heads, head_dim, _ptr(kv_off), _ptr(kv_len), _ptr(keep_idx),
                                         idx_stride, _ptr(n_keep), max_keep, _stream(stream))),
           "memosight_kv_gather")


def memosight_kv_append(k_cache, v_cache, kv_head_stride, n_slots, batch, n_kv_heads, head_dim, kv_off, kv_len,
                        kv_cap, k_step, v_step, q_off, n_cand, n_keep, max_nq, bump_len, overflow=None,
                        stream=None) -> None:
    _check(int(lib().memosight_kv_append(_ptr(k_cache), _ptr(v_cache), kv_head_stride, n_slots, batch, n_kv_heads,
                                         head_dim, _ptr(kv_off), _ptr(kv_len), _ptr(kv_cap), _ptr(k_step),
                                         _ptr(v_step), _ptr(q_off), _ptr(n_cand), _ptr(n_keep), max_nq,
                                         int(bool(bump_len)), _ptr(overflow), _stream(stream))),
           "memosight_kv_append")


def memosight_accept_workspace_bytes(total_rows: int, vocab: int) -> int:
    return int(lib().memosight_accept_workspace_bytes(total_rows, vocab))


def memosight_accept(logits, ld_v, vocab, row_off, batch, total_rows, draft, argmax_out, n_match, n_keep,
                     workspace, workspace_bytes, stream=None) -> None:
    _check(int(lib().memosight_accept(_ptr(logits), ld_v, vocab, _ptr(row_off), batch, total_rows, _ptr(draft),
                                      _ptr(argmax_out), _ptr(n_match), _ptr(n_keep), _ptr(workspace),
                                      workspace_bytes, _stream(stream))), "memosight_accept")


MS_ACCEPT_STATIC_MAX_PARTIALS = 65536


def memosight_accept_static(logits, ld_v, vocab, row_off, batch, total_rows, draft, argmax_out, n_match, n_keep,
                            stream=None) -> None:
    """memosight_accept for callers that cannot allocate: no workspace argument, the
    scratch is a fixed array inside the library (see include/memosight.h for the limit,
    the first-call rule and why concurrent calls on one GPU must not overlap)."""
    _check(int(lib().memosight_accept_static(_ptr(logits), ld_v, vocab, _ptr(row_off), batch, total_rows,
                                             _ptr(draft), _ptr(argmax_out), _ptr(n_match), _ptr(n_keep),
                                             _stream(stream))), "memosight_accept_static")
