"""ctypes wrapper around the fp64 CPU oracle (``memosight_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke check and the
benchmark's ``cpu_baseline`` / ``--impl reference`` legs may import this
package.  It shares no code with the CUDA path.  All arithmetic lives in the C
file; this module only builds it with gcc, loads it and marshals numpy arrays
(bf16 tensors travel as ``uint16`` bit patterns).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "memosight_oracle.c")
_LIB = os.path.join(_HERE, "libmemosight_oracle.so")
_lock = threading.Lock()
_lib = None

ROPE_INTERLEAVED = 1
POS_HALF_UNITS = 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the .so is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.run(
                ["gcc", "-O2", "-fopenmp", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                 "-o", tmp, _SRC, "-lm"],
                check=True,
            )
            os.replace(tmp, _LIB)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.ms_oracle_ama.restype = C.c_int32
        _lib.ms_oracle_out_pid.restype = C.c_int32
        _lib.ms_oracle_threads.restype = C.c_int32
        _lib.ms_oracle_visible.restype = C.c_int32
    return _lib


def _p(a, ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return a.ctypes.data_as(C.POINTER(ctype))


def _chk(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"oracle {what} rejected its arguments (code {rc})")


def threads() -> int:
    return int(lib().ms_oracle_threads())


def f64_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().ms_oracle_f64_to_bf16(_p(x, C.c_double), _p(out, C.c_uint16), C.c_int64(x.size))
    return out


def bf16_to_f64(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    out = np.empty(x.shape, dtype=np.float64)
    lib().ms_oracle_bf16_to_f64(_p(x, C.c_uint16), _p(out, C.c_double), C.c_int64(x.size))
    return out


def ama(n: int, c: int) -> int:
    r = int(lib().ms_oracle_ama(C.c_int32(n), C.c_int32(c)))
    _chk(min(r, 0), "ama")
    return r


def upl_pids(rho_first: int, n: int, c: int, half_units: bool = False) -> np.ndarray:
    out = np.empty(max(n, 1), dtype=np.int32)
    l = int(lib().ms_oracle_upl_pids(C.c_int32(rho_first), C.c_int32(n), C.c_int32(c),
                                     C.c_int32(int(half_units)), _p(out, C.c_int32)))
    _chk(min(l, 0), "upl_pids")
    return out[:l].copy()


def monotone_pids(rho_first: int, n: int, c: int) -> np.ndarray:
    out = np.empty(max(n, 1), dtype=np.int32)
    l = int(lib().ms_oracle_monotone_pids(C.c_int32(rho_first), C.c_int32(n), C.c_int32(c),
                                          _p(out, C.c_int32)))
    _chk(min(l, 0), "monotone_pids")
    return out[:l].copy()


def budget_pids(rho_first: int, n: int, l: int) -> np.ndarray:
    out = np.empty(max(l, 1), dtype=np.int32)
    r = int(lib().ms_oracle_budget_pids(C.c_int32(rho_first), C.c_int32(n), C.c_int32(l), _p(out, C.c_int32)))
    _chk(min(r, 0), "budget_pids")
    return out[:r].copy()


def out_pid(rho_first: int, n: int) -> int:
    return int(lib().ms_oracle_out_pid(C.c_int32(rho_first), C.c_int32(n)))


def step_pids(p0: int, n_c: int, d: int, anchor=None) -> np.ndarray:
    out = np.empty(n_c + d, dtype=np.int32)
    a = None if anchor is None else np.ascontiguousarray(anchor, dtype=np.int32)
    lib().ms_oracle_step_pids(C.c_int32(p0), C.c_int32(n_c), C.c_int32(d), _p(a, C.c_int32),
                              _p(out, C.c_int32))
    return out


def visible(i: int, j: int, n_c: int, a_i: int) -> bool:
    return bool(lib().ms_oracle_visible(C.c_int32(i), C.c_int32(j), C.c_int32(n_c), C.c_int32(a_i)))


def rope(x: np.ndarray, pos_id: np.ndarray, rope_base: float, inv_freq=None, flags: int = 0) -> np.ndarray:
    """x: uint16 (bf16 bits) [T][H][D]; returns the rotated copy."""
    x = np.array(x, dtype=np.uint16, order="C", copy=True)
    T, H, D = x.shape
    pos = np.ascontiguousarray(pos_id, dtype=np.int32)
    assert pos.shape == (T,)
    f = None if inv_freq is None else np.ascontiguousarray(inv_freq, dtype=np.float64)
    rc = lib().ms_oracle_rope(_p(x, C.c_uint16), _p(pos, C.c_int32), C.c_int32(T), C.c_int32(H),
                              C.c_int32(D), C.c_double(rope_base), _p(f, C.c_double),
                              C.c_uint32(flags))
    _chk(rc, "rope")
    return x


KIND_PROMPT, KIND_REASON, KIND_FORESIGHT, KIND_MEMORY, KIND_OUTPUT = 0, 1, 2, 3, 4


def attn_step(k_cache, v_cache, kv_head_stride, kv_off, kv_len, q_off, n_cand, anchor,
              q, k_step, v_step, sm_scale=None, tok_kind=None, tok_step=None):
    """One layer of step attention.  k_cache/v_cache: uint16 flat or [H_kv][slots][D];
    q: uint16 [T][H_q][D]; k_step/v_step: uint16 [T][H_kv][D].
    tok_kind (uint8 [T]) / tok_step (int32 [T]), both or neither: the block's own keys follow the
    training-time mask of Sec. 2.3 (KIND_* below) instead of the (n_cand, anchor) rule.
    Returns (out fp64 [T][H_q][D], lse fp64 [T][H_q])."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k_step = np.ascontiguousarray(k_step, dtype=np.uint16)
    v_step = np.ascontiguousarray(v_step, dtype=np.uint16)
    k_cache = np.ascontiguousarray(k_cache, dtype=np.uint16)
    v_cache = np.ascontiguousarray(v_cache, dtype=np.uint16)
    T, H_q, D = q.shape
    H_kv = k_step.shape[1]
    kv_off = np.ascontiguousarray(kv_off, dtype=np.int64)
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    q_off = np.ascontiguousarray(q_off, dtype=np.int32)
    n_cand = np.ascontiguousarray(n_cand, dtype=np.int32)
    B = kv_len.shape[0]
    assert q_off.shape == (B + 1,) and int(q_off[-1]) == T
    a = None if anchor is None else np.ascontiguousarray(anchor, dtype=np.int32)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(float(D))
    out = np.empty((T, H_q, D), dtype=np.float64)
    lse = np.empty((T, H_q), dtype=np.float64)
    tk = None if tok_kind is None else np.ascontiguousarray(tok_kind, dtype=np.uint8)
    ts = None if tok_step is None else np.ascontiguousarray(tok_step, dtype=np.int32)
    assert (tk is None) == (ts is None)
    rc = lib().ms_oracle_attn_block(
        C.c_int32(B), C.c_int32(H_q), C.c_int32(H_kv), C.c_int32(D),
        _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16), C.c_int64(kv_head_stride),
        _p(kv_off, C.c_int64), _p(kv_len, C.c_int32), _p(q_off, C.c_int32),
        _p(n_cand, C.c_int32), _p(a, C.c_int32), _p(tk, C.c_uint8), _p(ts, C.c_int32), _p(q, C.c_uint16), _p(k_step, C.c_uint16),
        _p(v_step, C.c_uint16), C.c_double(sm_scale), _p(out, C.c_double), _p(lse, C.c_double))
    _chk(rc, "attn_step")
    return out, lse


def kv_compact(k_cache, v_cache, n_layers, layer_stride, kv_head_stride, H_kv, D, kv_off, kv_len,
               seg_start, seg_len, idx_stride=0):
    """In place on the uint16 arrays k_cache, v_cache and the int32 array kv_len.
    Returns src_idx int32 [B][idx_stride] (or None when idx_stride == 0)."""
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16 and kv_len.dtype == np.int32
    kv_off = np.ascontiguousarray(kv_off, dtype=np.int64)
    seg_start = np.ascontiguousarray(seg_start, dtype=np.int32)
    seg_len = np.ascontiguousarray(seg_len, dtype=np.int32)
    B = kv_len.shape[0]
    src = np.full((B, idx_stride), -1, dtype=np.int32) if idx_stride else None
    rc = lib().ms_oracle_kv_compact(
        _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16), C.c_int32(n_layers),
        C.c_int64(layer_stride), C.c_int64(kv_head_stride), C.c_int32(B), C.c_int32(H_kv),
        C.c_int32(D), _p(kv_off, C.c_int64), _p(kv_len, C.c_int32), _p(seg_start, C.c_int32),
        _p(seg_len, C.c_int32), _p(src, C.c_int32), C.c_int32(idx_stride))
    _chk(rc, "kv_compact")
    return src


def kv_gather(k_cache, v_cache, n_layers, layer_stride, kv_head_stride, H_kv, D, kv_off, kv_len, keep_idx, n_keep):
    """In place on the uint16 arrays and on kv_len: new = old[keep_idx[b][:n_keep[b]]]."""
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16 and kv_len.dtype == np.int32
    kv_off = np.ascontiguousarray(kv_off, dtype=np.int64)
    keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
    n_keep = np.ascontiguousarray(n_keep, dtype=np.int32)
    B = kv_len.shape[0]
    rc = lib().ms_oracle_kv_gather(
        _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16), C.c_int32(n_layers), C.c_int64(layer_stride),
        C.c_int64(kv_head_stride), C.c_int32(B), C.c_int32(H_kv), C.c_int32(D), _p(kv_off, C.c_int64),
        _p(kv_len, C.c_int32), _p(keep_idx, C.c_int32), C.c_int32(keep_idx.shape[1]), _p(n_keep, C.c_int32))
    _chk(rc, "kv_gather")


def kv_append(k_cache, v_cache, kv_head_stride, H_kv, D, kv_off, kv_len, k_step, v_step, q_off,
              n_cand, n_keep, bump=True):
    """In place on k_cache, v_cache (one layer) and kv_len."""
    assert k_cache.dtype == np.uint16 and v_cache.dtype == np.uint16 and kv_len.dtype == np.int32
    kv_off = np.ascontiguousarray(kv_off, dtype=np.int64)
    k_step = np.ascontiguousarray(k_step, dtype=np.uint16)
    v_step = np.ascontiguousarray(v_step, dtype=np.uint16)
    q_off = np.ascontiguousarray(q_off, dtype=np.int32)
    n_cand = np.ascontiguousarray(n_cand, dtype=np.int32)
    n_keep = np.ascontiguousarray(n_keep, dtype=np.int32)
    B = kv_len.shape[0]
    rc = lib().ms_oracle_kv_append(
        _p(k_cache, C.c_uint16), _p(v_cache, C.c_uint16), C.c_int64(kv_head_stride), C.c_int32(B),
        C.c_int32(H_kv), C.c_int32(D), _p(kv_off, C.c_int64), _p(kv_len, C.c_int32),
        _p(k_step, C.c_uint16), _p(v_step, C.c_uint16), _p(q_off, C.c_int32),
        _p(n_cand, C.c_int32), _p(n_keep, C.c_int32), C.c_int32(int(bump)))
    _chk(rc, "kv_append")


def accept(logits: np.ndarray, V: int, row_off, draft):
    """logits fp32 [T][ld_v]; returns (argmax int32 [T], n_match int32 [B])."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, ld_v = logits.shape
    row_off = np.ascontiguousarray(row_off, dtype=np.int32)
    draft = np.ascontiguousarray(draft, dtype=np.int32)
    B = row_off.shape[0] - 1
    assert int(row_off[-1]) == T and draft.shape == (T,)
    am = np.empty(T, dtype=np.int32)
    nm = np.empty(B, dtype=np.int32)
    rc = lib().ms_oracle_accept(_p(logits, C.c_float), C.c_int64(ld_v), C.c_int32(V),
                                _p(row_off, C.c_int32), C.c_int32(B), _p(draft, C.c_int32),
                                _p(am, C.c_int32), _p(nm, C.c_int32))
    _chk(rc, "accept")
    return am, nm
