"""The C-ABI library without a GPU: it loads, exports every symbol the header
declares, validates arguments on the host, and its integer layout helpers agree
with the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2604_14889_b200 import binding as ms

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "memosight.h")).read()
    return sorted(set(re.findall(r"MS_API\s+[\w\s\*]+?\b(memosight_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 15 and "memosight_attn_step" in names and "memosight_accept" in names
    lib = ms.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert ms.memosight_version() >= 100
    assert lib.memosight_status_string(ms.MS_ERR_ALIGNMENT).decode().startswith("pointer")


def test_params_struct_matches_header_size():
    # struct_size is checked first; an empty batch then returns MS_OK without touching CUDA
    p = ms.AttnParams()
    p.struct_size = C.sizeof(ms.AttnParams)
    p.n_q_heads, p.n_kv_heads, p.head_dim, p.max_nq = 4, 2, 64, 4
    assert ms.lib().memosight_attn_step(C.byref(p), None) == ms.MS_OK
    p.struct_size += 8
    assert ms.lib().memosight_attn_step(C.byref(p), None) == ms.MS_ERR_INVALID_ARG


def test_host_side_validation_codes():
    L = ms.lib()
    assert L.memosight_rope_qk(None, None, None, -1, 1, 1, 64, 1e4, None, 0, None) == ms.MS_ERR_INVALID_ARG
    assert L.memosight_rope_qk(None, None, None, 4, 1, 1, 63, 1e4, None, 0, None) == ms.MS_ERR_UNSUPPORTED_SHAPE
    assert L.memosight_rope_qk(None, None, None, 4, 1, 1, 64, 1e4, None, 0, None) == ms.MS_ERR_INVALID_ARG
    assert L.memosight_rope_qk(None, None, None, 0, 1, 1, 64, 1e4, None, 0, None) == ms.MS_OK
    assert L.memosight_accept(None, 10, 20, None, 1, 1, None, None, None, None, None, 0, None) == ms.MS_ERR_INVALID_ARG
    assert L.memosight_accept_workspace_bytes(-1, 5) == 0
    assert L.memosight_accept_workspace_bytes(6, 1024) >= 6 * 8
    assert L.memosight_kv_compact(None, None, 1, 0, 0, 1, 1, 12, None, None, None, None, None, 0, 0, None) \
        == ms.MS_ERR_UNSUPPORTED_SHAPE
    assert L.memosight_kv_compact(None, None, 1, 0, 0, 0, 1, 64, None, None, None, None, None, 0, 0, None) == ms.MS_OK
    assert L.memosight_kv_append(None, None, 0, 0, 2, 1, 64, None, None, None, None, None, None, None, None, 4, 1,
                                 None, None) \
        == ms.MS_ERR_INVALID_ARG
    assert L.memosight_attn_workspace_bytes(1, 5, 2, 64, 10, 4) == 0          # H_q % H_kv != 0
    assert L.memosight_attn_workspace_bytes(1, 4, 2, 64, 10, 32769) == 0        # block too large
    assert L.memosight_attn_workspace_bytes(1, 4, 2, 64, 10, 4) > 256

    def params(**kw):
        p = ms.AttnParams()
        p.struct_size = C.sizeof(ms.AttnParams)
        p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = 1, 4, 2, 64
        p.max_kv_len, p.max_nq, p.total_rows, p.n_slots, p.kv_head_stride = 8, 4, 4, 16, 16 * 64
        for k, v in kw.items():
            setattr(p, k, v)
        return p
    assert L.memosight_attn_step(C.byref(params(n_q_heads=5)), None) == ms.MS_ERR_INVALID_ARG
    assert L.memosight_attn_step(C.byref(params(head_dim=48)), None) == ms.MS_ERR_UNSUPPORTED_SHAPE
    assert L.memosight_attn_step(C.byref(params(max_nq=32769)), None) == ms.MS_ERR_UNSUPPORTED_SHAPE
    assert L.memosight_attn_step(C.byref(params()), None) == ms.MS_ERR_INVALID_ARG       # null pointers
    fake = 0x1000
    full = dict(k_cache=fake, v_cache=fake, kv_off=fake, kv_len=fake, q_off=fake, n_cand=fake, q=fake,
                k_step=fake, v_step=fake, out=fake, workspace=fake)
    assert L.memosight_attn_step(C.byref(params(**full, workspace_bytes=16)), None) == ms.MS_ERR_WORKSPACE_TOO_SMALL
    bad = dict(full)
    bad["q"] = fake + 2
    assert L.memosight_attn_step(C.byref(params(**bad, workspace_bytes=1 << 30)), None) == ms.MS_ERR_ALIGNMENT
    assert L.memosight_attn_step(C.byref(params(**full, kv_head_stride=8)), None) == ms.MS_ERR_INVALID_ARG


def test_layout_helpers_agree_with_oracle():
    for n in range(0, 70):
        for c in range(1, 10):
            assert ms.memosight_ama(n, c) == oracle.ama(n, c)
            for rho in (0, 3, 4096):
                assert ms.memosight_upl_pids(rho, n, c).tolist() == oracle.upl_pids(rho, n, c).tolist()
                assert ms.memosight_upl_pids(rho, n, c, ms.MS_POS_HALF_UNITS).tolist() == \
                    oracle.upl_pids(rho, n, c, half_units=True).tolist()
                assert ms.memosight_out_pid(rho, n) == oracle.out_pid(rho, n)
                # ablation layouts (App. B.3): monotone PIDs (w/o UPL), fixed budget (w/o AMA)
                assert ms.memosight_upl_pids(rho, n, c, ms.MS_LAYOUT_MONOTONE).tolist() == \
                    oracle.monotone_pids(rho, n, c).tolist()
                if n >= 1:
                    assert ms.memosight_budget_pids(rho, n, c).tolist() == oracle.budget_pids(rho, n, c).tolist()
    with pytest.raises(ms.MemosightError):
        ms.memosight_ama(3, 0)
    with pytest.raises(ms.MemosightError):
        ms.memosight_budget_pids(0, 0, 9)
    with pytest.raises(ms.MemosightError):
        ms.memosight_upl_pids(0, 5, 2, 8)
    for p0 in (0, 9, 50000):
        for n_c in range(0, 6):
            for d in range(0, 6):
                assert ms.memosight_step_pids(p0, n_c, d).tolist() == oracle.step_pids(p0, n_c, d).tolist()
                anc = [(k * 7 + n_c) % (n_c + 1) for k in range(d)]
                assert ms.memosight_step_pids(p0, n_c, d, anc).tolist() == oracle.step_pids(p0, n_c, d, anc).tolist()
    with pytest.raises(ms.MemosightError):
        ms.memosight_step_pids(0, 2, 1, [3])
