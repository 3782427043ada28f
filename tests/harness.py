"""Glue used by the GPU parity tests: runs one problem through the CUDA library
(via the C-ABI binding) and through the CPU oracle, and compares.

A "problem" is a dict of torch tensors in the library's layout:
  k_cache, v_cache  bf16 [H_kv][n_slots][D] (one layer)
  kv_off int64 [B], kv_len int32 [B], q_off int32 [B+1], n_cand int32 [B], anchor int32 [T] | None
  q bf16 [T][H_q][D], k_step, v_step bf16 [T][H_kv][D]
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from conftest import bits
from paper_2604_14889_b200 import binding as ms

ABS_TOL, REL_TOL = 2e-2, 1e-2          # the stated gate: |g - o| <= 2e-2 + 1e-2 |o|
PEAK_TOL = 1e-2                        # self-imposed: max|g - o| <= 1e-2 max|o|


def random_problem(B, Hq, Hkv, D, lens, n_q_list, n_c_list, seed, headroom=5, qscale=1.0, anchors=False):
    g = torch.Generator().manual_seed(seed)
    offs, tot = [], 0
    for L in lens:
        offs.append(tot)
        tot += L + headroom
    tot = max(tot, 1)
    q_off = np.concatenate([[0], np.cumsum(n_q_list)]).astype(np.int32)
    T = int(q_off[-1])

    def rnd(*shape, scale=1.0):
        return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)
    P = dict(
        B=B, Hq=Hq, Hkv=Hkv, D=D, n_slots=tot, T=T, lens=list(lens), max_nq=max(list(n_q_list) + [1]),
        k_cache=rnd(Hkv, tot, D), v_cache=rnd(Hkv, tot, D),
        kv_off=torch.tensor(offs, dtype=torch.int64), kv_len=torch.tensor(lens, dtype=torch.int32),
        q_off=torch.from_numpy(q_off), n_cand=torch.tensor(n_c_list, dtype=torch.int32),
        q=rnd(max(T, 1), Hq, D, scale=qscale)[:T], k_step=rnd(max(T, 1), Hkv, D)[:T],
        v_step=rnd(max(T, 1), Hkv, D)[:T], anchor=None)
    if anchors:
        a = torch.zeros(T, dtype=torch.int32)
        for b in range(B):
            for i in range(n_q_list[b]):
                a[q_off[b] + i] = int(torch.randint(0, n_c_list[b] + 1, (1,), generator=g))
        P["anchor"] = a
    return P


def problem_from_inputs(inp, layer=0, q=None, k_step=None):
    """View one layer of synth.StepInputs as a problem dict (tensors stay where they are)."""
    c = inp.cfg
    return dict(B=c.batch, Hq=c.n_q_heads, Hkv=c.n_kv_heads, D=c.head_dim, n_slots=inp.n_slots,
                T=inp.q.shape[0], lens=list(inp.lens), max_nq=c.n_q,
                k_cache=inp.k_cache[layer], v_cache=inp.v_cache[layer], kv_off=inp.kv_off, kv_len=inp.kv_len,
                q_off=inp.q_off, n_cand=inp.n_cand, q=inp.q if q is None else q,
                k_step=inp.k_step if k_step is None else k_step, v_step=inp.v_step, anchor=None)


def gpu_attn(P, sm_scale=0.0, want_lse=True, canary=True, device="cuda", ws_min_bytes=0):
    """Runs memosight_attn_step; returns (out bf16 [T][Hq][D] on host, lse fp32 [T][Hq] on host).
    The workspace has exactly the size the library asks for (or ws_min_bytes if that is more) and
    a canary region behind it that must come back untouched."""
    dev = torch.device(device)
    d = {k: (v.to(dev) if torch.is_tensor(v) else v) for k, v in P.items()}
    T, Hq, D = P["T"], P["Hq"], P["D"]
    pad = 64 if canary else 0
    out_buf = torch.full((max(T, 1) * Hq * D + 2 * pad,), 7.0, dtype=torch.bfloat16, device=dev)
    out = out_buf[pad:pad + T * Hq * D].view(T, Hq, D)
    lse_buf = torch.full((max(T, 1) * Hq + 2 * pad,), 7.0, dtype=torch.float32, device=dev)
    lse = lse_buf[pad:pad + T * Hq].view(T, Hq)
    max_kv = max(P["lens"] + [0, P.get("max_kv_len", 0)])      # the host's bound may exceed every actual length
    ws_bytes = ms.memosight_attn_workspace_bytes(P["B"], Hq, P["Hkv"], D, max_kv, P["max_nq"])
    assert ws_bytes > 0
    ws_bytes = max(ws_bytes, ws_min_bytes)
    guard = 1 << 16
    ws_buf = torch.full((ws_bytes + guard,), 0xA5, dtype=torch.uint8, device=dev)
    ws = ws_buf[:ws_bytes]
    ms.memosight_attn_step(
        batch=P["B"], n_q_heads=Hq, n_kv_heads=P["Hkv"], head_dim=D, k_cache=d["k_cache"], v_cache=d["v_cache"],
        kv_head_stride=P["n_slots"] * D, n_slots=P["n_slots"], kv_off=d["kv_off"], kv_len=d["kv_len"],
        max_kv_len=max_kv, max_nq=P["max_nq"], q_off=d["q_off"], n_cand=d["n_cand"], anchor=d["anchor"],
        total_rows=T, sm_scale=sm_scale, q=d["q"], k_step=d["k_step"], v_step=d["v_step"], out=out,
        lse=lse if want_lse else None, workspace=ws, workspace_bytes=ws_bytes)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    assert bool(torch.all(ws_buf[ws_bytes:] == 0xA5)), "workspace overrun"
    if canary:
        assert torch.all(out_buf[:pad] == 7.0) and torch.all(out_buf[pad + T * Hq * D:] == 7.0), "out overrun"
        if want_lse:
            assert torch.all(lse_buf[:pad] == 7.0) and torch.all(lse_buf[pad + T * Hq:] == 7.0), "lse overrun"
    return out.cpu(), lse.cpu()


def oracle_attn(P, sm_scale=None):
    h = {k: (v.cpu() if torch.is_tensor(v) else v) for k, v in P.items()}
    return oracle.attn_step(
        bits(h["k_cache"]), bits(h["v_cache"]), P["n_slots"] * P["D"], h["kv_off"].numpy(), h["kv_len"].numpy(),
        h["q_off"].numpy(), h["n_cand"].numpy(), None if h["anchor"] is None else h["anchor"].numpy(),
        bits(h["q"]).reshape(P["T"], P["Hq"], P["D"]), bits(h["k_step"]).reshape(P["T"], P["Hkv"], P["D"]),
        bits(h["v_step"]).reshape(P["T"], P["Hkv"], P["D"]), sm_scale)


def assert_attn_close(got_out, got_lse, want_out, want_lse, what=""):
    g = got_out.double().numpy()
    err = np.abs(g - want_out)
    gate = ABS_TOL + REL_TOL * np.abs(want_out)
    worst = float((err - gate).max()) if err.size else -1.0
    assert worst <= 0, f"{what}: |g-o| exceeds 2e-2 + 1e-2|o| by {worst:.3e} (max err {err.max():.3e})"
    if err.size:
        peak = float(np.abs(want_out).max())
        assert err.max() <= PEAK_TOL * peak + 1e-30, \
            f"{what}: max err {err.max():.3e} > 1e-2 * max|ref| ({peak:.3e})"
    if got_lse is not None and want_lse is not None and want_lse.size:
        lerr = np.abs(got_lse.double().numpy() - want_lse)
        assert lerr.max() <= 2e-3 + 1e-4 * np.abs(want_lse).max(), f"{what}: lse err {lerr.max():.3e}"


def check_attn(P, what="", sm_scale=0.0):
    out, lse = gpu_attn(P, sm_scale=sm_scale)
    want, want_lse = oracle_attn(P, None if sm_scale == 0.0 else sm_scale)
    assert_attn_close(out, lse, want, want_lse, what)
    return out, lse
