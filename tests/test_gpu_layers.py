"""memosight_attn_step_layers against the CPU oracle: stacked layers that share the step's
metadata (Algorithm 1 forwards the whole model per step; every layer keeps a cache of the same
length).  The keys-on-lanes kernel walks all layers in one launch -- units cut across CTAs at
layer boundaries included -- and the other kernels are issued layer by layer; both must give,
layer for layer, what the one-layer oracle gives on that layer's tensors."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import assert_attn_close
from paper_2604_14889_b200 import binding as ms

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layers_case(NL, B, Hq, Hkv, D, lens, n_q, n_c, seed, pad_layers=0, with_lse=True):
    g = torch.Generator().manual_seed(seed)
    offs, tot = [], 0
    for L in lens:
        offs.append(tot)
        tot += L + 3
    n_slots = max(tot, 1)
    q_off = np.concatenate([[0], np.cumsum(n_q)]).astype(np.int32)
    T = int(q_off[-1])

    def rnd(*shape):
        return torch.randn(shape, generator=g).to(torch.bfloat16)
    # a layer stride larger than one layer's tensor: the layers need not be packed
    kv_ls = (Hkv * n_slots + 8 * pad_layers) * D
    q_ls, ks_ls = (T * Hq + 8 * pad_layers) * D, (T * Hkv + 8 * pad_layers) * D
    lse_ls = T * Hq + 4 * pad_layers
    k_cache, v_cache = rnd(NL * kv_ls), rnd(NL * kv_ls)
    q, k_step, v_step = rnd(NL * q_ls), rnd(NL * ks_ls), rnd(NL * ks_ls)
    kv_off = torch.tensor(offs, dtype=torch.int64)
    kv_len = torch.tensor(lens, dtype=torch.int32)
    n_cand = torch.tensor(n_c, dtype=torch.int32)
    out = torch.full((NL * q_ls,), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.full((NL * lse_ls,), 7.0, dtype=torch.float32, device=DEV)
    max_kv, max_nq = max(lens + [0]), max(n_q + [1])
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, max_nq)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    dq, dks, dvs = q.to(DEV), k_step.to(DEV), v_step.to(DEV)
    dk, dv = k_cache.to(DEV), v_cache.to(DEV)
    p = ms.attn_params(batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=dk, v_cache=dv,
                       kv_head_stride=n_slots * D, n_slots=n_slots, kv_off=kv_off.to(DEV), kv_len=kv_len.to(DEV),
                       max_kv_len=max_kv, max_nq=max_nq, q_off=torch.from_numpy(q_off).to(DEV),
                       n_cand=n_cand.to(DEV), anchor=None, total_rows=T, sm_scale=0.0, q=dq, k_step=dks, v_step=dvs,
                       out=out, lse=lse if with_lse else None, workspace=ws, workspace_bytes=wsb)
    ms.memosight_attn_step_layers(p, NL, kv_ls, q_ls, ks_ls, q_ls, lse_ls)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    out_h, lse_h = out.cpu(), lse.cpu()
    for l in range(NL):
        kc = bits(k_cache[l * kv_ls:l * kv_ls + Hkv * n_slots * D]).reshape(Hkv, n_slots, D)
        vc = bits(v_cache[l * kv_ls:l * kv_ls + Hkv * n_slots * D]).reshape(Hkv, n_slots, D)
        want, want_lse = oracle.attn_step(
            kc, vc, n_slots * D, kv_off.numpy(), kv_len.numpy(), q_off, n_cand.numpy(), None,
            bits(q[l * q_ls:l * q_ls + T * Hq * D]).reshape(T, Hq, D),
            bits(k_step[l * ks_ls:l * ks_ls + T * Hkv * D]).reshape(T, Hkv, D),
            bits(v_step[l * ks_ls:l * ks_ls + T * Hkv * D]).reshape(T, Hkv, D), None)
        got = out_h[l * q_ls:l * q_ls + T * Hq * D].view(T, Hq, D)
        got_lse = lse_h[l * lse_ls:l * lse_ls + T * Hq].view(T, Hq) if with_lse else None
        assert_attn_close(got, got_lse, want, want_lse, f"layer {l}")
        # the padding between the layers' outputs is untouched
        assert bool(torch.all(out_h[l * q_ls + T * Hq * D:(l + 1) * q_ls] == 7.0))


def test_three_ragged_layers_in_one_launch():
    lens = [700, 0, 129, 2048, 1, 385]
    _layers_case(3, 6, 8, 2, 128, lens, [6, 3, 6, 5, 6, 1], [3, 1, 3, 5, 0, 1], seed=3, pad_layers=1)


def test_units_cut_at_layer_boundaries():
    # one sequence, one KV head, 5 layers of 150 tiles each over 148 CTAs: CTA ranges straddle the
    # layer boundaries, every unit is cut and merged in the kernel's tail
    _layers_case(5, 1, 4, 1, 128, [149 * 128 + 77], [6], [3], seed=4)


def test_many_small_layers_and_no_lse():
    _layers_case(32, 3, 8, 2, 128, [130, 40, 257], [4, 4, 4], [2, 2, 2], seed=5, with_lse=False)


def test_one_layer_equals_the_plain_call_and_other_kernels_loop():
    _layers_case(1, 2, 8, 2, 128, [300, 17], [6, 6], [3, 3], seed=6)
    # head_dim 64 (mma.sync kernel) and a large block (row-tiled kernel): layer by layer
    _layers_case(2, 2, 8, 2, 64, [300, 17], [6, 6], [3, 3], seed=7, pad_layers=1)
    _layers_case(2, 2, 8, 2, 128, [300, 17], [40, 33], [40, 33], seed=8)
