"""GPU parity of the training-time attention mask (Sec. 2.3) over augmented sequences
(Sec. 2.2): memosight_attn_step with tok_kind / tok_step against the oracle, through the
large-block tcgen05 kernel (head_dim 128) and the general kernel (head_dim 64)."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import assert_attn_close
from paper_2604_14889_b200 import binding as ms
from test_oracle_train_mask import augmented_sequence

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(D, G, Hkv, seqs, lens, seed, qscale=1.0):
    """seqs: list of (n_prompt, step_lens, c); lens: cache lengths in front of each block."""
    g = torch.Generator().manual_seed(seed)
    metas = [augmented_sequence(*sq) for sq in seqs]
    n_q = [len(m[0]) for m in metas]
    kind = np.concatenate([m[0] for m in metas])
    step = np.concatenate([m[1] for m in metas])
    B, Hq, T = len(seqs), G * Hkv, int(sum(n_q))
    offs = np.concatenate([[0], np.cumsum([L + 3 for L in lens])])[:-1].astype(np.int64)
    n_slots = int(sum(L + 3 for L in lens)) + 1
    rnd = lambda *shape, s=1.0: (torch.randn(shape, generator=g) * s).to(torch.bfloat16)
    kc, vc = rnd(Hkv, n_slots, D), rnd(Hkv, n_slots, D)
    q, ks, vs = rnd(T, Hq, D, s=qscale), rnd(T, Hkv, D), rnd(T, Hkv, D)
    q_off = np.concatenate([[0], np.cumsum(n_q)]).astype(np.int32)
    kv_len = np.array(lens, np.int32)
    want, want_lse = oracle.attn_step(bits(kc), bits(vc), n_slots * D, offs, kv_len, q_off, np.array(n_q, np.int32),
                                      None, bits(q), bits(ks), bits(vs), tok_kind=kind, tok_step=step)
    out = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((T, Hq), dtype=torch.float32, device=DEV)
    max_nq, max_kv = max(n_q), max(lens)
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, max_nq)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(DEV)
    ms.memosight_attn_step(batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=kc.to(DEV), v_cache=vc.to(DEV),
                           kv_head_stride=n_slots * D, n_slots=n_slots, kv_off=t(offs, torch.int64),
                           kv_len=t(kv_len, torch.int32), max_kv_len=max_kv, max_nq=max_nq, q_off=t(q_off, torch.int32),
                           n_cand=t(np.array(n_q), torch.int32), anchor=None, total_rows=T, sm_scale=0.0, q=q.to(DEV),
                           k_step=ks.to(DEV), v_step=vs.to(DEV), out=out, lse=lse, workspace=ws, workspace_bytes=wsb,
                           tok_kind=t(kind, torch.uint8), tok_step=t(step, torch.int32))
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    assert_attn_close(out.cpu(), lse.cpu(), want, want_lse, f"training mask D={D} G={G}")


def test_training_mask_large_block_kernel():
    _case(128, 4, 2, [(37, [20, 33, 7, 12], 3), (5, [9, 1, 40], 5)], [0, 0], seed=1)


def test_training_mask_behind_a_cached_prefix_and_peaked():
    _case(128, 4, 2, [(0, [25, 31], 3), (11, [6, 6, 6, 6, 6, 6], 2)], [300, 129], seed=2, qscale=4.0)


def test_training_mask_other_group_sizes():
    _case(128, 7, 1, [(20, [15, 22], 4)], [0], seed=3)
    _case(128, 1, 3, [(64, [70, 50], 5)], [0], seed=4)


def test_training_mask_general_kernel_head_dim_64():
    _case(64, 2, 2, [(10, [8, 13], 3), (3, [5], 2)], [0, 17], seed=5)
