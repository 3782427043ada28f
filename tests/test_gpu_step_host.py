"""memosight_step_host -- one whole step with the step's inputs and results in (pinned) host
memory -- must leave exactly what the separate calls leave on device-resident inputs: the
rotated Q/K, the attention output, argmax / n_match / n_keep, the cache after append and
compaction.  Two steps in a row with different logits, so that the second step's logits
(copied on the library's own copy stream while the attention runs) must wait for the first
step's accept, and the second accept for its own logits."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_step_host_equals_the_separate_calls_two_steps():
    cfg = synth.StepConfig("host", 5, 32, 8, 128, 600, 2100, 3, 3, 5.0e5, 40000, headroom=64, seed=0x5EED0201)
    B, Hq, Hkv, D, nq = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_q
    T = B * nq
    inp = synth.make_step_inputs(cfg, device=DEV)
    accs = [synth.make_accept_inputs(cfg, device=DEV),
            synth.make_accept_inputs(synth.StepConfig("host2", 5, 32, 8, 128, 600, 2100, 3, 3, 5.0e5, 40000,
                                                      headroom=64, seed=0x5EED0202), device=DEV)]
    assert not torch.equal(accs[0].logits, accs[1].logits)
    stride = inp.n_slots * D
    max_kv = cfg.len_hi + cfg.headroom
    pos = torch.from_numpy(np.concatenate(
        [ms.memosight_step_pids(inp.p0[b], cfg.n_cand, cfg.d) for b in range(B)])).to(DEV)
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq)
    awb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    seg_start = torch.zeros(B, dtype=torch.int32, device=DEV)
    seg_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    seg_start[2] = inp.lens[2] - 50
    seg_len[2] = 30
    snap = dict(k=inp.k_cache.clone(), v=inp.v_cache.clone(), len=inp.kv_len.clone())

    def buffers():
        return dict(out=torch.zeros((T, Hq, D), dtype=torch.bfloat16, device=DEV),
                    ws=torch.zeros(wsb, dtype=torch.uint8, device=DEV), aws=torch.zeros(awb, dtype=torch.uint8, device=DEV),
                    am=torch.zeros(T, dtype=torch.int32, device=DEV), nm=torch.zeros(B, dtype=torch.int32, device=DEV),
                    nk=torch.zeros(B, dtype=torch.int32, device=DEV))

    # ---- reference: the separate calls on device-resident inputs, two steps
    want = []
    t = buffers()
    for s in range(2):
        q, ks = inp.q.clone(), inp.k_step.clone()
        ms.memosight_rope_qk(q, ks, pos, T, Hq, Hkv, D, cfg.rope_base)
        ms.memosight_attn_step(
            batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
            kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
            max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=q, k_step=ks,
            v_step=inp.v_step, out=t["out"], lse=None, workspace=t["ws"], workspace_bytes=wsb)
        a = accs[s]
        ms.memosight_accept(a.logits, a.ld_v, cfg.vocab, a.row_off, B, T, a.draft, t["am"], t["nm"], t["nk"], t["aws"], awb)
        ms.memosight_kv_append(inp.k_cache[0], inp.v_cache[0], stride, inp.n_slots, B, Hkv, D, inp.kv_off, inp.kv_len,
                               None, ks, inp.v_step, inp.q_off, inp.n_cand, t["nk"], nq, 1)
        if s == 0:
            ms.memosight_kv_compact(inp.k_cache, inp.v_cache, 1, Hkv * stride, stride, B, Hkv, D, inp.kv_off,
                                    inp.kv_len, seg_start, seg_len, None, 0, 20)
        torch.cuda.synchronize()
        want.append(dict(out=t["out"].clone(), am=t["am"].clone(), nm=t["nm"].clone(), len=inp.kv_len.clone(),
                         k=inp.k_cache.clone(), v=inp.v_cache.clone()))
    am_o, nm_o = oracle.accept(accs[1].logits.cpu().numpy(), cfg.vocab, accs[1].row_off.cpu().numpy(),
                               accs[1].draft.cpu().numpy())
    assert np.array_equal(want[1]["am"].cpu().numpy(), am_o) and np.array_equal(want[1]["nm"].cpu().numpy(), nm_o)

    # ---- the same two steps through memosight_step_host, inputs and results in pinned host memory
    inp.k_cache.copy_(snap["k"])
    inp.v_cache.copy_(snap["v"])
    inp.kv_len.copy_(snap["len"])
    g = buffers()
    h_q, h_ks, h_vs = inp.q.cpu().pin_memory(), inp.k_step.cpu().pin_memory(), inp.v_step.cpu().pin_memory()
    h_pos = pos.cpu().pin_memory()
    h_logits = [a.logits.cpu().pin_memory() for a in accs]
    h_draft = [a.draft.cpu().pin_memory() for a in accs]
    h_out = torch.zeros((T, Hq, D), dtype=torch.bfloat16).pin_memory()
    h_am, h_nm = torch.zeros(T, dtype=torch.int32).pin_memory(), torch.zeros(B, dtype=torch.int32).pin_memory()
    d_q, d_ks, d_vs = torch.empty_like(inp.q), torch.empty_like(inp.k_step), torch.empty_like(inp.v_step)
    d_pos, d_draft, d_logits = torch.empty_like(pos), torch.empty_like(accs[0].draft), torch.empty_like(accs[0].logits)
    p = ms.StepHostParams()
    p.struct_size = C.sizeof(ms.StepHostParams)
    p.attn = ms.attn_params(
        batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
        kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
        max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=d_q, k_step=d_ks,
        v_step=d_vs, out=g["out"], lse=None, workspace=g["ws"], workspace_bytes=wsb)
    p.h_q, p.h_k_step, p.h_v_step = h_q.data_ptr(), h_ks.data_ptr(), h_vs.data_ptr()
    p.h_pos_id, p.d_pos_id = h_pos.data_ptr(), d_pos.data_ptr()
    p.rope_base, p.rope_flags, p.vocab = cfg.rope_base, 0, cfg.vocab
    p.ld_v, p.d_logits, p.d_draft = accs[0].ld_v, d_logits.data_ptr(), d_draft.data_ptr()
    p.d_argmax, p.d_n_match, p.d_n_keep = g["am"].data_ptr(), g["nm"].data_ptr(), g["nk"].data_ptr()
    p.accept_workspace, p.accept_workspace_bytes = g["aws"].data_ptr(), awb
    p.max_tail = 20
    p.h_out, p.h_argmax, p.h_n_match = h_out.data_ptr(), h_am.data_ptr(), h_nm.data_ptr()
    for s in range(2):                       # queued back to back, no host synchronisation in between
        p.h_logits, p.h_draft = h_logits[s].data_ptr(), h_draft[s].data_ptr()
        p.d_seg_start, p.d_seg_len = (seg_start.data_ptr(), seg_len.data_ptr()) if s == 0 else (None, None)
        ms.memosight_step_host(p)
    torch.cuda.synchronize()
    assert ms.memosight_attn_status(g["ws"]) == ms.MS_OK
    assert torch.equal(h_out, want[1]["out"].cpu())
    assert torch.equal(h_am, want[1]["am"].cpu()) and torch.equal(h_nm, want[1]["nm"].cpu())
    assert torch.equal(inp.kv_len, want[1]["len"])
    assert torch.equal(inp.k_cache, want[1]["k"]) and torch.equal(inp.v_cache, want[1]["v"])

    # ---- and once more with no host buffers at all: the whole device-resident step queued by one call.
    #      The step's tensors are put into the device staging buffers beforehand; nothing is copied.
    inp.k_cache.copy_(snap["k"])
    inp.v_cache.copy_(snap["v"])
    inp.kv_len.copy_(snap["len"])
    g["out"].zero_()
    for name in ("h_q", "h_k_step", "h_v_step", "h_pos_id", "h_logits", "h_draft", "h_out", "h_argmax", "h_n_match"):
        setattr(p, name, None)
    d_pos.copy_(pos)
    for s in range(2):
        d_q.copy_(inp.q)
        d_ks.copy_(inp.k_step)
        d_vs.copy_(inp.v_step)
        p.d_logits, p.d_draft = accs[s].logits.data_ptr(), accs[s].draft.data_ptr()
        p.d_seg_start, p.d_seg_len = (seg_start.data_ptr(), seg_len.data_ptr()) if s == 0 else (None, None)
        ms.memosight_step_host(p)
    torch.cuda.synchronize()
    assert ms.memosight_attn_status(g["ws"]) == ms.MS_OK
    assert torch.equal(g["out"], want[1]["out"])
    assert torch.equal(g["am"], want[1]["am"]) and torch.equal(g["nm"], want[1]["nm"])
    assert torch.equal(inp.kv_len, want[1]["len"])
    assert torch.equal(inp.k_cache, want[1]["k"]) and torch.equal(inp.v_cache, want[1]["v"])
