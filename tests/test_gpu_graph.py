"""The step's calls only queue work on the stream they are given (no allocation, no
synchronisation, no host read), so a whole step -- RoPE, step attention, greedy accept,
append, compaction -- can be captured once in a CUDA graph and replayed.  The replay must
leave exactly the bytes and integers the eagerly launched step leaves, and those are checked
against the oracle by the parity tests; here one replayed step is also compared with the
oracle directly."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import assert_attn_close
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _state(cfg):
    inp = synth.make_step_inputs(cfg, device=DEV)
    acc = synth.make_accept_inputs(cfg, device=DEV)
    return inp, acc


@pytest.mark.parametrize("cfg", [
    synth.StepConfig("graph-d128", 6, 32, 8, 128, 700, 1500, 3, 3, 5.0e5, 4096, headroom=64, seed=0x5EED0101),
    synth.StepConfig("graph-d64", 3, 4, 2, 64, 100, 900, 2, 2, 1.0e4, 1024, headroom=64, seed=0x5EED0102),
], ids=lambda c: c.name)
def test_captured_step_replays_like_the_eager_step(cfg):
    B, Hq, Hkv, D, nq = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_q
    T = B * nq
    inp, acc = _state(cfg)
    stride = inp.n_slots * D
    max_kv = cfg.len_hi + cfg.headroom
    pos = torch.from_numpy(np.concatenate(
        [ms.memosight_step_pids(inp.p0[b], cfg.n_cand, cfg.d) for b in range(B)])).to(DEV)
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq)
    awb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    # one sequence ends a reasoning step here: its last 24 entries before a 5-entry tail are evicted
    seg_start = torch.zeros(B, dtype=torch.int32, device=DEV)
    seg_len = torch.zeros(B, dtype=torch.int32, device=DEV)
    seg_start[1] = inp.lens[1] - 40
    seg_len[1] = 24

    snap = dict(k=inp.k_cache.clone(), v=inp.v_cache.clone(), len=inp.kv_len.clone(), q=inp.q.clone(),
                ks=inp.k_step.clone())

    def fresh():
        inp.k_cache.copy_(snap["k"])
        inp.v_cache.copy_(snap["v"])
        inp.kv_len.copy_(snap["len"])
        return dict(q=snap["q"].clone(), ks=snap["ks"].clone(),
                    out=torch.zeros((T, Hq, D), dtype=torch.bfloat16, device=DEV),
                    lse=torch.zeros((T, Hq), dtype=torch.float32, device=DEV),
                    ws=torch.zeros(wsb, dtype=torch.uint8, device=DEV),
                    aws=torch.zeros(awb, dtype=torch.uint8, device=DEV),
                    am=torch.zeros(T, dtype=torch.int32, device=DEV), nm=torch.zeros(B, dtype=torch.int32, device=DEV),
                    nk=torch.zeros(B, dtype=torch.int32, device=DEV))

    def step(t):
        ms.memosight_rope_qk(t["q"], t["ks"], pos, T, Hq, Hkv, D, cfg.rope_base)
        ms.memosight_attn_step(
            batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
            kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
            max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=t["q"],
            k_step=t["ks"], v_step=inp.v_step, out=t["out"], lse=t["lse"], workspace=t["ws"], workspace_bytes=wsb)
        ms.memosight_accept(acc.logits, acc.ld_v, cfg.vocab, acc.row_off, B, T, acc.draft, t["am"], t["nm"], t["nk"],
                            t["aws"], awb)
        ms.memosight_kv_append(inp.k_cache[0], inp.v_cache[0], stride, inp.n_slots, B, Hkv, D, inp.kv_off, inp.kv_len,
                               None, t["ks"], inp.v_step, inp.q_off, inp.n_cand, t["nk"], nq, 1)
        ms.memosight_kv_compact(inp.k_cache, inp.v_cache, 1, Hkv * stride, stride, B, Hkv, D, inp.kv_off,
                                inp.kv_len, seg_start, seg_len, None, 0, 5)

    # eager: the step as the other tests launch it
    e = fresh()
    step(e)
    torch.cuda.synchronize()
    eager = {k: v.clone() for k, v in e.items() if k not in ("ws", "aws")}
    eager.update(k=inp.k_cache.clone(), v=inp.v_cache.clone(), len=inp.kv_len.clone())

    # captured: the same calls recorded into a graph on a side stream (nothing runs while capturing),
    # then the state is put back and the graph launched once
    g_t = fresh()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        step(g_t)
    torch.cuda.synchronize()
    assert torch.equal(inp.kv_len, snap["len"]), "capturing must not execute the step"
    q0, ks0 = snap["q"], snap["ks"]
    g_t["q"].copy_(q0)
    g_t["ks"].copy_(ks0)
    graph.replay()
    torch.cuda.synchronize()
    assert ms.memosight_attn_status(g_t["ws"]) == ms.MS_OK
    for name in ("q", "ks", "out", "am", "nm", "nk"):
        assert torch.equal(g_t[name], eager[name]), name
    assert torch.equal(g_t["lse"], eager["lse"])
    assert torch.equal(inp.kv_len, eager["len"])
    assert torch.equal(inp.k_cache, eager["k"]) and torch.equal(inp.v_cache, eager["v"])

    # a second replay advances the state once more (lengths grow by the accepted counts again)
    len1 = inp.kv_len.clone()
    seg_len.zero_()
    g_t["q"].copy_(q0)
    g_t["ks"].copy_(ks0)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(inp.kv_len, len1 + g_t["nk"])

    # and the replayed step is the oracle's step: integers exact, attention within the bf16 tolerance
    kv_len0 = np.array(inp.lens, np.int32)
    pid = pos.cpu().numpy()
    q_o = oracle.rope(bits(snap["q"]), pid, cfg.rope_base)
    k_o = oracle.rope(bits(snap["ks"]), pid, cfg.rope_base)
    want, want_lse = oracle.attn_step(bits(snap["k"][0]), bits(snap["v"][0]), stride, np.array(inp.offs, np.int64),
                                      kv_len0, inp.q_off.cpu().numpy(), inp.n_cand.cpu().numpy(), None, q_o, k_o,
                                      bits(inp.v_step))
    assert_attn_close(eager["out"].cpu(), eager["lse"].cpu(), want, want_lse, "captured step")
    am_o, nm_o = oracle.accept(acc.logits.cpu().numpy(), cfg.vocab, acc.row_off.cpu().numpy(), acc.draft.cpu().numpy())
    assert np.array_equal(eager["am"].cpu().numpy(), am_o) and np.array_equal(eager["nm"].cpu().numpy(), nm_o)
