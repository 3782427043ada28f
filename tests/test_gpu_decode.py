"""GPU parity of the whole inference loop (Algorithm 1): the device-resident bookkeeping calls
(memosight_decode_*) drive RoPE, step attention, greedy accept, append, the compression
block (large-block attention) and the eviction over two layers, with a toy model in place of
the language model.  The same loop runs on the CPU oracle; every step's metadata and integer
results must be identical, attention outputs within tolerance, and at the end the token
streams, cache lengths and cache contents must agree -- and the tokens must be what plain
token-by-token greedy decoding gives."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits, from_bits
from oracle import decode as od
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth
from test_oracle_decode import plain_greedy

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _i32(x):
    return torch.tensor(x, dtype=torch.int32, device=DEV)


@pytest.mark.parametrize("d,hit,c", [(3, 70, 3), (1, 40, 5), (0, 0, 2)])
def test_loop_matches_oracle_loop(d, hit, c):
    m = synth.ToyModel(hit_pct=hit, step_len=19, eos_after=110, vocab=1000)
    B, Hq, Hkv, D, NL, base, max_mem = 5, 8, 2, 128, 2, 1.0e4, 64
    kv0 = [40, 0, 300, 129, 77]
    pid0 = [40, 0, 900, 129, 5]
    cap = 420
    offs = [sum(k + cap for k in kv0[:b]) for b in range(B)]
    n_slots = sum(k + cap for k in kv0)
    stride, lstride = n_slots * D, Hkv * n_slots * D
    k_cache = synth.normal_bf16(NL * lstride, 7, synth.STREAM_KCACHE).view(NL, Hkv, n_slots, D)
    v_cache = synth.normal_bf16(NL * lstride, 7, synth.STREAM_VCACHE).view(NL, Hkv, n_slots, D)
    first = [m.truth(b, pid0[b], pid0[b]) for b in range(B)]
    V, max_out = m.vocab, 400

    # ---- oracle side
    p = od.Params(d, c, max_out, max_mem, m.tok_f, m.tok_m, m.tok_o, m.tok_delim, m.tok_eos)
    seqs = [od.Seq(kv_len=kv0[b], pos_next=pid0[b], seg_start=kv0[b], seg_n=0, seg_pid0=pid0[b], cand=[first[b]])
            for b in range(B)]
    kb, vb = bits(k_cache), bits(v_cache)
    o_len = np.array(kv0, np.int32)
    kv_off = np.array(offs, np.int64)

    # ---- device side
    gk, gv = k_cache.to(DEV), v_cache.to(DEV)
    g_len, g_off = _i32(kv0), torch.tensor(offs, dtype=torch.int64, device=DEV)
    cand = torch.zeros((B, d + 1), dtype=torch.int32, device=DEV)
    cand[:, 0] = _i32(first)
    st_t = dict(kv_len=g_len, pos_next=_i32(pid0), seg_start=_i32(kv0), seg_n=_i32([0] * B), seg_pid0=_i32(pid0),
                cand=cand, n_cand=_i32([1] * B), flags=_i32([0] * B),
                out_tok=torch.zeros((B, max_out), dtype=torch.int32, device=DEV), n_out=_i32([0] * B))
    st = ms.decode_state(B, d, c, max_out, max_mem, m.tok_f, m.tok_m, m.tok_o, m.tok_delim, m.tok_eos, **st_t)
    T_cap = B * max(2 * d + 1, max_mem + 1)
    q_off, n_blk = torch.zeros(B + 1, dtype=torch.int32, device=DEV), torch.zeros(B, dtype=torch.int32, device=DEV)
    row_tok, pos_id, draft = (torch.zeros(T_cap, dtype=torch.int32, device=DEV) for _ in range(3))
    n_keep, seg_s, seg_l = (torch.zeros(B, dtype=torch.int32, device=DEV) for _ in range(3))
    summary = torch.zeros(4, dtype=torch.int32, device=DEV)
    scratch = torch.empty(ms.memosight_decode_scratch_bytes(B), dtype=torch.uint8, device=DEV)
    am, nm = torch.zeros(T_cap, dtype=torch.int32, device=DEV), torch.zeros(B, dtype=torch.int32, device=DEV)
    aws = torch.empty(ms.memosight_accept_workspace_bytes(T_cap, V), dtype=torch.uint8, device=DEV)
    max_kv = max(kv0) + cap

    def forward(q_off_h, n_blk_h, row_tok_h, pos_h, draft_h, max_nq):
        """One forward pass of the toy model through both implementations; returns device argmax/n_match."""
        T = int(q_off_h[-1])
        seq_of_row = np.repeat(np.arange(B), np.diff(q_off_h))
        outs = []
        ks_layers, vs_layers = [], []
        for layer in range(NL):
            q, k, v = m.qkv(seq_of_row, row_tok_h, pos_h, layer, Hq, Hkv, D)
            # oracle
            q_o = oracle.rope(bits(q), pos_h, base)
            k_o = oracle.rope(bits(k), pos_h, base)
            want, _ = oracle.attn_step(kb[layer], vb[layer], stride, kv_off, o_len, q_off_h, n_blk_h, None, q_o, k_o,
                                       bits(v))
            # device
            gq, gks, gvs = q.to(DEV), k.to(DEV), v.to(DEV)
            ms.memosight_rope_qk(gq, gks, _i32(pos_h), T, Hq, Hkv, D, base)
            out = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=DEV)
            wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, max_nq)
            ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
            ms.memosight_attn_step(batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=gk[layer],
                                   v_cache=gv[layer], kv_head_stride=stride, n_slots=n_slots, kv_off=g_off,
                                   kv_len=g_len, max_kv_len=max_kv, max_nq=max_nq, q_off=q_off, n_cand=n_blk,
                                   anchor=None, total_rows=T, sm_scale=0.0, q=gq, k_step=gks, v_step=gvs, out=out,
                                   lse=None, workspace=ws, workspace_bytes=wsb)
            assert ms.memosight_attn_status(ws) == ms.MS_OK
            err = np.abs(out.cpu().double().numpy() - want)
            assert np.all(err <= 2e-2 + 1e-2 * np.abs(want)), f"attention, layer {layer}: {err.max():.3e}"
            ks_layers.append((gks, gvs, k_o, bits(v)))
        lg = m.logits(seq_of_row, row_tok_h, pos_h, pid0)
        am_o, nm_o = oracle.accept(lg.numpy(), V, q_off_h, draft_h)
        ms.memosight_accept(lg.to(DEV), V, V, q_off, B, T, _i32(draft_h), am, nm, None, aws, aws.numel())
        torch.cuda.synchronize()
        assert np.array_equal(am[:T].cpu().numpy(), am_o) and np.array_equal(nm.cpu().numpy(), nm_o)
        return am_o, nm_o, ks_layers

    steps = compressions = 0
    while True:
        # ---------------- Predict+Verify block
        ms.memosight_decode_plan(st, q_off, n_blk, row_tok, pos_id, draft, summary, scratch)
        T, live, pending, _ = summary.cpu().tolist()
        o_plan = od.plan(seqs, p)
        assert T == len(o_plan[2])
        for got, want in zip((q_off, n_blk, row_tok[:T], pos_id[:T], draft[:T]), o_plan):
            assert np.array_equal(got.cpu().numpy(), want)
        assert live == sum(1 for s in seqs if not (s.flags & (od.DONE | od.COMPRESS)))
        if T == 0 and pending == 0:
            break
        if T > 0:
            q_off_h, n_blk_h, row_tok_h, pos_h, draft_h = o_plan
            am_o, nm_o, layers = forward(q_off_h, n_blk_h, row_tok_h, pos_h, draft_h, 2 * d + 1)
            keep_o = od.commit(seqs, p, q_off_h, am_o, nm_o)
            ms.memosight_decode_commit(st, q_off, am, nm, n_keep)
            for layer, (gks, gvs, k_o, v_o) in enumerate(layers):
                ms.memosight_kv_append(gk[layer], gv[layer], stride, n_slots, B, Hkv, D, g_off, g_len, None, gks, gvs,
                                       q_off, n_blk, n_keep, 2 * d + 1, layer == NL - 1)
                oracle.kv_append(kb[layer], vb[layer], stride, Hkv, D, kv_off, o_len, k_o, v_o, q_off_h, n_blk_h,
                                 keep_o, bump=(layer == NL - 1))
            torch.cuda.synchronize()
            assert np.array_equal(n_keep.cpu().numpy(), keep_o) and np.array_equal(g_len.cpu().numpy(), o_len)
            steps += 1
        # ---------------- compression of the steps that just ended
        if any((s.flags & od.COMPRESS) and not (s.flags & od.DONE) for s in seqs):
            ms.memosight_decode_plan_compress(st, q_off, n_blk, row_tok, pos_id, n_keep, seg_s, seg_l, summary,
                                              scratch)
            o_c = od.plan_compress(seqs, p)
            T = int(summary[0])
            for got, want in zip((q_off, n_blk, row_tok[:T], pos_id[:T], n_keep, seg_s, seg_l), o_c):
                assert np.array_equal(got.cpu().numpy(), want)
            q_off_h, n_blk_h, row_tok_h, pos_h, keep_o, seg_s_o, seg_l_o = o_c
            am_o, _, layers = forward(q_off_h, n_blk_h, row_tok_h, pos_h, np.full(T, -1, np.int32), max_mem + 1)
            for layer, (gks, gvs, k_o, v_o) in enumerate(layers):
                ms.memosight_kv_append(gk[layer], gv[layer], stride, n_slots, B, Hkv, D, g_off, g_len, None, gks, gvs,
                                       q_off, n_blk, n_keep, max_mem + 1, layer == NL - 1)
                oracle.kv_append(kb[layer], vb[layer], stride, Hkv, D, kv_off, o_len, k_o, v_o, q_off_h, n_blk_h,
                                 keep_o, bump=(layer == NL - 1))
            ms.memosight_kv_compact(gk, gv, NL, lstride, stride, B, Hkv, D, g_off, g_len, seg_s, seg_l, None, 0,
                                    max_mem + 1)
            oracle.kv_compact(kb, vb, NL, lstride, stride, Hkv, D, kv_off, o_len, seg_s_o, seg_l_o)
            ms.memosight_decode_commit_compress(st, q_off, am)
            od.commit_compress(seqs, p, q_off_h, am_o, o_len)
            torch.cuda.synchronize()
            assert np.array_equal(g_len.cpu().numpy(), o_len)
            compressions += 1
        assert steps < 2000

    # ---- the end state
    assert compressions >= 3 and steps >= 10
    n_out = st_t["n_out"].cpu().tolist()
    for b, s in enumerate(seqs):
        got = st_t["out_tok"][b, :n_out[b]].cpu().tolist()
        assert got == s.out == plain_greedy(m, b, pid0[b], max_out)
        assert got[-1] == m.tok_eos
    for name in ("pos_next", "seg_start", "seg_n", "seg_pid0"):
        assert st_t[name].cpu().tolist() == [getattr(s, name) for s in seqs], name
    # caches: identical bits in every valid entry, up to the rare last-bit difference of the two
    # RoPE implementations (fp64 sin/cos) in the appended K rows
    for b in range(B):
        sl = slice(offs[b], offs[b] + int(o_len[b]))
        assert np.array_equal(bits(gv[:, :, sl]), vb[:, :, sl])
        diff = bits(gk[:, :, sl]).astype(np.int32) - kb[:, :, sl].astype(np.int32)
        assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) <= max(1, diff.size // 20000)
