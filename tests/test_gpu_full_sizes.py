"""Parity at the full sizes of the workload configs, in the launch configuration the
benchmark times.  The oracle cannot afford whole launches here, so it recomputes
sampled (sequence, KV head) units one by one from the very tensors the GPU read;
integer/byte work is still compared bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import ABS_TOL, PEAK_TOL, REL_TOL
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _attn_all(inp, layer=0, q=None, ks=None):
    c = inp.cfg
    T = c.batch * c.n_q
    out = torch.empty((T, c.n_q_heads, c.head_dim), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((T, c.n_q_heads), dtype=torch.float32, device=DEV)
    max_kv = max(inp.lens)
    wsb = ms.memosight_attn_workspace_bytes(c.batch, c.n_q_heads, c.n_kv_heads, c.head_dim, max_kv, c.n_q)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ms.memosight_attn_step(
        batch=c.batch, n_q_heads=c.n_q_heads, n_kv_heads=c.n_kv_heads, head_dim=c.head_dim,
        k_cache=inp.k_cache[layer], v_cache=inp.v_cache[layer], kv_head_stride=inp.n_slots * c.head_dim,
        n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv, max_nq=c.n_q,
        q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0,
        q=inp.q if q is None else q, k_step=inp.k_step if ks is None else ks, v_step=inp.v_step, out=out, lse=lse,
        workspace=ws, workspace_bytes=wsb)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    return out, lse


def _check_sampled_units(inp, out, lse, n_samples, seed, layer=0, units=None):
    """Oracle on single (sequence, KV head) units cut out of the device tensors (`units`: explicit
    (sequence, KV head) pairs instead of hashed ones)."""
    c = inp.cfg
    G, D, nq = c.group, c.head_dim, c.n_q
    worst, peak_ref = 0.0, 0.0
    for i in range(n_samples if units is None else len(units)):
        h = synth.hash_scalar(i, seed, 99)
        b, kvh = (h % c.batch, (h >> 20) % c.n_kv_heads) if units is None else units[i]
        L, o = inp.lens[b], inp.offs[b]
        kc = bits(inp.k_cache[layer, kvh, o:o + L])[None]
        vc = bits(inp.v_cache[layer, kvh, o:o + L])[None]
        rows = slice(b * nq, (b + 1) * nq)
        heads = slice(kvh * G, (kvh + 1) * G)
        want, want_lse = oracle.attn_step(
            kc, vc, max(L, 1) * D, [0], [L], [0, nq], [c.n_cand], None, bits(inp.q[rows, heads]),
            bits(inp.k_step[rows, kvh:kvh + 1]), bits(inp.v_step[rows, kvh:kvh + 1]))
        got = out[rows, heads].double().cpu().numpy()
        err = np.abs(got - want)
        assert np.all(err <= ABS_TOL + REL_TOL * np.abs(want)), (b, kvh, float(err.max()))
        assert err.max() <= PEAK_TOL * np.abs(want).max(), (b, kvh, float(err.max()), float(np.abs(want).max()))
        assert np.abs(lse[rows, heads].double().cpu().numpy() - want_lse).max() < 2e-3
        worst, peak_ref = max(worst, float(err.max())), max(peak_ref, float(np.abs(want).max()))
    return worst, peak_ref


def test_bench_workload_batch128_kv16k_sampled_units():
    cfg = synth.sweep(128, 3, 16384, True)
    inp = synth.make_step_inputs(cfg, device=DEV)
    out, lse = _attn_all(inp)
    out2, lse2 = _attn_all(inp)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)            # run-to-run bit identical
    assert bool(torch.isfinite(out.float()).all())
    _check_sampled_units(inp, out, lse, 24, seed=1)


def test_bench_workload_accept_full():
    cfg = synth.sweep(128, 3, 16384, True)
    a = synth.make_accept_inputs(cfg, device=DEV)
    B, T = cfg.batch, cfg.batch * cfg.n_q
    am = torch.empty(T, dtype=torch.int32, device=DEV)
    nm = torch.empty(B, dtype=torch.int32, device=DEV)
    nk = torch.empty(B, dtype=torch.int32, device=DEV)
    wsb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ms.memosight_accept(a.logits, a.ld_v, cfg.vocab, a.row_off, B, T, a.draft, am, nm, nk, ws, wsb)
    torch.cuda.synchronize()
    want_am, want_nm = oracle.accept(a.logits.cpu().numpy(), cfg.vocab, a.row_off.cpu().numpy(), a.draft.cpu().numpy())
    assert np.array_equal(am.cpu().numpy(), want_am) and np.array_equal(nm.cpu().numpy(), want_nm)
    assert np.array_equal(nk.cpu().numpy(), want_nm + 1)


@pytest.mark.parametrize("d", [1, 2, 3, 4, 5, 6, 7])
def test_sweep_foresight_depths_kv16k(d):
    cfg = synth.sweep(4, d, 16384, True)                   # n_c = d: rows 8 .. 56
    inp = synth.make_step_inputs(cfg, device=DEV)
    out, lse = _attn_all(inp)
    _check_sampled_units(inp, out, lse, 6, seed=10 + d)


def test_sweep_predict_only_and_uncompressed_48k():
    cfg = synth.sweep(2, 3, 49152, False, n_cand=1)        # pure Predict block against the 48K cache
    inp = synth.make_step_inputs(cfg, device=DEV)
    out, lse = _attn_all(inp)
    _check_sampled_units(inp, out, lse, 4, seed=30)


def test_long_cot_config_two_physical_layers_attention_and_compaction():
    # config 4 at full batch and lengths, with 2 of the 32 layers resident (each layer is ~5.4 GB)
    c4 = synth.LONGCOT
    cfg = synth.StepConfig(c4.name, c4.batch, c4.n_q_heads, c4.n_kv_heads, c4.head_dim, c4.len_lo, c4.len_hi,
                           c4.n_cand, c4.d, c4.rope_base, c4.vocab, n_layers=2, headroom=64, seed=c4.seed)
    inp = synth.make_step_inputs(cfg, device=DEV)
    for layer in range(2):
        out, lse = _attn_all(inp, layer=layer)
        _check_sampled_units(inp, out, lse, 8, seed=40 + layer, layer=layer)
    # the compaction event: every sequence drops a 512-token step that is followed by 170 memory
    # tokens and <o>; all layers, K and V
    B, Hkv, D = cfg.batch, cfg.n_kv_heads, cfg.head_dim
    seg_start = [L - 171 - 512 for L in inp.lens]
    samples = [(synth.hash_scalar(i, 7, 98) % B, (synth.hash_scalar(i, 7, 97)) % Hkv, i % 2, i % 2 == 0)
               for i in range(24)]
    before = {s: bits((inp.k_cache if s[3] else inp.v_cache)[s[2], s[1], inp.offs[s[0]]:inp.offs[s[0]] + inp.lens[s[0]]])
              for s in samples}
    g_len = inp.kv_len.clone()
    src = torch.full((B, 33000), -1, dtype=torch.int32, device=DEV)
    stride = inp.n_slots * D
    ms.memosight_kv_compact(inp.k_cache, inp.v_cache, 2, Hkv * stride, stride, B, Hkv, D, inp.kv_off, g_len,
                            torch.tensor(seg_start, dtype=torch.int32, device=DEV),
                            torch.full((B,), 512, dtype=torch.int32, device=DEV), src, 33000, 171)
    torch.cuda.synchronize()
    assert g_len.cpu().tolist() == [L - 512 for L in inp.lens]
    for s in samples:
        b, kvh, layer, is_k = s
        L = inp.lens[b]
        k1 = before[s][None, None].copy()                  # [1 layer][1 head][L][D]
        v1 = k1.copy()
        ln = np.array([L], np.int32)
        want_src = oracle.kv_compact(k1, v1, 1, L * D, L * D, 1, D, [0], ln, [seg_start[b]], [512], idx_stride=L)
        got = bits((inp.k_cache if is_k else inp.v_cache)[layer, kvh, inp.offs[b]:inp.offs[b] + L - 512])
        assert np.array_equal(got, k1[0, 0, :L - 512])
        assert np.array_equal(src[b, :L - 512].cpu().numpy(), want_src[0, :L - 512])


def test_compression_event_batch64_sampled_units():
    # the secondary benchmark's launch: 64 sequences, cache 16 384 + the 512-token step, a causal
    # block of 170 memory tokens + <o> per sequence (six row tiles per KV head, the last one 44 rows)
    cfg = synth.StepConfig("compress-full", 64, 32, 8, 128, 16896, 16896, 171, 0, 5.0e5, 1024, seed=0x5EED0004)
    inp = synth.make_step_inputs(cfg, device=DEV)
    out, lse = _attn_all(inp)
    out2, lse2 = _attn_all(inp)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    assert bool(torch.isfinite(out.float()).all())
    _check_sampled_units(inp, out, lse, 3, seed=5)


def test_wide_group_step_blocks_batch128_units_of_the_cut_last_round():
    # G = 8, 12-token blocks (96 packed rows) at batch 128: 512 units for the large-block kernel;
    # on 148 CTAs units 444..511 (sequences 111..127) are the ones cut into chunks and merged
    cfg = synth.StepConfig("g8-full", 128, 32, 4, 128, 16384, 16384, 6, 6, 5.0e5, 1024, seed=0x5EED0006)
    inp = synth.make_step_inputs(cfg, device=DEV)
    out, lse = _attn_all(inp)
    out2, lse2 = _attn_all(inp)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    _check_sampled_units(inp, out, lse, 0, seed=6, units=[(0, 0), (57, 3), (110, 3), (111, 0), (119, 2), (127, 3)])
