"""GPU parity: every call of the C-ABI library against the CPU oracle, element by
element, on the same seeded inputs.  Integer and byte work must be bit-exact;
attention stays within |g - o| <= 2e-2 + 1e-2 |o| and max|g - o| <= 1e-2 max|o|."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import (assert_attn_close, check_attn, gpu_attn, oracle_attn, problem_from_inputs,
                     random_problem)
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


# --------------------------------------------------------------------------- RoPE

@pytest.mark.parametrize("D,base,flags", [(64, 1e4, 0), (128, 1e6, 0), (128, 5e5, ms.MS_ROPE_INTERLEAVED),
                                          (64, 1e4, ms.MS_POS_HALF_UNITS), (32, 1e4, 0), (256, 1e4, 0)])
def test_rope_matches_oracle(D, base, flags):
    T, Hq, Hkv = 37, 8, 2
    q = synth.normal_bf16(T * Hq * D, 1, synth.STREAM_Q).view(T, Hq, D)
    k = synth.normal_bf16(T * Hkv * D, 1, synth.STREAM_KSTEP).view(T, Hkv, D)
    pos = torch.tensor([synth.hash_scalar(i, 2, 3) % 150000 for i in range(T)], dtype=torch.int32)
    pos[:4] = torch.tensor([0, 1, 49152, 149999])
    want_q = oracle.rope(bits(q), pos.numpy(), base, flags=flags)
    want_k = oracle.rope(bits(k), pos.numpy(), base, flags=flags)
    gq, gk = q.to(DEV), k.to(DEV)
    ms.memosight_rope_qk(gq, gk, pos.to(DEV), T, Hq, Hkv, D, base, None, flags)
    torch.cuda.synchronize()
    for got, want in ((bits(gq), want_q), (bits(gk), want_k)):
        diff = got.astype(np.int32) - want.astype(np.int32)
        # fp64 on both sides: at most the last bf16 bit may differ, and only where sin/cos
        # implementations differ in their last fp64 bit right at a rounding boundary
        assert np.abs(diff).max() <= 1
        assert np.count_nonzero(diff) <= max(1, diff.size // 100000)


def test_rope_inv_freq_table_and_q_only():
    T, H, D = 5, 3, 64
    q = synth.normal_bf16(T * H * D, 4, synth.STREAM_Q).view(T, H, D)
    pos = torch.tensor([3, 70, 500, 9000, 12], dtype=torch.int32)
    inv = np.geomspace(1.0, 1e-4, D // 2)
    want = oracle.rope(bits(q), pos.numpy(), 0.0, inv_freq=inv)
    gq = q.to(DEV)
    ms.memosight_rope_qk(gq, None, pos.to(DEV), T, H, 0, D, 0.0, inv, 0)
    torch.cuda.synchronize()
    assert np.array_equal(bits(gq), want)


# --------------------------------------------------------------------------- attention

def test_attn_tiny_config():
    inp = synth.make_step_inputs(synth.TINY)
    check_attn(problem_from_inputs(inp), "tiny")
    check_attn(problem_from_inputs(synth.make_step_inputs(synth.TINY, peaked=True)), "tiny peaked")


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("G,Hkv", [(1, 3), (2, 2), (4, 2), (7, 1), (8, 1)])
def test_attn_ragged_lengths_across_tile_edges(D, G, Hkv):
    lens = [0, 1, 127, 128, 129, 255, 256, 700, 1, 1500]
    B = len(lens)
    n_q = [1 + (3 * b) % min(8, 64 // G) for b in range(B)]
    n_c = [(b * 5) % (n_q[b] + 1) for b in range(B)]
    P = random_problem(B, G * Hkv, Hkv, D, lens, n_q, n_c, seed=D + G, anchors=True)
    check_attn(P, f"ragged D={D} G={G}")


@pytest.mark.parametrize("n_c,d", [(1, 0), (1, 3), (3, 3), (0, 4), (8, 0), (4, 4), (7, 7), (8, 8)])
def test_attn_block_shapes(n_c, d):
    G = 4 if (n_c + d) * 4 <= 64 else 64 // (n_c + d)
    if G == 3:
        G = 2
    P = random_problem(3, 2 * G, 2, 128, [300, 64, 1025], [n_c + d] * 3, [n_c] * 3, seed=10 * n_c + d)
    check_attn(P, f"block n_c={n_c} d={d} G={G}")


def test_attn_peaked_scores_and_custom_scale():
    P = random_problem(4, 8, 2, 128, [513, 2000, 90, 128], [6] * 4, [3] * 4, seed=5, qscale=6.0)
    check_attn(P, "peaked")
    P = random_problem(2, 8, 2, 64, [513, 77], [6] * 2, [3] * 2, seed=6)
    check_attn(P, "custom scale", sm_scale=0.31)


def test_attn_empty_blocks_and_empty_batch():
    # sequences without rows are skipped; a batch of zero rows is a no-op
    P = random_problem(4, 8, 2, 128, [100, 300, 0, 50], [0, 6, 3, 0], [0, 3, 3, 0], seed=7)
    check_attn(P, "empty blocks")


def test_attn_general_path_shapes():
    # head_dim outside {64,128} and blocks with more than 64 packed rows take the ALU path
    check_attn(random_problem(2, 4, 2, 32, [70, 5], [5, 2], [2, 1], seed=8, anchors=True), "D=32")
    check_attn(random_problem(2, 4, 2, 96, [70, 129], [5, 2], [2, 1], seed=9), "D=96")
    check_attn(random_problem(1, 2, 1, 256, [40], [4], [4], seed=10), "D=256")
    check_attn(random_problem(2, 16, 1, 128, [200, 31], [8, 6], [4, 6], seed=11), "rows=128")


def test_attn_is_deterministic_and_leaves_inputs_alone():
    P = random_problem(5, 32, 8, 128, [5000, 130, 2048, 3, 900], [6] * 5, [3] * 5, seed=12)
    a, la = gpu_attn(P)
    b, lb = gpu_attn(P)
    assert torch.equal(a, b) and torch.equal(la, lb)


def test_attn_garbage_beyond_length_is_ignored():
    # slots behind each sequence's valid entries hold NaN/Inf bit patterns: nothing may leak
    P = random_problem(3, 8, 2, 128, [100, 257, 1], [6] * 3, [3] * 3, seed=13, headroom=140)
    want, want_lse = oracle_attn(P)
    for b in range(3):
        lo = int(P["kv_off"][b]) + P["lens"][b]
        P["k_cache"][:, lo:lo + 140] = float("nan")
        P["v_cache"][:, lo:lo + 140] = float("inf")
    out, lse = gpu_attn(P)
    assert_attn_close(out, lse, want, want_lse, "garbage tail")


def test_attn_qwen_shaped_config_full():
    inp = synth.make_step_inputs(synth.QWEN7B)
    check_attn(problem_from_inputs(inp), "config 2")
    check_attn(problem_from_inputs(synth.make_step_inputs(synth.QWEN7B, peaked=True)), "config 2 peaked")


def test_attn_llama_ragged_config_full():
    inp = synth.make_step_inputs(synth.LLAMA8B_RAGGED, device=DEV)
    check_attn(problem_from_inputs(inp), "config 3")


# --------------------------------------------------------------------------- compaction / append

def _compact_both(inp, seg_start, seg_len, idx_stride):
    c = inp.cfg
    kb, vb = bits(inp.k_cache), bits(inp.v_cache)
    kv_len = inp.kv_len.cpu().numpy().copy()
    layer_stride = c.n_kv_heads * inp.n_slots * c.head_dim
    want_src = oracle.kv_compact(kb, vb, c.n_layers, layer_stride, inp.n_slots * c.head_dim, c.n_kv_heads,
                                 c.head_dim, inp.kv_off.cpu().numpy(), kv_len, seg_start, seg_len, idx_stride)
    gk, gv = inp.k_cache.to(DEV).clone(), inp.v_cache.to(DEV).clone()
    g_len = inp.kv_len.to(DEV).clone()
    g_src = torch.full((c.batch, idx_stride), -1, dtype=torch.int32, device=DEV)
    tails = [L - s - n for L, s, n in zip(inp.lens, seg_start, seg_len)]
    ms.memosight_kv_compact(gk, gv, c.n_layers, layer_stride, inp.n_slots * c.head_dim, c.batch, c.n_kv_heads,
                            c.head_dim, inp.kv_off.to(DEV), g_len,
                            torch.tensor(seg_start, dtype=torch.int32, device=DEV),
                            torch.tensor(seg_len, dtype=torch.int32, device=DEV), g_src, idx_stride,
                            max(tails + [0]))
    torch.cuda.synchronize()
    assert np.array_equal(g_len.cpu().numpy(), kv_len)
    # compare every valid entry of every layer/head, bit for bit; slots past the new length are free
    offs = inp.offs
    for b in range(c.batch):
        n = int(kv_len[b])
        assert np.array_equal(bits(gk[:, :, offs[b]:offs[b] + n]), kb[:, :, offs[b]:offs[b] + n])
        assert np.array_equal(bits(gv[:, :, offs[b]:offs[b] + n]), vb[:, :, offs[b]:offs[b] + n])
        assert np.array_equal(g_src[b, :n].cpu().numpy(), want_src[b, :n])
    return gk, gv, g_len


def test_compact_tiny_config_paper_shape():
    # config 1: the cache is [192 kept | 64-token step]; 8 memory tokens + <o> are appended
    # behind it (265 entries); evicting the step leaves 201 entries
    cfg = synth.StepConfig("tiny-compact", 1, 4, 2, 64, 265, 265, 3, 3, 1e4, 1024, seed=0x5EED0000)
    inp = synth.make_step_inputs(cfg)
    assert ms.memosight_ama(64, 8) == 8
    _, _, g_len = _compact_both(inp, [192], [64], 272)
    assert g_len.tolist() == [201]
    # segment in mid-cache with a longer tail (tail > n: overlapping move)
    _compact_both(inp, [40], [30], 272)


def test_compact_multi_layer_ragged_overlapping_and_skips():
    cfg = synth.StepConfig("c", 6, 8, 4, 128, 300, 2600, 3, 3, 1e4, 100, n_layers=3, seed=77)
    inp = synth.make_step_inputs(cfg)
    L = inp.lens
    seg_start = [L[0] - 180, 10, 0, L[3] - 1, 5, 17]
    seg_len = [9, 1, 0, 1, L[4] - 5, 512 if L[5] >= 700 else 100]    # tail>n, n=1, skip, last entry, tail=0
    _compact_both(inp, seg_start, seg_len, 2700)


def test_compact_long_cot_shape_512_to_171():
    # config 4's event: a 512-token step followed by 170 memory tokens + <o>
    cfg = synth.StepConfig("c4", 3, 32, 8, 128, 9000, 12000, 4, 4, 5e5, 100, n_layers=2, seed=78)
    inp = synth.make_step_inputs(cfg)
    seg_start = [L - 171 - 512 for L in inp.lens]
    _compact_both(inp, seg_start, [512] * 3, 12000)


def test_append_accepted_candidates():
    cfg = synth.StepConfig("a", 5, 8, 2, 128, 10, 400, 4, 3, 1e4, 100, headroom=8, seed=79)
    inp = synth.make_step_inputs(cfg)
    n_keep = [0, 1, 4, 2, 9]            # 9 > n_cand: clamped to 4 by the library
    kb, vb = bits(inp.k_cache[0]), bits(inp.v_cache[0])
    kv_len = inp.kv_len.numpy().copy()
    oracle.kv_append(kb, vb, inp.n_slots * 128, 2, 128, inp.kv_off.numpy(), kv_len, bits(inp.k_step),
                     bits(inp.v_step), inp.q_off.numpy(), inp.n_cand.numpy(), [0, 1, 4, 2, 4])
    gk, gv, g_len = inp.k_cache[0].to(DEV).clone(), inp.v_cache[0].to(DEV).clone(), inp.kv_len.to(DEV).clone()
    args = (gk, gv, inp.n_slots * 128, inp.n_slots, 5, 2, 128, inp.kv_off.to(DEV), g_len, None, inp.k_step.to(DEV),
            inp.v_step.to(DEV), inp.q_off.to(DEV), inp.n_cand.to(DEV),
            torch.tensor(n_keep, dtype=torch.int32, device=DEV), cfg.n_q)
    ms.memosight_kv_append(*args, 0)
    torch.cuda.synchronize()
    assert g_len.tolist() == inp.lens                         # not bumped
    ms.memosight_kv_append(*args, 1)
    torch.cuda.synchronize()
    assert np.array_equal(g_len.cpu().numpy(), kv_len)
    assert np.array_equal(bits(gk), kb) and np.array_equal(bits(gv), vb)   # whole buffers, untouched slots too


@pytest.mark.parametrize("with_cap", [True, False])
def test_append_stops_at_the_capacity(with_cap):
    # Sequences that have (almost) no room left: the append takes what fits, reports it, moves the
    # length by that much, and writes neither into the neighbour's slots nor behind the tensor.
    cfg = synth.StepConfig("cap", 3, 8, 2, 128, 30, 90, 4, 2, 1e4, 100, headroom=2, seed=80)
    inp = synth.make_step_inputs(cfg)
    n_slots, D, Hkv = inp.n_slots, 128, 2
    if with_cap:
        want_keep = [4, 2, 4]
        cap = [inp.lens[0] + 1, inp.lens[1] + 2, inp.lens[2]]            # room for 1, for 2, for none
        room = [1, 2, 0]
    else:
        want_keep = [2, 2, 4]
        cap = None
        room = [2, 2, 2]            # every sequence has 2 free slots; behind the last one the tensor ends
    keep = [min(w, r) for w, r in zip(want_keep, room)]
    kb, vb = bits(inp.k_cache[0]), bits(inp.v_cache[0])
    kv_len = inp.kv_len.numpy().copy()
    oracle.kv_append(kb, vb, n_slots * D, Hkv, D, inp.kv_off.numpy(), kv_len, bits(inp.k_step), bits(inp.v_step),
                     inp.q_off.numpy(), inp.n_cand.numpy(), keep)
    # the cache tensors sit inside larger buffers whose surroundings must not change
    guard = 4096
    def guarded(t):
        buf = torch.full((t.numel() + 2 * guard,), 7.0, dtype=torch.bfloat16, device=DEV)
        view = buf[guard:guard + t.numel()].view(t.shape)
        view.copy_(t)
        return buf, view
    kbuf, gk = guarded(inp.k_cache[0])
    vbuf, gv = guarded(inp.v_cache[0])
    g_len = inp.kv_len.to(DEV).clone()
    flag = torch.zeros(1, dtype=torch.int32, device=DEV)
    ms.memosight_kv_append(gk, gv, n_slots * D, n_slots, 3, Hkv, D, inp.kv_off.to(DEV), g_len,
                           None if cap is None else torch.tensor(cap, dtype=torch.int32, device=DEV),
                           inp.k_step.to(DEV), inp.v_step.to(DEV), inp.q_off.to(DEV), inp.n_cand.to(DEV),
                           torch.tensor(want_keep, dtype=torch.int32, device=DEV), cfg.n_q, 1, flag)
    torch.cuda.synchronize()
    assert g_len.tolist() == [L + k for L, k in zip(inp.lens, keep)]
    assert int(flag.item()) == 1
    assert np.array_equal(bits(gk), kb) and np.array_equal(bits(gv), vb)
    for buf in (kbuf, vbuf):
        assert bool(torch.all(buf[:guard] == 7.0)) and bool(torch.all(buf[-guard:] == 7.0)), "wrote outside the tensor"


# --------------------------------------------------------------------------- accept

def _accept_both(logits, V, row_off, draft):
    T, ld = logits.shape
    B = len(row_off) - 1
    want_am, want_nm = oracle.accept(logits.cpu().numpy(), V, row_off, draft)
    g_am = torch.full((T + 1,), -7, dtype=torch.int32, device=DEV)
    g_nm = torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)
    g_nk = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    wsb = ms.memosight_accept_workspace_bytes(T, V)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ms.memosight_accept(logits.to(DEV), ld, V, torch.tensor(row_off, dtype=torch.int32, device=DEV), B, T,
                        torch.tensor(draft, dtype=torch.int32, device=DEV), g_am, g_nm, g_nk, ws, wsb)
    torch.cuda.synchronize()
    assert np.array_equal(g_am[:T].cpu().numpy(), want_am)
    assert np.array_equal(g_nm[:B].cpu().numpy(), want_nm)
    rows = np.diff(np.asarray(row_off))
    assert np.array_equal(g_nk.cpu().numpy(), np.where(rows > 0, want_nm + 1, 0))
    assert int(g_am[T]) == -7 and int(g_nm[B]) == -7
    return want_am, want_nm


def test_accept_tiny_and_planted_prefix_lengths():
    for cfg in (synth.TINY, synth.StepConfig("acc", 37, 4, 2, 64, 8, 8, 5, 3, 1e4, 20011, seed=5)):
        a = synth.make_accept_inputs(cfg)
        am, nm = _accept_both(a.logits, cfg.vocab, a.row_off.tolist(), a.draft.tolist())
        assert am.tolist() == a.target
    assert set(nm.tolist()) == set(range(5))          # every prefix length 0..n_c-1 occurs


def test_accept_many_sequences_takes_the_two_launch_form():
    # more rows than the in-kernel tail has counters for: pass 2 is then a launch of its own
    cfg = synth.StepConfig("acc-wide", 700, 4, 2, 64, 8, 8, 2, 1, 1e4, 8192 + 64, seed=15)
    a = synth.make_accept_inputs(cfg)
    am, nm = _accept_both(a.logits, cfg.vocab, a.row_off.tolist(), a.draft.tolist())
    assert am.tolist() == a.target and set(nm.tolist()) == {0, 1}


def test_accept_unplanted_ties_nan_inf_and_unaligned_rows():
    cfg = synth.StepConfig("acc2", 9, 4, 2, 64, 8, 8, 3, 2, 1e4, 8193 + 5, seed=6)
    a = synth.make_accept_inputs(cfg, plant=False, pad=3)       # ld_v not a multiple of 4: scalar path
    lg = a.logits
    lg[1, [9, 8197]] = 50.0
    lg[2, [8196, 0]] = 50.0
    lg[3, 77] = float("inf")
    lg[4, :] = float("-inf")
    lg[5, [30, 8192]] = float("nan")
    lg[5, 10] = float("inf")
    lg[6, :] = 0.0
    lg[6, 5] = -0.0
    lg[:, cfg.vocab:] = 1000.0                                  # padding columns must be ignored
    _accept_both(lg, cfg.vocab, a.row_off.tolist(), a.draft.tolist())
    b = synth.make_accept_inputs(cfg, plant=False, pad=2)       # ld_v % 4 == 0: vector path, same cases
    assert b.ld_v % 4 == 0
    b.logits[:, :cfg.vocab] = lg[:, :cfg.vocab]
    b.logits[:, cfg.vocab:] = 1000.0
    _accept_both(b.logits, cfg.vocab, a.row_off.tolist(), a.draft.tolist())


@pytest.mark.parametrize("V", [4, 132, 8192, 8204, 3 * 8192 + 512, 151936])
def test_accept_streaming_form_ordering_rule(V):
    """16-byte-aligned rows and a vocabulary that is a multiple of 4 take the streaming pass 1
    (bulk copies into a shared-memory ring, branch-free per-lane maxima): ties across lanes, chunks
    and float4 components, NaN, +-inf and all-equal rows must come out by the same ordering rule."""
    cfg = synth.StepConfig("acc3", 12, 4, 2, 64, 8, 8, 3, 2, 1e4, V, seed=7)
    a = synth.make_accept_inputs(cfg, plant=False)
    assert a.ld_v % 4 == 0
    lg = a.logits
    T = lg.shape[0]
    assert T >= 14
    col = lambda x: min(max(int(x), 0), V - 1)
    lg[1, [col(9), col(V - 3)]] = 50.0                      # same maximum early and in the last chunk: first wins
    lg[2, [col(V - 1), col(0)]] = 50.0
    lg[3, [col(128 + 1), col(128 + 2), col(4 * 32 * 5 + 3)]] = 60.0   # same lane, neighbouring components, later group
    lg[4, :] = float("-inf")                                # nothing beats -inf: index 0
    lg[5, col(77)] = float("inf")
    lg[6, [col(30), col(V - 2)]] = float("nan")             # first NaN wins, also over +inf
    lg[6, col(10)] = float("inf")
    lg[7, :] = 0.0
    lg[7, col(5)] = -0.0                                    # -0 == +0: index 0
    lg[8, col(V // 2)] = float("inf")
    lg[8, col(V // 2 + 1)] = float("-inf")                  # +inf and -inf in one float4 group: not a NaN
    lg[9, :] = -3.0e38
    lg[9, col(V - 1)] = -2.9e38
    lg[10, col(3)] = float("nan")
    lg[11, [col(8191), col(8192)]] = 70.0                   # across a chunk boundary
    lg[12, col(V - 1)] = float("nan")
    lg[13, :] = float("nan")
    _accept_both(lg, V, a.row_off.tolist(), a.draft.tolist())


def test_accept_llama_vocab_config():
    cfg = synth.LLAMA8B_RAGGED
    a = synth.make_accept_inputs(cfg, device=DEV)
    am, nm = _accept_both(a.logits, cfg.vocab, a.row_off.tolist(), a.draft.tolist())
    assert am.tolist() == a.target


# --------------------------------------------------------------------------- whole step

def test_whole_step_chain_rope_attn_accept_append():
    """One decode step end to end on both sides: PIDs -> RoPE -> attention -> accept -> append."""
    cfg = synth.StepConfig("chain", 4, 8, 2, 128, 200, 1500, 3, 3, 1e6, 5000, headroom=16, seed=91)
    inp = synth.make_step_inputs(cfg)
    acc = synth.make_accept_inputs(cfg)
    B, nq, nc, d = cfg.batch, cfg.n_q, cfg.n_cand, cfg.d
    # oracle side
    pid_o = np.concatenate([oracle.step_pids(inp.p0[b], nc, d) for b in range(B)])
    q_o = oracle.rope(bits(inp.q), pid_o, cfg.rope_base)
    ks_o = oracle.rope(bits(inp.k_step), pid_o, cfg.rope_base)
    kb, vb = bits(inp.k_cache[0]), bits(inp.v_cache[0])
    want, want_lse = oracle.attn_step(kb, vb, inp.n_slots * 128, inp.kv_off.numpy(), inp.kv_len.numpy(),
                                      inp.q_off.numpy(), inp.n_cand.numpy(), None, q_o, ks_o, bits(inp.v_step))
    am_o, nm_o = oracle.accept(acc.logits.numpy(), cfg.vocab, acc.row_off.numpy(), acc.draft.numpy())
    len_o = inp.kv_len.numpy().copy()
    oracle.kv_append(kb, vb, inp.n_slots * 128, 2, 128, inp.kv_off.numpy(), len_o, ks_o, bits(inp.v_step),
                     inp.q_off.numpy(), inp.n_cand.numpy(), nm_o + 1)
    # CUDA side, through the C ABI only
    pid_g = torch.from_numpy(np.concatenate([ms.memosight_step_pids(inp.p0[b], nc, d) for b in range(B)])).to(DEV)
    q, ks, vs = inp.q.to(DEV), inp.k_step.to(DEV), inp.v_step.to(DEV)
    ms.memosight_rope_qk(q, ks, pid_g, B * nq, 8, 2, 128, cfg.rope_base)
    P = problem_from_inputs(inp, q=q, k_step=ks)
    out, lse = gpu_attn(P)
    assert_attn_close(out, lse, want, want_lse, "chain attention")
    T = B * nq
    am = torch.empty(T, dtype=torch.int32, device=DEV)
    nm = torch.empty(B, dtype=torch.int32, device=DEV)
    nk = torch.empty(B, dtype=torch.int32, device=DEV)
    wsb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ms.memosight_accept(acc.logits.to(DEV), acc.ld_v, cfg.vocab, acc.row_off.to(DEV), B, T, acc.draft.to(DEV),
                        am, nm, nk, ws, wsb)
    gk, gv, g_len = inp.k_cache[0].to(DEV).clone(), inp.v_cache[0].to(DEV).clone(), inp.kv_len.to(DEV).clone()
    ms.memosight_kv_append(gk, gv, inp.n_slots * 128, inp.n_slots, B, 2, 128, inp.kv_off.to(DEV), g_len, None, ks, vs,
                           inp.q_off.to(DEV), inp.n_cand.to(DEV), nk, nq, 1)
    torch.cuda.synchronize()
    assert np.array_equal(am.cpu().numpy(), am_o) and np.array_equal(nm.cpu().numpy(), nm_o)
    assert np.array_equal(g_len.cpu().numpy(), len_o)
    assert np.array_equal(bits(ks), ks_o) and np.array_equal(bits(q), q_o)
    assert np.array_equal(bits(gk), kb) and np.array_equal(bits(gv), vb)


def test_generator_is_identical_on_cpu_and_gpu():
    a = synth.normal_bf16(100000, 3, synth.STREAM_KCACHE, device="cpu", offset=12345)
    b = synth.normal_bf16(100000, 3, synth.STREAM_KCACHE, device=DEV, offset=12345)
    assert torch.equal(a, b.cpu())
    c = synth.normal_f32(100000, 3, synth.STREAM_LOGITS, 2.0, device="cpu", offset=999)
    d = synth.normal_f32(100000, 3, synth.STREAM_LOGITS, 2.0, device=DEV, offset=999)
    assert torch.equal(c, d.cpu())


# --------------------------------------------------------------------------- eviction by keep list

def _gather_both(inp, keeps, idx_stride):
    c = inp.cfg
    B = c.batch
    idx = np.full((B, idx_stride), -1, np.int32)
    for b, kp in enumerate(keeps):
        idx[b, :len(kp)] = kp
    n_keep = np.array([len(kp) for kp in keeps], np.int32)
    kb, vb = bits(inp.k_cache), bits(inp.v_cache)
    kv_len = inp.kv_len.cpu().numpy().copy()
    layer_stride = c.n_kv_heads * inp.n_slots * c.head_dim
    oracle.kv_gather(kb, vb, c.n_layers, layer_stride, inp.n_slots * c.head_dim, c.n_kv_heads, c.head_dim,
                     inp.kv_off.cpu().numpy(), kv_len, idx, n_keep)
    gk, gv = inp.k_cache.to(DEV).clone(), inp.v_cache.to(DEV).clone()
    g_len = inp.kv_len.to(DEV).clone()
    ms.memosight_kv_gather(gk, gv, c.n_layers, layer_stride, inp.n_slots * c.head_dim, B, c.n_kv_heads,
                           c.head_dim, inp.kv_off.to(DEV), g_len, torch.from_numpy(idx).to(DEV), idx_stride,
                           torch.from_numpy(n_keep).to(DEV), int(n_keep.max()))
    torch.cuda.synchronize()
    assert np.array_equal(g_len.cpu().numpy(), kv_len)
    for b in range(B):
        sl = slice(inp.offs[b], inp.offs[b] + int(kv_len[b]))
        assert np.array_equal(bits(gk[:, :, sl]), kb[:, :, sl]) and np.array_equal(bits(gv[:, :, sl]), vb[:, :, sl])
    # slots of other sequences' slack and everything beyond the old lengths are never written
    for b in range(B):
        sl = slice(inp.offs[b] + inp.lens[b], inp.offs[b] + inp.lens[b] + c.headroom)
        assert np.array_equal(bits(gk[:, :, sl]), bits(inp.k_cache[:, :, sl]))


def test_gather_keep_lists_of_other_eviction_policies():
    cfg = synth.StepConfig("g", 6, 8, 4, 128, 300, 2600, 3, 3, 1e4, 100, n_layers=2, seed=91, headroom=32)
    inp = synth.make_step_inputs(cfg)
    rng = np.random.default_rng(4)
    keeps = []
    for b, L in enumerate(inp.lens):
        if b == 0:      # heavy-hitter style: a recent window plus scattered older entries
            old = sorted(rng.choice(L - 256, size=128, replace=False).tolist())
            keeps.append(old + list(range(L - 256, L)))
        elif b == 1:    # separator style: initial tokens, every 17th entry, the neighbourhood
            keeps.append(sorted(set(range(4)) | set(range(0, L, 17)) | set(range(L - 64, L))))
        elif b == 2:    # keep everything
            keeps.append(list(range(L)))
        elif b == 3:    # keep nothing
            keeps.append([])
        elif b == 4:    # the method's own eviction: everything but one step
            keeps.append(list(range(0, 50)) + list(range(50 + 200, L)))
        else:           # only the last entry
            keeps.append([L - 1])
    _gather_both(inp, keeps, 2700)


def test_gather_random_lists_and_head_dim_64():
    cfg = synth.StepConfig("g64", 9, 4, 2, 64, 1, 700, 3, 3, 1e4, 100, n_layers=3, seed=92, headroom=16)
    inp = synth.make_step_inputs(cfg)
    rng = np.random.default_rng(5)
    keeps = [sorted(rng.choice(L, size=int(rng.integers(0, L + 1)), replace=False).tolist()) for L in inp.lens]
    _gather_both(inp, keeps, 704)
