"""Pins for the oracle of the decoding-loop bookkeeping (oracle/decode.py; Algorithm 1)."""
import numpy as np
import pytest

import oracle
from oracle import decode as od
from paper_2604_14889_b200 import synth


def _params(m, d, c=3, max_out=10000, max_mem=64):
    return od.Params(d, c, max_out, max_mem, m.tok_f, m.tok_m, m.tok_o, m.tok_delim, m.tok_eos)


def run_oracle_loop(m, p, pid0s, kv0s, max_steps=100000, trace=None):
    """Drives the oracle bookkeeping with the toy model; the cache is only counted here."""
    B = len(pid0s)
    seqs = [od.Seq(kv_len=kv0s[b], pos_next=pid0s[b], seg_start=kv0s[b], seg_n=0, seg_pid0=pid0s[b],
                   cand=[m.truth(b, pid0s[b], pid0s[b])]) for b in range(B)]
    steps = 0
    while steps < max_steps:
        q_off, n_cand, row_tok, pos_id, draft = od.plan(seqs, p)
        pending = [s for s in seqs if (s.flags & od.COMPRESS) and not (s.flags & od.DONE)]
        if len(row_tok) == 0 and not pending:
            break
        if len(row_tok):
            seq_of_row = np.repeat(np.arange(B), np.diff(q_off))
            win = np.array([m.predict(int(seq_of_row[r]), int(row_tok[r]), int(pos_id[r]), pid0s[int(seq_of_row[r])])
                            for r in range(len(row_tok))], np.int32)
            # greedy accept by definition: longest prefix of rows whose prediction equals the draft
            n_match = []
            for b in range(B):
                mlen = 0
                for r in range(q_off[b], q_off[b + 1]):
                    if draft[r] < 0 or win[r] != draft[r]:
                        break
                    mlen += 1
                n_match.append(mlen)
            n_keep = od.commit(seqs, p, q_off, win, n_match)
            for b, s in enumerate(seqs):
                s.kv_len += int(n_keep[b])
            if trace is not None:
                trace.append(("step", n_keep.tolist()))
            steps += 1
        if any((s.flags & od.COMPRESS) and not (s.flags & od.DONE) for s in seqs):
            q_off, n_cand, row_tok, pos_id, n_keep, seg_start, seg_len = od.plan_compress(seqs, p)
            seq_of_row = np.repeat(np.arange(B), np.diff(q_off))
            win = np.array([m.predict(int(seq_of_row[r]), int(row_tok[r]), int(pos_id[r]), pid0s[int(seq_of_row[r])])
                            for r in range(len(row_tok))], np.int32)
            kv_len = np.array([s.kv_len + int(n_keep[b]) - int(seg_len[b]) for b, s in enumerate(seqs)])
            od.commit_compress(seqs, p, q_off, win, kv_len)
            if trace is not None:
                trace.append(("compress", n_keep.tolist(), seg_len.tolist()))
    return seqs, steps


def plain_greedy(m, b, pid0, max_out):
    """Token-by-token greedy decoding with the same model: the stream speculation must reproduce."""
    out, pid, tok = [], pid0, m.truth(b, pid0, pid0)
    while len(out) < max_out:
        out.append(tok)
        if tok == m.tok_eos:
            break
        if tok == m.tok_delim:
            o_pid = pid + 1                      # <o> sits behind the step; the next step follows it
            tok, pid = m.predict(b, m.tok_o, o_pid, pid0), o_pid + 1
        else:
            tok, pid = m.predict(b, tok, pid, pid0), pid + 1
    return out


@pytest.mark.parametrize("d,hit", [(0, 0), (1, 50), (2, 70), (3, 0), (3, 60), (3, 100), (7, 80)])
def test_speculation_reproduces_plain_greedy_decoding(d, hit):
    m = synth.ToyModel(hit_pct=hit, eos_after=300)
    pid0s, kv0s = [0, 17, 4096, 5], [10, 0, 700, 33]
    seqs, steps = run_oracle_loop(m, _params(m, d), pid0s, kv0s)
    for b, s in enumerate(seqs):
        assert s.out == plain_greedy(m, b, pid0s[b], 10000)
        assert s.out[-1] == m.tok_eos and (s.flags & od.DONE)
    if d == 0 or hit == 0:
        assert steps == max(len(s.out) for s in seqs)            # one token per step
    if hit == 100 and d > 0:
        assert steps < max(len(s.out) for s in seqs) / 2          # drafts pay


def test_paper_figure_first_block_accepts_two_tokens():
    # Fig. 1: with d = 3 the Predict pass drafts three tokens behind the model's own next token;
    # the first draft is right, the second is not: two tokens become permanent in the Verify pass
    m = synth.ToyModel(hit_pct=100, step_len=10 ** 9, eos_after=10 ** 9)
    p = _params(m, 3)
    s = od.Seq(kv_len=2, pos_next=2, seg_start=2, seg_n=0, seg_pid0=2, cand=[m.truth(0, 2, 0)])
    q_off, n_cand, row_tok, pos_id, draft = od.plan([s], p)
    assert pos_id.tolist() == [2, 3, 4, 5] and row_tok.tolist()[1:] == [m.tok_f] * 3      # <f> PIDs 3,4,5
    t = [m.truth(0, i, 0) for i in range(8)]
    od.commit([s], p, q_off, np.array([t[3], t[4], t[5] + 1, t[6]]), [0])                 # second draft wrong
    assert s.out == [t[2]] and s.cand == [t[3], t[4], t[5] + 1, t[6]]
    q_off, n_cand, row_tok, pos_id, draft = od.plan([s], p)
    assert draft.tolist()[:4] == [t[4], t[5] + 1, t[6], -1]
    n_keep = od.commit([s], p, q_off, np.array([t[4], t[5], 0, 0, 0, 0, 0]), [1])
    assert n_keep.tolist() == [2] and s.out == [t[2], t[3], t[4]] and s.cand == [t[5]]     # r3, r4 accepted


def test_compression_block_layout_and_cache_accounting():
    m = synth.ToyModel(hit_pct=70, step_len=9, eos_after=150)
    p = _params(m, 3, c=3)
    trace = []
    seqs, _ = run_oracle_loop(m, p, [5], [40], trace=trace)
    # paper example (Fig. 3): a step of PIDs 1..3 with c = 3 gets one <m> at PID 2 and <o> at PID 4
    s = od.Seq(kv_len=3, pos_next=4, seg_start=0, seg_n=3, seg_pid0=1, cand=[0], flags=od.COMPRESS)
    q_off, n_cand, row_tok, pos_id, n_keep, seg_start, seg_len = od.plan_compress([s], p)
    assert row_tok.tolist() == [m.tok_m, m.tok_o] and pos_id.tolist() == [2, 4]
    assert n_keep.tolist() == [2] and seg_start.tolist() == [0] and seg_len.tolist() == [3]
    od.commit_compress([s], p, q_off, np.array([7, 9]), [2])
    assert s.cand == [9] and s.pos_next == 5 and s.seg_start == 2 and s.seg_n == 0 and not s.flags
    # every compression replaces the n entries of a step by ceil(n/c) + 1
    kv = 40
    for ev in trace:
        if ev[0] == "step":
            kv += ev[1][0]
        else:
            n = ev[2][0]
            assert ev[1][0] == oracle.ama(n, 3) + 1
            kv += ev[1][0] - n
    assert kv == seqs[0].kv_len
    n_delims = seqs[0].out.count(m.tok_delim)
    assert sum(1 for ev in trace if ev[0] == "compress") == n_delims > 3


def test_output_budget_ends_a_sequence():
    m = synth.ToyModel(hit_pct=100, step_len=10 ** 9, eos_after=10 ** 9)
    seqs, _ = run_oracle_loop(m, _params(m, 3, max_out=10), [0], [0], max_steps=50)
    assert len(seqs[0].out) == 10 and (seqs[0].flags & od.DONE)
    assert seqs[0].out == plain_greedy(m, 0, 0, 10)


def test_compression_block_is_forwarded_before_the_eviction():
    # The reading this repository takes of Algorithm 1 (Forward of <m_1..m_l, o>, then UpdateCache):
    # the whole compression block -- <o> included -- is one causal block forwarded while the finished
    # step's verbose entries are still in the cache, so every row of it attends to them (Sec. 2.3
    # names reasoning and memory tokens as attending to the current step; <o> follows the memory
    # tokens in the same forward pass and is given the same view).  Pinned here: perturbing one
    # verbose entry changes the memory tokens' AND <o>'s output; after the eviction a later block no
    # longer sees that entry.
    from conftest import bits, from_bits
    import torch
    g = torch.Generator().manual_seed(3)
    D, n, l = 32, 6, 2                                    # a 6-token step, two memory tokens + <o>
    L0 = 5                                                # prompt entries in front of the step
    rnd = lambda *s: torch.randn(s, generator=g).to(torch.bfloat16)
    k_cache, v_cache = rnd(1, 32, D), rnd(1, 32, D)
    q, ks, vs = rnd(l + 1, 1, D), rnd(l + 1, 1, D), rnd(l + 1, 1, D)
    kv_off, kv_len = np.array([0], np.int64), np.array([L0 + n], np.int32)
    q_off, n_cand = np.array([0, l + 1], np.int32), np.array([l + 1], np.int32)

    def forward(kc):
        out, _ = oracle.attn_step(bits(kc), bits(v_cache), 32 * D, kv_off, kv_len, q_off, n_cand, None, bits(q), bits(ks),
                                  bits(vs))
        return out
    base = forward(k_cache)
    k2 = k_cache.clone()
    k2[0, L0 + 2] = rnd(D) * 4                            # one verbose entry of the finished step
    moved = forward(k2)
    for row in range(l + 1):                              # both <m> rows and the <o> row see it
        assert np.abs(moved[row] - base[row]).max() > 1e-3
    # after UpdateCache the entry is gone for everybody that comes later
    kb, vb, len2 = bits(k2), bits(v_cache), kv_len.copy()
    oracle.kv_append(kb[0], vb[0], 32 * D, 1, D, kv_off, len2, bits(ks), bits(vs), q_off, n_cand, np.array([l + 1]))
    oracle.kv_compact(kb, vb, 1, 32 * D, 32 * D, 1, D, kv_off, len2, [L0], [n])
    assert len2.tolist() == [L0 + l + 1]
    kb0 = bits(k_cache)
    len0 = kv_len.copy()
    oracle.kv_append(kb0[0], vb[0].copy(), 32 * D, 1, D, kv_off, len0, bits(ks), bits(vs), q_off, n_cand, np.array([l + 1]))
    oracle.kv_compact(kb0, vb.copy(), 1, 32 * D, 32 * D, 1, D, kv_off, len0, [L0], [n])
    assert np.array_equal(kb[0][0, :L0 + l + 1], kb0[0][0, :L0 + l + 1])
