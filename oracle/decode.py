"""Oracle of the loop bookkeeping of MemoSight's iterative inference (paper App. A,
Algorithm 1; Sec. 2.1.1 for the Predict+Verify block, Sec. 2.1.2 / Sec. 2.2 for the
compression block).  Test infrastructure only: plain Python over numpy arrays, one
sequence at a time, in the order the paper states the steps.

Readings where the paper is silent (the same ones the CUDA library documents):
  * c_0, the first pending token, was the model's own prediction and is not re-verified;
    the tokens made permanent in a step are c_0..c_m, m = length of the matching draft prefix;
  * they are cut behind the first step delimiter <e> or <eos> among them;
  * the next c_0 is the model's prediction behind the last permanent token; the foresight
    predictions become the next drafts only if every candidate of the block was accepted;
  * after a delimiter the step is compressed first, and the next step's first token is the
    prediction of <o> (the output token "used to generate subsequent content").
"""
from __future__ import annotations

import dataclasses

import numpy as np

from . import ama, out_pid, step_pids, upl_pids

DONE, COMPRESS = 1, 2


@dataclasses.dataclass
class Seq:
    kv_len: int
    pos_next: int
    seg_start: int
    seg_n: int
    seg_pid0: int
    cand: list          # pending candidates, c_0 first
    flags: int = 0
    out: list = dataclasses.field(default_factory=list)


@dataclasses.dataclass
class Params:
    d: int
    c: int
    max_out: int
    max_mem: int
    tok_f: int
    tok_m: int
    tok_o: int
    tok_delim: int
    tok_eos: int


def plan(seqs, p: Params):
    """Blocks of the live sequences -> (q_off, n_cand, row_tok, pos_id, draft)."""
    q_off, n_cand, row_tok, pos_id, draft = [0], [], [], [], []
    for s in seqs:
        live = not (s.flags & (DONE | COMPRESS))
        n = len(s.cand) if live else 0
        n_cand.append(n)
        if live:
            row_tok += list(s.cand) + [p.tok_f] * p.d
            pos_id += step_pids(s.pos_next, n, p.d).tolist()          # Sec. 2.1.1 / 2.2 layout
            draft += [s.cand[i + 1] if i + 1 < n else -1 for i in range(n)] + [-1] * p.d
        q_off.append(len(row_tok))
    return (np.array(q_off, np.int32), np.array(n_cand, np.int32), np.array(row_tok, np.int32),
            np.array(pos_id, np.int32), np.array(draft, np.int32))


def commit(seqs, p: Params, q_off, argmax, n_match):
    """Applies one verified block per sequence; returns n_keep per sequence."""
    n_keep = []
    for b, s in enumerate(seqs):
        r0, rows = int(q_off[b]), int(q_off[b + 1] - q_off[b])
        if rows == 0:
            n_keep.append(0)
            continue
        n = rows - p.d
        accepted = s.cand[:min(int(n_match[b]), n - 1) + 1]           # c_0 .. c_m
        kept = 0
        for t in accepted:
            if len(s.out) < p.max_out:
                s.out.append(t)
            else:
                s.out_overflow = getattr(s, "out_overflow", 0) + 1
            kept += 1
            if t == p.tok_eos:
                s.flags |= DONE
                break
            if t == p.tok_delim:
                s.flags |= COMPRESS
                break
            if len(s.out) + getattr(s, "out_overflow", 0) >= p.max_out:
                s.flags |= DONE
                break
        s.seg_n += kept
        s.pos_next += kept
        nxt = [int(argmax[r0 + kept - 1])]
        if kept == n and not (s.flags & (DONE | COMPRESS)):
            nxt += [int(argmax[r0 + n + k]) for k in range(p.d)]
        s.cand = nxt
        n_keep.append(kept)
    return np.array(n_keep, np.int32)


def plan_compress(seqs, p: Params):
    """Compression blocks -> (q_off, n_cand, row_tok, pos_id, n_keep, seg_start, seg_len)."""
    q_off, n_cand, row_tok, pos_id, n_keep, seg_start, seg_len = [0], [], [], [], [], [], []
    for s in seqs:
        on = (s.flags & COMPRESS) and not (s.flags & DONE)
        if on:
            l = min(ama(s.seg_n, p.c), p.max_mem)                      # AMA
            pids = upl_pids(s.seg_pid0, s.seg_n, p.c)[:l].tolist()     # UPL centres
            row_tok += [p.tok_m] * l + [p.tok_o]
            pos_id += pids + [out_pid(s.seg_pid0, s.seg_n)]
            n_cand.append(l + 1)
            n_keep.append(l + 1)
            seg_start.append(s.seg_start)
            seg_len.append(s.seg_n)
        else:
            n_cand.append(0)
            n_keep.append(0)
            seg_start.append(0)
            seg_len.append(0)
        q_off.append(len(row_tok))
    return (np.array(q_off, np.int32), np.array(n_cand, np.int32), np.array(row_tok, np.int32),
            np.array(pos_id, np.int32), np.array(n_keep, np.int32), np.array(seg_start, np.int32),
            np.array(seg_len, np.int32))


def commit_compress(seqs, p: Params, q_off, argmax, kv_len):
    for b, s in enumerate(seqs):
        r0, rows = int(q_off[b]), int(q_off[b + 1] - q_off[b])
        if rows == 0:
            continue
        o_pid = out_pid(s.seg_pid0, s.seg_n)
        s.cand = [int(argmax[r0 + rows - 1])]
        s.pos_next = o_pid + 1
        s.seg_pid0 = o_pid + 1
        s.kv_len = int(kv_len[b])
        s.seg_start = s.kv_len
        s.seg_n = 0
        s.flags &= ~COMPRESS
