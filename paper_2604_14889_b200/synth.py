"""Seeded synthetic inputs shaped like MemoSight's decode workloads.

This module only *draws numbers and lays out buffers*; it contains none of the
method's arithmetic (no attention, RoPE, masks, position layout, compaction or
argmax).  It serves the tests, the benchmark and the smoke check, which hand
the same tensors to the CUDA path and to the CPU oracle.

Generator: a counter-based hash (splitmix64 finaliser over the element's linear
index, mixed with a seed and a per-tensor stream id) picks one of 65 536
equal-probability quantiles of the standard normal.  It is integer-only up to a
table lookup, so the CPU and the GPU produce identical bits and any slice of a
huge device-generated tensor can be regenerated on the host from (seed, stream,
offset) alone.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

_M64 = (1 << 64) - 1
_TABLE_CACHE: dict = {}

# per-tensor stream ids
STREAM_Q, STREAM_KSTEP, STREAM_VSTEP, STREAM_KCACHE, STREAM_VCACHE, STREAM_LOGITS = 1, 2, 3, 4, 5, 6
STREAM_LEN, STREAM_TARGET, STREAM_ACCEPT, STREAM_NEEDLE = 7, 8, 9, 10


def _s64(c: int) -> int:
    """Python int -> the int64 two's-complement value with the same low 64 bits."""
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(idx: torch.Tensor, seed: int, stream: int) -> torch.Tensor:
    """splitmix64 finaliser of (idx + key(seed, stream)); idx int64, result int64 bits."""
    key = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _M64
    z = idx + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(0xBF58476D1CE4E5B9)
    z = (z ^ _lsr(z, 27)) * _s64(0x94D049BB133111EB)
    return z ^ _lsr(z, 31)


def hash_scalar(i: int, seed: int, stream: int) -> int:
    """Same hash for one Python integer; returns an unsigned 64-bit value."""
    key = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _M64
    z = (i + key) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _normal_table(device) -> torch.Tensor:
    """fp32 table of the 65 536 mid-quantiles of N(0,1), plus one end guard."""
    key = str(device)
    if key not in _TABLE_CACHE:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        t = math.sqrt(2.0) * torch.special.erfinv(2.0 * p - 1.0)
        t = torch.cat([t, t[-1:]]).to(torch.float32)
        _TABLE_CACHE[key] = t.to(device)
    return _TABLE_CACHE[key]


def normal_bf16(numel: int, seed: int, stream: int, device="cpu", offset: int = 0,
                out: Optional[torch.Tensor] = None, chunk: int = 1 << 25) -> torch.Tensor:
    """bf16 ~ N(0,1): element i is bf16(table[top 16 bits of hash(offset + i)])."""
    if out is None:
        out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    assert flat.numel() == numel
    table = _normal_table(flat.device).to(torch.bfloat16)
    for s in range(0, numel, chunk):
        e = min(numel, s + chunk)
        idx = torch.arange(offset + s, offset + e, dtype=torch.int64, device=flat.device)
        flat[s:e] = table[_lsr(hash64(idx, seed, stream), 48)]
    return out


def normal_f32(numel: int, seed: int, stream: int, sigma: float, device="cpu", offset: int = 0,
               out: Optional[torch.Tensor] = None, chunk: int = 1 << 24) -> torch.Tensor:
    """fp32 ~ N(0, sigma^2): table quantile from the top 16 hash bits, linearly
    interpolated towards the next quantile with the following 16 bits (three
    separately rounded fp32 operations, identical on CPU and GPU)."""
    if out is None:
        out = torch.empty(numel, dtype=torch.float32, device=device)
    flat = out.view(-1)
    assert flat.numel() == numel
    table = _normal_table(flat.device)
    for s in range(0, numel, chunk):
        e = min(numel, s + chunk)
        idx = torch.arange(offset + s, offset + e, dtype=torch.int64, device=flat.device)
        h = hash64(idx, seed, stream)
        hi = _lsr(h, 48)
        frac = (_lsr(h, 32) & 0xFFFF).to(torch.float32) * (1.0 / 65536.0)
        lo_v = table[hi]
        step = table[hi + 1] - lo_v
        step = step * frac
        val = lo_v + step
        flat[s:e] = val * sigma
    return out


def uniform_ints(n: int, lo: int, hi: int, seed: int, stream: int) -> list:
    """n integers uniform in [lo, hi] (inclusive), on the host."""
    span = hi - lo + 1
    return [lo + hash_scalar(i, seed, stream) % span for i in range(n)]


# --------------------------------------------------------------------------- #
# Workload shapes                                                              #
# --------------------------------------------------------------------------- #

@dataclasses.dataclass(frozen=True)
class StepConfig:
    """Shape of one decode-step workload (one attention layer unless n_layers > 1)."""
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    len_lo: int            # compacted cache length, uniform in [len_lo, len_hi]
    len_hi: int
    n_cand: int            # pending candidate tokens per block
    d: int                 # foresight tokens per block
    rope_base: float
    vocab: int
    n_layers: int = 1
    pos_factor: int = 3    # first step PID = pos_factor * L_b (positions keep counting evicted tokens)
    headroom: int = 64     # free slots behind each sequence's entries
    logit_sigma: float = 2.0
    seed: int = 0x5EED0000

    @property
    def n_q(self) -> int:
        return self.n_cand + self.d

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


# The five workload families of this repository's baseline description.  Config
# 4 is listed with one physical layer here; the benchmark chooses how many
# physical layers fit.  Config 5 is a family: `sweep()` instantiates it.
TINY = StepConfig("tiny", 1, 4, 2, 64, 256, 256, 3, 3, 1.0e4, 1024, seed=0x5EED0000)
QWEN7B = StepConfig("qwen2.5-7b-shaped", 1, 28, 4, 128, 4096, 4096, 3, 3, 1.0e6, 152064, seed=0x5EED0001)
LLAMA8B_RAGGED = StepConfig("llama3-8b-shaped-ragged", 16, 32, 8, 128, 2048, 16384, 3, 3, 5.0e5, 128256,
                            seed=0x5EED0002)
LONGCOT = StepConfig("long-cot-serving", 64, 32, 8, 128, 8192, 32768, 4, 4, 5.0e5, 128256,
                     headroom=768, seed=0x5EED0003)


def sweep(batch: int, d: int, kv_len: int, compacted: bool, n_cand: Optional[int] = None,
          headroom: int = 64) -> StepConfig:
    """Config-5 point: 8B shape, fixed cache length, vocabulary 151 936."""
    return StepConfig(f"sweep-b{batch}-d{d}-L{kv_len}", batch, 32, 8, 128, kv_len, kv_len,
                      d if n_cand is None else n_cand, d, 5.0e5, 151936,
                      pos_factor=3 if compacted else 1, headroom=headroom, seed=0x5EED0004)


@dataclasses.dataclass
class StepInputs:
    cfg: StepConfig
    k_cache: torch.Tensor      # bf16 [n_layers][H_kv][slots][D]
    v_cache: torch.Tensor
    n_slots: int
    kv_off: torch.Tensor       # int64 [B]
    kv_len: torch.Tensor       # int32 [B]
    q_off: torch.Tensor        # int32 [B+1]
    n_cand: torch.Tensor       # int32 [B]
    p0: list                   # first step PID of each sequence (host ints)
    q: torch.Tensor            # bf16 [T][H_q][D]  (pre-RoPE)
    k_step: torch.Tensor       # bf16 [T][H_kv][D] (pre-RoPE)
    v_step: torch.Tensor       # bf16 [T][H_kv][D]
    lens: list                 # host copy of kv_len
    offs: list                 # host copy of kv_off


def make_lengths(cfg: StepConfig) -> list:
    if cfg.len_lo == cfg.len_hi:
        return [cfg.len_lo] * cfg.batch
    return uniform_ints(cfg.batch, cfg.len_lo, cfg.len_hi, cfg.seed, STREAM_LEN)


def make_step_inputs(cfg: StepConfig, device="cpu", peaked: bool = False,
                     lens: Optional[list] = None) -> StepInputs:
    """Allocate and fill one workload.  Cache K is drawn directly as post-RoPE
    N(0,1) (a rotation keeps the distribution).  `peaked` scales q by 6 and
    plants four needle keys per (sequence, KV head) -- copies of a query row
    at the first, last and two tile-edge positions -- so that a wrong index or
    mask cannot hide under averaging."""
    B, Hq, Hkv, D = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    lens = make_lengths(cfg) if lens is None else list(lens)
    assert len(lens) == B
    offs, tot = [], 0
    for L in lens:
        offs.append(tot)
        tot += L + cfg.headroom
    n_slots = max(tot, 1)
    T = B * cfg.n_q
    per_layer = Hkv * n_slots * D
    k_cache = torch.empty((cfg.n_layers, Hkv, n_slots, D), dtype=torch.bfloat16, device=device)
    v_cache = torch.empty_like(k_cache)
    normal_bf16(cfg.n_layers * per_layer, cfg.seed, STREAM_KCACHE, out=k_cache)
    normal_bf16(cfg.n_layers * per_layer, cfg.seed, STREAM_VCACHE, out=v_cache)
    q = normal_bf16(T * Hq * D, cfg.seed, STREAM_Q, device=device).view(T, Hq, D)
    k_step = normal_bf16(T * Hkv * D, cfg.seed, STREAM_KSTEP, device=device).view(T, Hkv, D)
    v_step = normal_bf16(T * Hkv * D, cfg.seed, STREAM_VSTEP, device=device).view(T, Hkv, D)
    if peaked:
        q = (q.float() * 6.0).to(torch.bfloat16)
        G = cfg.group
        for b in range(B):
            L = lens[b]
            if L == 0:
                continue
            for h in range(Hkv):
                row = b * cfg.n_q + (hash_scalar(b * Hkv + h, cfg.seed, STREAM_NEEDLE) % cfg.n_q)
                needle = (q[row, h * G].float() * 0.05).to(torch.bfloat16)
                for pos in {0, L - 1, min(127, L - 1), min(128, L - 1)}:
                    k_cache[:, h, offs[b] + pos] = needle
    dev = k_cache.device
    return StepInputs(
        cfg=cfg, k_cache=k_cache, v_cache=v_cache, n_slots=n_slots,
        kv_off=torch.tensor(offs, dtype=torch.int64, device=dev),
        kv_len=torch.tensor(lens, dtype=torch.int32, device=dev),
        q_off=torch.arange(0, T + 1, cfg.n_q, dtype=torch.int32, device=dev),
        n_cand=torch.full((B,), cfg.n_cand, dtype=torch.int32, device=dev),
        p0=[cfg.pos_factor * L for L in lens], q=q, k_step=k_step, v_step=v_step,
        lens=lens, offs=offs)


def regenerate_cache_unit(cfg: StepConfig, n_slots: int, layer: int, head: int, first_slot: int,
                          n_entries: int, which: str) -> torch.Tensor:
    """Host copy of `n_entries` cache rows of one (layer, KV head), regenerated
    from the seed alone (valid for caches that were not modified afterwards and
    were not built with `peaked`)."""
    D = cfg.head_dim
    stream = STREAM_KCACHE if which == "k" else STREAM_VCACHE
    off = ((layer * cfg.n_kv_heads + head) * n_slots + first_slot) * D
    return normal_bf16(n_entries * D, cfg.seed, stream, device="cpu", offset=off).view(n_entries, D)


@dataclasses.dataclass
class AcceptInputs:
    logits: torch.Tensor       # fp32 [T][ld_v]
    ld_v: int
    row_off: torch.Tensor      # int32 [B+1]
    draft: torch.Tensor        # int32 [T]
    target: list               # planted winner of each row (host), -1 where none is planted


def make_accept_inputs(cfg: StepConfig, device="cpu", plant: bool = True, pad: int = 0) -> AcceptInputs:
    """fp32 logits ~ N(0, sigma^2).  With `plant`, every row gets one clear
    winner (+40) at a hashed column, and the drafts of a block agree with the
    winners on a hashed-length prefix and disagree right after it, so that
    accepted-prefix lengths cover 0 .. n_cand-1.  Draft convention: row i of a
    block carries the candidate that follows it (candidate i+1); the last
    candidate row and the foresight rows carry -1."""
    B, V, nq, nc = cfg.batch, cfg.vocab, cfg.n_q, cfg.n_cand
    T = B * nq
    ld_v = V + pad
    logits = torch.empty((T, ld_v), dtype=torch.float32, device=device)
    normal_f32(T * ld_v, cfg.seed, STREAM_LOGITS, cfg.logit_sigma, out=logits)
    target = [-1] * T
    draft = [-1] * T
    for b in range(B):
        n_ok = hash_scalar(b, cfg.seed, STREAM_ACCEPT) % max(nc, 1)   # matching prefix length
        for i in range(nq):
            r = b * nq + i
            if plant:
                target[r] = hash_scalar(r, cfg.seed, STREAM_TARGET) % V
            if i < nc - 1:
                if plant:
                    draft[r] = target[r] if i < n_ok else (target[r] + 1) % V
                else:
                    draft[r] = hash_scalar(r, cfg.seed, STREAM_TARGET) % V
    if plant:
        rows = torch.arange(T, device=logits.device)
        cols = torch.tensor(target, dtype=torch.int64, device=logits.device)
        logits[rows, cols] = 40.0
    dev = logits.device
    return AcceptInputs(
        logits=logits, ld_v=ld_v,
        row_off=torch.arange(0, T + 1, nq, dtype=torch.int32, device=dev),
        draft=torch.tensor(draft, dtype=torch.int32, device=dev), target=target)


# --------------------------------------------------------------------------- #
# A toy "model" for driving the inference loop                                 #
# --------------------------------------------------------------------------- #

STREAM_TOY_TOKEN, STREAM_TOY_HIT, STREAM_TOY_DELIM, STREAM_TOY_ROW = 20, 21, 22, 23


@dataclasses.dataclass(frozen=True)
class ToyModel:
    """Stands in for the language model when the decoding loop is exercised: there are no
    weights in this repository.  Every sequence has a fixed "true" continuation indexed by
    position ID; a regular row (a candidate, or <o>) predicts the true token of the next
    position; a foresight row predicts it only with probability `hit_pct` % (decided by a hash
    of sequence and position), otherwise a wrong token -- which is what makes drafts fail.  The
    q/k/v rows handed to the attention are pseudo-random functions of (sequence, token,
    position, layer).  Holds no arithmetic of the method: it only produces its inputs."""
    vocab: int = 1000           # regular tokens are 0 .. vocab-6; the specials sit above
    hit_pct: int = 60
    step_len: int = 23          # a delimiter roughly every step_len positions
    eos_after: int = 400        # positions (from the sequence's first) after which <eos> comes
    seed: int = 0x70F0

    @property
    def tok_f(self): return self.vocab - 5
    @property
    def tok_m(self): return self.vocab - 4
    @property
    def tok_o(self): return self.vocab - 3
    @property
    def tok_delim(self): return self.vocab - 2
    @property
    def tok_eos(self): return self.vocab - 1

    def truth(self, b: int, pid: int, pid0: int) -> int:
        """True token of sequence b at position pid (pid0 = the sequence's first position)."""
        if pid - pid0 >= self.eos_after:
            return self.tok_eos
        if hash_scalar(b * 1000003 + pid, self.seed, STREAM_TOY_DELIM) % self.step_len == 0:
            return self.tok_delim
        return hash_scalar(b * 1000003 + pid, self.seed, STREAM_TOY_TOKEN) % (self.vocab - 5)

    def predict(self, b: int, tok: int, pid: int, pid0: int) -> int:
        """Token the model's head puts first on a row holding `tok` at position `pid`."""
        t = self.truth(b, pid + 1, pid0)
        if tok == self.tok_f and hash_scalar(b * 1000003 + pid, self.seed, STREAM_TOY_HIT) % 100 >= self.hit_pct:
            return (t + 1) % (self.vocab - 5)
        if tok == self.tok_m:
            return hash_scalar(pid, self.seed, STREAM_TOY_TOKEN) % (self.vocab - 5)
        return t

    def logits(self, seq_of_row, row_tok, pos_id, pid0) -> torch.Tensor:
        """fp32 [T][vocab]: small seeded noise with the predicted token planted 40 above it."""
        T = len(row_tok)
        lg = normal_f32(T * self.vocab, self.seed, STREAM_LOGITS, 2.0).view(T, self.vocab).clone()
        for r in range(T):
            lg[r, self.predict(int(seq_of_row[r]), int(row_tok[r]), int(pos_id[r]), pid0[int(seq_of_row[r])])] += 40.0
        return lg

    def qkv(self, seq_of_row, row_tok, pos_id, layer: int, Hq: int, Hkv: int, D: int):
        """bf16 q [T][Hq][D], k, v [T][Hkv][D] of one layer: each row is its own seeded draw."""
        T = len(row_tok)
        q = torch.empty((T, Hq, D), dtype=torch.bfloat16)
        k = torch.empty((T, Hkv, D), dtype=torch.bfloat16)
        v = torch.empty((T, Hkv, D), dtype=torch.bfloat16)
        for r in range(T):
            key = hash_scalar((int(seq_of_row[r]) * 4099 + int(row_tok[r])) * 65537 + int(pos_id[r]) * 7 + layer,
                              self.seed, STREAM_TOY_ROW) % (1 << 40)
            q[r] = normal_bf16(Hq * D, self.seed, STREAM_Q, offset=key).view(Hq, D)
            k[r] = normal_bf16(Hkv * D, self.seed, STREAM_KSTEP, offset=key).view(Hkv, D)
            v[r] = normal_bf16(Hkv * D, self.seed, STREAM_VSTEP, offset=key).view(Hkv, D)
        return q, k, v
