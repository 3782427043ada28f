#!/usr/bin/env python
"""Benchmark of the MemoSight per-step hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch: step position IDs ->
RoPE at those IDs -> step attention over the compacted KV cache (split-KV + merge)
-> greedy accept -> append of the accepted candidates -> KV compaction of the
sequence(s) whose reasoning step just ended.  The workload is the one the
headline metric is quoted on: Llama-3-8B-shaped layer (H_q=32, H_kv=8, D=128),
compacted cache of 16K entries per sequence, d=3 foresight + 3 candidate tokens
per block, batch 128, vocabulary 151 936, synthetic seeded data.

One JSON line is printed by rank 0.  `value` is step query tokens/s with all
inputs resident in HBM; `e2e` is the same through memosight_step_host with the
step's inputs and results in pinned host memory; `roofline` is the split-KV
attention kernel against the measured HBM copy bandwidth; `cpu_baseline` is the
fp64 oracle on the machine's host cores on a bounded sample.

With --impl reference the "reference" is that oracle (there is no other
implementation of the method): each step runs it on a one-sequence sample.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2604_14889_b200 import synth

METRIC = "step query tokens/s (Predict+Verify attention step, 8B-shape, compacted KV 16K)"
UNIT = "tokens/s"
METRIC_CONFIG = "step query tokens/s (Predict+Verify step of the named configuration: RoPE, attention, accept, append, all layers)"
SEG_LEN, MEM_TOKENS = 512, 170          # one compaction: 512-token step -> 170 memory tokens + <o>
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes the split kernel moved per algorithmic byte in an ncu capture of the batch-48 point
# of the same workload (scaled by the bytes streamed); taken with the kernel as it stands.
NCU_TRAFFIC_PER_ALGO_BYTE = 1.011
KERNELS_PER_STEP = 5                    # rope, attention (merge in its tail), accept, append, compaction


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--kv-len", type=int, default=16384)
    ap.add_argument("--d", type=int, default=3)
    ap.add_argument("--e2e-steps", type=int, default=12)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-sample-seqs", type=int, default=32)
    ap.add_argument("--workload", default="step", choices=["step", "compress", "loop", "cacheops"],
                    help="step: the Predict+Verify step the headline metric is quoted on (default); "
                         "compress: the compression event (forward of the memory tokens + <o>, append, eviction); "
                         "loop: the whole inference loop of Algorithm 1 with a toy model, d = 0..4 x c = 3, 5 x batch 1, 64; "
                         "cacheops: compaction, keep-list eviction, RoPE, append and merge kernels, each timed alone")
    ap.add_argument("--sweep", action="store_true",
                    help="the foresight/batch/cache-length sweep (8B shape): one device-resident run per point, "
                         "a table of KV bytes read, step tokens/s and HBM fraction on stdout")
    ap.add_argument("--graph", action="store_true",
                    help="after the timed region, also capture K further steps in one CUDA graph and time its "
                         "replay (adds a \"graph\" object; needs --no-e2e)")
    ap.add_argument("--uncompressed", action="store_true",
                    help="the cache is an uncompressed one (position IDs = cache indices); with --kv-len 49152 "
                         "it is the counterpart of the compacted 16K cache")
    ap.add_argument("--config", default=None, choices=["tiny", "qwen7b", "llama8b-ragged", "longcot", "all"],
                    help="one of the named workload configurations (ragged lengths, its own shapes and vocabulary) "
                         "instead of the headline sweep point; 'all' runs the four one after the other (a process "
                         "each) and prints a table")
    ap.add_argument("--layers", type=int, default=0, help="--config longcot: logical layers (default 32)")
    ap.add_argument("--cpu-only", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--attn-path", default="auto", choices=["auto", "mma_sync", "tcgen05", "tcgen05_keys"],
                    help="attention kernel: by shape (default), or forced for A/B timing")
    return ap.parse_args()


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- schedule (host side)

class Schedule:
    """Host-side replay of what the step loop does to the cache lengths: the
    synthetic drafts fix every sequence's accepted count, and every sequence ends
    a 512-token reasoning step and is compacted once per 128 steps (round-robin:
    one sequence per step at batch 128).  Gives the algorithmic bytes of each
    step and the compaction requests."""

    def __init__(self, cfg, lens0, n_steps):
        B = cfg.batch
        self.keep = [synth.hash_scalar(b, cfg.seed, synth.STREAM_ACCEPT) % max(cfg.n_cand, 1) + 1 for b in range(B)]
        lens = list(lens0)
        tail = MEM_TOKENS + 1
        self.len_at = []                       # lengths seen by the attention of step s
        self.seg_start = np.zeros((n_steps, B), np.int32)
        self.seg_len = np.zeros((n_steps, B), np.int32)
        for s in range(n_steps):
            self.len_at.append(list(lens))
            for b in range(B):
                lens[b] += self.keep[b]
            b = s % max(B, 128)
            if b < B and lens[b] >= SEG_LEN + tail:
                self.seg_start[s, b] = lens[b] - tail - SEG_LEN
                self.seg_len[s, b] = SEG_LEN
                lens[b] -= SEG_LEN
        self.final = lens
        self.max_len = max(max(l) for l in self.len_at + [lens])

    def kv_bytes(self, s, cfg):
        return sum(self.len_at[s]) * cfg.n_kv_heads * cfg.head_dim * 2 * 2


# --------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (read-only NVML)."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.times, self.reasons, self.max_mhz = index, [], [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.times.append(time.perf_counter())
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop_evt.wait(0.02)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# --------------------------------------------------------------------------- the oracle legs

def oracle_step_sample(cfg, n_seqs, seed_shift=0, gen_device="cpu"):
    """Builds an n_seqs-sequence sample of the workload (drawn on `gen_device`, then
    held on the host) and returns a callable running ONE whole step on it with the
    CPU oracle (as it stands)."""
    import oracle
    sub = synth.StepConfig(cfg.name + "-sample", n_seqs, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                           cfg.len_lo, cfg.len_hi, cfg.n_cand, cfg.d, cfg.rope_base, cfg.vocab,
                           headroom=SEG_LEN + 256, seed=cfg.seed + seed_shift)
    inp = synth.make_step_inputs(sub, device=gen_device)
    acc = synth.make_accept_inputs(sub, device=gen_device)
    for obj in (inp, acc):                       # everything the oracle touches lives on the host
        for k, v in vars(obj).items():
            if torch.is_tensor(v):
                setattr(obj, k, v.cpu())
    D, Hkv = sub.head_dim, sub.n_kv_heads
    kb, vb = bits(inp.k_cache), bits(inp.v_cache)
    qb, ksb, vsb = bits(inp.q), bits(inp.k_step), bits(inp.v_step)
    logits = acc.logits.numpy()
    stride = inp.n_slots * D
    state = {"len": inp.kv_len.numpy().copy()}

    def step():
        pid = np.concatenate([oracle.step_pids(inp.p0[b], sub.n_cand, sub.d) for b in range(n_seqs)])
        q_r = oracle.rope(qb, pid, sub.rope_base)
        k_r = oracle.rope(ksb, pid, sub.rope_base)
        lens = state["len"].copy()
        oracle.attn_step(kb[0], vb[0], stride, inp.kv_off.numpy(), lens, inp.q_off.numpy(), inp.n_cand.numpy(),
                         None, q_r, k_r, vsb)
        _, nm = oracle.accept(logits, sub.vocab, acc.row_off.numpy(), acc.draft.numpy())
        oracle.kv_append(kb[0], vb[0], stride, Hkv, D, inp.kv_off.numpy(), lens, k_r, vsb, inp.q_off.numpy(),
                         inp.n_cand.numpy(), nm + 1)
        seg_start = np.maximum(lens - (MEM_TOKENS + 1) - SEG_LEN, 0).astype(np.int32)
        seg_len = np.zeros(n_seqs, np.int32)
        seg_len[0] = SEG_LEN if lens[0] >= SEG_LEN + MEM_TOKENS + 1 else 0
        oracle.kv_compact(kb, vb, 1, Hkv * stride, stride, Hkv, D, inp.kv_off.numpy(), lens, seg_start, seg_len)
        # keep the sample stationary: the next call sees the original lengths again
        return n_seqs * sub.n_q

    return step, oracle.threads()


def cpu_baseline(cfg, n_seqs, gen_device, min_seconds=10.0, max_steps=8):
    """The oracle as it stands on the host cores: whole steps of a sample of the batch, repeated
    until about ten seconds of CPU work have been timed."""
    step, cores = oracle_step_sample(cfg, n_seqs, gen_device=gen_device)
    tokens, n_steps = 0, 0
    t0 = time.perf_counter()
    while n_steps < max_steps and (n_steps == 0 or time.perf_counter() - t0 < min_seconds):
        tokens += step()
        n_steps += 1
    dt = time.perf_counter() - t0
    return {"value": tokens / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_steps} whole steps (rope, attention, accept, append, compaction) of {n_seqs} of the "
                      f"{cfg.batch} sequences (L={cfg.len_lo}, {cfg.n_q} block rows each), {dt:.1f} s"}


def run_reference(args):
    """--impl reference: the fp64 oracle on the host cores, K timed steps of a one-sequence sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.sweep(args.batch, args.d, args.kv_len, True)
    step, cores = oracle_step_sample(cfg, 1)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    tokens = 0
    for _ in range(args.steps):
        tokens += step()
    dt = time.perf_counter() - t0
    val = tokens / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(cfg, args), sample="each timed step is one whole hot-path step of ONE of the "
                                                          "workload's sequences (the oracle is far too slow for the batch)"),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "each step = one whole hot-path step of 1 of the workload's sequences"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, args):
    return {"workload": f"8B-shape attention layer H_q={cfg.n_q_heads} H_kv={cfg.n_kv_heads} D={cfg.head_dim}, "
                        f"batch {cfg.batch} per GPU, {'uncompressed' if args.uncompressed else 'compacted'} KV {cfg.len_lo} "
                        f"per sequence, "
                        f"{cfg.n_cand} candidate + d={cfg.d} foresight rows per block, vocab {cfg.vocab}, 1 layer",
            "global_batch": cfg.batch * args.gpus, "kv_len": cfg.len_lo, "n_cand": cfg.n_cand, "d": cfg.d,
            "l2": ("per-step inputs (KV cache of several GB, logits) are far larger than the 126 MB L2; no flush"
                   if cfg.batch * cfg.len_lo * cfg.n_kv_heads * cfg.head_dim * 4 > 4 * 126e6 else
                   "the KV cache of this point is not much larger than the 126 MB L2: its bandwidth figure is "
                   "not an HBM figure"),
            "parallelism": f"dp{args.gpus} (independent replicas by sequence, no collective on the data path)"}


# --------------------------------------------------------------------------- multi-rank aggregation

def whole_job_throughput(units_per_rank: int, elapsed_ms_local: float, world: int, device="cpu") -> tuple:
    """Weak-scaling aggregate: every rank processed `units_per_rank` units; the job's
    time is the slowest rank's.  Returns (units/s over all ranks, max elapsed ms)."""
    elapsed = float(elapsed_ms_local)
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([elapsed], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed = float(t.item())
    return world * units_per_rank / (elapsed * 1e-3), elapsed


# --------------------------------------------------------------------------- our arm

def run_sweep(args):
    """Runs this script once per sweep point (fresh process each: the caches are up to 26 GB) and
    prints one table row per point plus the JSON lines."""
    import subprocess
    rows, lines = [], []
    print("| d | batch | cache | KV GB/step | step ms (5 Python calls) | step ms (one call) | step ms (CUDA graph) | "
          "attention µs | step tokens/s (one call) | step tokens/s (CUDA graph) | attention GB/s | of measured HBM | "
          "of 8 TB/s |")
    print("|---:|---:|---|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|", flush=True)
    for kv_len, unc in ((16384, False), (49152, True)):
        for d in range(1, 8):
            for batch in (1, 8, 32, 128):
                cmd = [sys.executable, os.path.abspath(__file__), "--batch", str(batch), "--d", str(d), "--kv-len",
                       str(kv_len), "--steps", str(args.steps if args.steps != 200 else 30), "--warmup", "3",
                       "--no-e2e", "--no-cpu-baseline", "--graph"] + (["--uncompressed"] if unc else [])
                out = subprocess.run(cmd, capture_output=True, text=True)
                if out.returncode != 0:
                    print(out.stderr[-2000:], file=sys.stderr)
                    raise SystemExit(out.returncode)
                j = json.loads(out.stdout.strip().splitlines()[-1])
                lines.append(j)
                r = j["roofline"]
                print(f"| {d} | {batch} | {'48K uncompressed' if unc else '16K compacted'} | {j['kv_gb_per_step']:.3f} | "
                      f"{j['ms_per_step']:.3f} | {j['one_call']['ms_per_step']:.3f} | {j['graph']['ms_per_step']:.3f} | "
                      f"{r['avg_launch_ms'] * 1e3:.1f} | {j['one_call']['value']:.0f} | {j['graph']['value']:.0f} | "
                      f"{r['achieved']:.0f} | "
                      f"{r['frac']:.2f}{' (L2)' if j['kv_gb_per_step'] < 0.5 else ''} | {r['frac_of_nominal_8000']:.2f} |",
                      flush=True)
    for j in lines:
        print(json.dumps(j))


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.config == "all":
        run_all_configs(args)
        return
    if args.config and args.cpu_only:
        print(json.dumps(config_cpu_baseline(CONFIGS[args.config](), args.config)), flush=True)
        return
    from paper_2604_14889_b200 import binding as ms

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    ms.memosight_attn_set_path({"auto": ms.MS_ATTN_PATH_AUTO, "mma_sync": ms.MS_ATTN_PATH_MMA_SYNC,
                                "tcgen05": ms.MS_ATTN_PATH_TCGEN05,
                                "tcgen05_keys": ms.MS_ATTN_PATH_TCGEN05_KEYS}[args.attn_path])
    if args.workload == "compress":
        run_compress(args, ms, dev, world, rank)
        return
    if args.workload == "loop":
        run_loop(args, ms, dev)
        return
    if args.workload == "cacheops":
        run_cacheops(args, ms, dev)
        return
    if args.config:
        assert world == 1, "--config is a single-GPU measurement"
        run_config(args, ms, dev)
        return
    K, W = args.steps, max(args.warmup, 3)
    cfg0 = synth.sweep(args.batch, args.d, args.kv_len, not args.uncompressed)
    n_e2e = 0 if args.no_e2e else max(1, min(args.e2e_steps, K))
    n_total = W + K
    if args.graph and n_e2e:
        raise SystemExit("--graph needs --no-e2e")
    n_sched = n_total + (3 + n_e2e if n_e2e else 0) + (2 * K + 1 if args.graph else 0)
    growth = max(3, cfg0.n_cand) * n_sched + SEG_LEN + 64
    cfg = synth.StepConfig(cfg0.name, cfg0.batch, cfg0.n_q_heads, cfg0.n_kv_heads, cfg0.head_dim, cfg0.len_lo,
                           cfg0.len_hi, cfg0.n_cand, cfg0.d, cfg0.rope_base, cfg0.vocab, headroom=growth,
                           seed=cfg0.seed + 1000 * rank)
    B, Hq, Hkv, D, nq = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_q
    T = B * nq
    inp = synth.make_step_inputs(cfg, device=dev)
    acc = synth.make_accept_inputs(cfg, device=dev)
    sched = Schedule(cfg, inp.lens, n_sched)
    seg_start = torch.from_numpy(sched.seg_start).to(dev)
    seg_len = torch.from_numpy(sched.seg_len).to(dev)
    max_kv = sched.max_len + 8
    assert max_kv <= cfg.len_hi + growth

    # a1: position IDs of every block (host integer helper of the library)
    pos = torch.from_numpy(np.concatenate(
        [ms.memosight_step_pids(inp.p0[b], cfg.n_cand, cfg.d) for b in range(B)])).to(dev)
    q_work, ks_work = inp.q.clone(), inp.k_step.clone()
    out = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((T, Hq), dtype=torch.float32, device=dev)
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    awb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    aws = torch.empty(awb, dtype=torch.uint8, device=dev)
    am = torch.empty(T, dtype=torch.int32, device=dev)
    nm = torch.empty(B, dtype=torch.int32, device=dev)
    nk = torch.empty(B, dtype=torch.int32, device=dev)
    stride = inp.n_slots * D
    ev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a_, b_ in ev_pairs:            # create the underlying cudaEvents
        a_.record()
        b_.record()

    plain = ms.attn_params(
        batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
        kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
        max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=q_work,
        k_step=ks_work, v_step=inp.v_step, out=out, lse=lse, workspace=ws, workspace_bytes=wsb)

    def step(s, ev=None):
        ms.memosight_rope_qk(q_work, ks_work, pos, T, Hq, Hkv, D, cfg.rope_base)
        if ev is not None:
            ms.memosight_attn_debug_events(ev[0].cuda_event, ev[1].cuda_event)
        ms.memosight_attn_step(plain)
        if ev is not None:
            ms.memosight_attn_debug_events(None, None)
        ms.memosight_accept(acc.logits, acc.ld_v, cfg.vocab, acc.row_off, B, T, acc.draft, am, nm, nk, aws, awb)
        ms.memosight_kv_append(inp.k_cache[0], inp.v_cache[0], stride, inp.n_slots, B, Hkv, D, inp.kv_off,
                               inp.kv_len, None, ks_work, inp.v_step, inp.q_off, inp.n_cand, nk, nq, 1)
        ms.memosight_kv_compact(inp.k_cache, inp.v_cache, 1, Hkv * stride, stride, B, Hkv, D, inp.kv_off,
                                inp.kv_len, seg_start[s], seg_len[s], None, 0, MEM_TOKENS + 1)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for s in range(W):
        step(s)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    sampler = ClockSampler(physical_gpu_index(local))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    t_wall0 = time.perf_counter()
    e0.record()
    for s in range(K):
        step(W + s, ev_pairs[s])
    e1.record()
    barrier()
    t_wall1 = time.perf_counter()
    clocks = sampler.finish()
    elapsed_ms = e0.elapsed_time(e1)
    split_ms = [a_.elapsed_time(b_) for a_, b_ in ev_pairs]
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    # the device really did the work the schedule predicts (accepted counts, appends, compactions)
    lens_after = sched.len_at[n_total] if n_sched > n_total else sched.final
    assert inp.kv_len.cpu().tolist() == lens_after, "cache lengths differ from the replayed schedule"
    assert nm.cpu().tolist() == [k - 1 for k in sched.keep]

    value, elapsed_ms = whole_job_throughput(T * K, elapsed_ms, world, dev)

    graph_info = None
    if args.graph:
        # the same K-step loop as one CUDA graph: what the step costs once the host's launch work is gone
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            for s in range(K):
                step(n_total + s)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        g0.record()
        g.replay()
        g1.record()
        barrier()
        assert ms.memosight_attn_status(ws) == ms.MS_OK
        assert inp.kv_len.cpu().tolist() == sched.len_at[n_total + K], "graph replay: cache lengths differ"
        g_value, g_ms = whole_job_throughput(T * K, g0.elapsed_time(g1), world, dev)
        graph_info = {"ms_per_step": g_ms / K, "value": g_value, "unit": UNIT,
                      "note": "K further steps captured once in a CUDA graph, one replay timed"}

    one_call = None
    if args.graph:
        # the same step queued by ONE call into the library (memosight_step_host with no host buffers):
        # what an eager step costs a caller that does not go through five Python calls
        import ctypes as C
        sp = ms.StepHostParams()
        sp.struct_size = C.sizeof(ms.StepHostParams)
        sp.attn = plain
        sp.d_pos_id = pos.data_ptr()
        sp.rope_base, sp.rope_flags, sp.vocab = cfg.rope_base, 0, cfg.vocab
        sp.ld_v, sp.d_logits, sp.d_draft = acc.ld_v, acc.logits.data_ptr(), acc.draft.data_ptr()
        sp.d_argmax, sp.d_n_match, sp.d_n_keep = am.data_ptr(), nm.data_ptr(), nk.data_ptr()
        sp.accept_workspace, sp.accept_workspace_bytes = aws.data_ptr(), awb
        sp.max_tail = MEM_TOKENS + 1
        first = n_total + K
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def call_step(s):
            sp.d_seg_start, sp.d_seg_len = seg_start[s].data_ptr(), seg_len[s].data_ptr()
            ms.memosight_step_host(sp)
        call_step(first)
        barrier()
        o0.record()
        for s in range(K):
            call_step(first + 1 + s)
        o1.record()
        barrier()
        assert ms.memosight_attn_status(ws) == ms.MS_OK
        assert inp.kv_len.cpu().tolist() == sched.final, "one-call steps: cache lengths differ"
        oc_value, oc_ms = whole_job_throughput(T * K, o0.elapsed_time(o1), world, dev)
        one_call = {"ms_per_step": oc_ms / K, "value": oc_value, "unit": UNIT,
                    "note": "K further eager steps, each queued by one memosight_step_host call without host buffers"}

    # roofline of the dominant kernel (split-KV attention): algorithmic KV bytes per launch / its duration
    kv_bytes = [sched.kv_bytes(W + s, cfg) for s in range(K)]
    step_local = T * (2 * Hq + 2 * Hkv) * D * 2
    algo_per_launch = float(np.mean(kv_bytes)) + step_local
    split_avg_ms = float(np.mean(split_ms))
    achieved = algo_per_launch / (split_avg_ms * 1e-3) / 1e9
    peak, peak_kind = peak_hbm()
    rows = nq * (Hq // Hkv)
    path = args.attn_path
    if path == "auto":
        path = "tcgen05_keys" if rows <= 64 else "tcgen05"
    kernel_name = {"tcgen05_keys": f"attn_umma_t_kernel<{(rows + 15) // 16 * 16}>", "tcgen05": "attn_umma_kernel<128>",
                   "mma_sync": f"attn_split_kernel<128,{1 if rows <= 16 else 2 if rows <= 32 else 4}>"}[path]
    roofline = {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                "frac_of_nominal_8000": achieved / 8000.0, "avg_launch_ms": split_avg_ms,
                "algorithmic_bytes_per_launch": algo_per_launch,
                "traffic": None if NCU_TRAFFIC_PER_ALGO_BYTE is None else NCU_TRAFFIC_PER_ALGO_BYTE * algo_per_launch,
                "share_of_step_time": split_avg_ms * K / elapsed_ms}

    # a long run: the attention kernel's time binned by the SM clock that was sampled while it ran
    sustained = None
    if elapsed_ms >= 1000.0 and len(sampler.samples) >= 20:
        ts, mhz = np.array(sampler.times), np.array(sampler.samples, dtype=float)
        # steps are issued back to back and the device is the bottleneck: step i ran at about this wall time
        step_t = t_wall1 - (elapsed_ms * 1e-3) * (1.0 - (np.arange(K) + 0.5) / K)
        step_mhz = mhz[np.clip(np.searchsorted(ts, step_t), 0, len(mhz) - 1)]
        bins = []
        for c in sorted(set(step_mhz.tolist())):
            sel = step_mhz == c
            ms_c = float(np.mean(np.array(split_ms)[sel]))
            by_c = float(np.mean(np.array(kv_bytes)[sel])) + step_local
            bins.append({"sm_mhz": c, "steps": int(sel.sum()), "attn_ms": ms_c, "gbs": by_c / (ms_c * 1e-3) / 1e9,
                         "attn_ms_x_ghz": ms_c * c / 1000.0})
        sustained = {"timed_seconds": elapsed_ms / 1e3, "median_sm_mhz": float(np.median(mhz)),
                     "attn_ms_x_median_ghz": split_avg_ms * float(np.median(mhz)) / 1000.0, "by_clock": bins,
                     "note": "per-step time of the split-KV kernel grouped by the SM clock sampled nearest to the step "
                             "(NVML, every 20 ms); a bandwidth that does not follow the clock is HBM-bound"}

    # ---- end to end: the step's inputs and results live in pinned host memory
    e2e = None
    if not args.no_e2e:
        # every rank runs its own end-to-end steps; the job's time is the slowest rank's
        e2e = run_e2e(ms, n_e2e, n_total, cfg, inp, acc, sched, seg_start, seg_len, ws, wsb, aws, awb, am, nm,
                      nk, out, lse, pos, max_kv)
        e2e["value"], e2e_ms = whole_job_throughput(T * n_e2e, e2e["ms_per_step"] * n_e2e, world, dev)
        e2e["ms_per_step"] = e2e_ms / n_e2e
        if world > 1:
            e2e["note"] = "every rank measured; time = max over ranks, tokens = sum over ranks"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(cfg, args),
        "attention_only_tokens_per_s": world * T / (split_avg_ms * 1e-3),
        "kv_gb_per_step": float(np.mean(kv_bytes)) / 1e9,
        "roofline": roofline, "clocks": clocks, "gpu_launches": KERNELS_PER_STEP * K,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if graph_info is not None:
        line["graph"] = graph_info
    if one_call is not None:
        line["one_call"] = one_call
    if sustained is not None:
        line["sustained"] = sustained
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            del inp, acc
            torch.cuda.empty_cache()
            line["cpu_baseline"] = cpu_baseline(cfg, args.cpu_sample_seqs, dev)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()



# --------------------------------------------------------------------------- the named configurations

CONFIGS = {"tiny": lambda: synth.TINY, "qwen7b": lambda: synth.QWEN7B,
           "llama8b-ragged": lambda: synth.LLAMA8B_RAGGED, "longcot": lambda: synth.LONGCOT}
COLD_BYTES = 512e6            # small caches rotate over copies worth at least this much, so that reads come from HBM


def config_cpu_baseline(cfg, name, min_seconds=4.0):
    """The oracle, as it stands, on the host cores: whole steps (one layer) of the configuration --
    every sequence for the first three, a seeded subset extrapolated linearly for the long-CoT one."""
    import oracle
    full = name != "longcot"
    n_seqs = cfg.batch if full else 4
    sub = synth.StepConfig(cfg.name + "-cpu", n_seqs, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.len_lo,
                           cfg.len_hi, cfg.n_cand, cfg.d, cfg.rope_base, cfg.vocab, headroom=64, seed=cfg.seed)
    lens = synth.make_lengths(cfg)[:n_seqs]
    inp = synth.make_step_inputs(sub, lens=lens)
    acc = synth.make_accept_inputs(sub)
    D, Hkv = sub.head_dim, sub.n_kv_heads
    kb, vb = bits(inp.k_cache), bits(inp.v_cache)
    qb, ksb, vsb = bits(inp.q), bits(inp.k_step), bits(inp.v_step)
    stride = inp.n_slots * D

    def step():
        pid = np.concatenate([oracle.step_pids(inp.p0[b], sub.n_cand, sub.d) for b in range(n_seqs)])
        q_r, k_r = oracle.rope(qb, pid, sub.rope_base), oracle.rope(ksb, pid, sub.rope_base)
        lens_now = inp.kv_len.numpy().copy()
        oracle.attn_step(kb[0], vb[0], stride, inp.kv_off.numpy(), lens_now, inp.q_off.numpy(), inp.n_cand.numpy(),
                         None, q_r, k_r, vsb)
        _, nm = oracle.accept(acc.logits.numpy(), sub.vocab, acc.row_off.numpy(), acc.draft.numpy())
        oracle.kv_append(kb[0], vb[0], stride, Hkv, D, inp.kv_off.numpy(), lens_now, k_r, vsb, inp.q_off.numpy(),
                         inp.n_cand.numpy(), nm + 1)

    step()
    n, t0 = 0, time.perf_counter()
    while n == 0 or (time.perf_counter() - t0 < min_seconds and n < 200):
        step()
        n += 1
    dt = (time.perf_counter() - t0) / n
    kv_bytes = sum(lens) * Hkv * D * 4
    scale = 1.0 if full else cfg.batch / n_seqs
    layers = 1 if full else 32
    out = {"value": cfg.batch * sub.n_q / (dt * scale * layers), "unit": UNIT, "cores": oracle.threads(),
           "kind": "oracle", "ms_per_layer_step": dt * 1e3 * scale, "effective_gbs": kv_bytes / dt / 1e9,
           "sample": (f"{n} whole one-layer steps (rope, attention, accept, append) of all {n_seqs} sequences"
                      if full else
                      f"{n} whole one-layer steps of {n_seqs} of the {cfg.batch} sequences; ms_per_layer_step is "
                      f"extrapolated linearly to the batch (x{scale:.0f}), value to 32 layers -- extrapolated")}
    return out


def run_all_configs(args):
    import subprocess
    lines = []
    for name in ("tiny", "qwen7b", "llama8b-ragged", "longcot"):
        cmd = [sys.executable, os.path.abspath(__file__), "--config", name, "--steps", str(args.steps), "--warmup",
               str(args.warmup)] + (["--no-cpu-baseline"] if args.no_cpu_baseline else [])
        out = subprocess.run(cmd, capture_output=True, text=True)
        if out.returncode != 0:
            print(out.stderr[-3000:], file=sys.stderr)
            raise SystemExit(out.returncode)
        lines.append(json.loads(out.stdout.strip().splitlines()[-1]))
    print("| config | batch | layers | rows | KV GB/step | step ms | step ms (CUDA graph) | step tokens/s (CUDA graph) | attention ms/step | attention GB/s | "
          "of measured HBM | of 8 TB/s | L2-warm attention GB/s | rope µs | accept µs | append µs | compaction event µs "
          "(amortised µs/step) | oracle tokens/s (cores) |")
    print("|---|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|---:|")
    for j in lines:
        r, c, pt = j["roofline"], j["config"], j["parts"]
        cb = j.get("cpu_baseline")
        warm = j.get("l2_warm")
        print(f"| {c['name']} | {c['global_batch']} | {c['layers']} | {c['rows']} | {j['kv_gb_per_step']:.4f} | "
              f"{j['ms_per_step']:.4f} | {j['graph']['ms_per_step']:.4f} | {j['graph']['value']:.0f} | "
              f"{r['avg_launch_ms'] * r['launches_per_step']:.4f} | "
              f"{r['achieved']:.0f} | {r['frac']:.2f} | {r['frac_of_nominal_8000']:.2f} | "
              f"{'' if warm is None else format(warm['achieved'], '.0f')} | {pt['rope_us']:.1f} | {pt['accept_us']:.1f} | "
              f"{pt['append_us']:.1f} | {pt['compaction_event_us']:.1f} ({pt['compaction_amortised_us_per_step']:.2f}) | "
              f"{'' if cb is None else format(cb['value'], '.1f') + ' (' + str(cb['cores']) + ')'} |")
    for j in lines:
        print(json.dumps(j))


def run_config(args, ms, dev):
    """One named configuration, device-resident.  A step = for every layer: RoPE of the block at its
    position IDs -> step attention -> append of the accepted candidates; once per step the greedy
    accept.  The long-CoT configuration stacks 32 logical layers over as many physical cache layers
    as fit in 70 % of the free memory (each layer is far larger than the L2, so cycling over them
    reuses nothing), issues its attention through the stacked-layer entry (and, for comparison, layer
    by layer) and times its compaction event (every sequence, every layer, 512 -> 170 + <o>)
    separately: the event happens once per 512 generated tokens and is reported amortised.  The two
    small configurations rotate over enough copies of their cache to exceed 512 MB, so that their
    bandwidth is an HBM figure; the figure with one copy (L2-warm) is reported beside it."""
    name = args.config
    cfg0 = CONFIGS[name]()
    K, W = args.steps if args.steps != 200 else 50, max(args.warmup, 3)
    B, Hq, Hkv, D, nq = cfg0.batch, cfg0.n_q_heads, cfg0.n_kv_heads, cfg0.head_dim, cfg0.n_q
    T = B * nq
    lens0 = synth.make_lengths(cfg0)
    n_rounds = 5                                    # whole, graph, parts, split kernel, per-layer (or L2-warm)
    growth = cfg0.n_cand * (W + K + 2) * (n_rounds + 1) + 64
    if name == "longcot":
        growth = max(growth, SEG_LEN + MEM_TOKENS + 64)
    layer_bytes = 2 * Hkv * (sum(lens0) + B * growth) * D * 2
    NL = (args.layers or 32) if name == "longcot" else 1
    if name == "longcot":
        free, _ = torch.cuda.mem_get_info()
        n_phys = max(1, min(NL, int(0.7 * free // layer_bytes)))
    elif layer_bytes < COLD_BYTES:
        n_phys = int(-(-COLD_BYTES // layer_bytes))
    else:
        n_phys = 1
    cfg = synth.StepConfig(cfg0.name, B, Hq, Hkv, D, cfg0.len_lo, cfg0.len_hi, cfg0.n_cand, cfg0.d, cfg0.rope_base,
                           cfg0.vocab, n_layers=n_phys, headroom=growth, seed=cfg0.seed)
    inp = synth.make_step_inputs(cfg, device=dev, lens=lens0)
    acc = synth.make_accept_inputs(cfg, device=dev)
    keep = [synth.hash_scalar(b, cfg.seed, synth.STREAM_ACCEPT) % max(cfg.n_cand, 1) + 1 for b in range(B)]
    stride, lstride = inp.n_slots * D, Hkv * inp.n_slots * D
    max_kv = max(lens0) + growth
    pos1 = np.concatenate([ms.memosight_step_pids(inp.p0[b], cfg.n_cand, cfg.d) for b in range(B)])
    pos = torch.from_numpy(np.tile(pos1, NL)).to(dev)
    # step tensors of every logical layer (the same values in every layer: the generator's draw of one layer)
    q_all = inp.q.unsqueeze(0).repeat(NL, 1, 1, 1).contiguous()
    ks_all = inp.k_step.unsqueeze(0).repeat(NL, 1, 1, 1).contiguous()
    vs_all = inp.v_step.unsqueeze(0).repeat(NL, 1, 1, 1).contiguous()
    out_all = torch.empty((NL, T, Hq, D), dtype=torch.bfloat16, device=dev)
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    awb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    aws = torch.empty(awb, dtype=torch.uint8, device=dev)
    am = torch.empty(T, dtype=torch.int32, device=dev)
    nm = torch.empty(B, dtype=torch.int32, device=dev)
    nk = torch.empty(B, dtype=torch.int32, device=dev)
    q_ls, ks_ls = T * Hq * D, T * Hkv * D
    state = {"step": 0}

    def params(phys, logical):
        return ms.attn_params(
            batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[phys], v_cache=inp.v_cache[phys],
            kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
            max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=q_all[logical],
            k_step=ks_all[logical], v_step=vs_all[logical], out=out_all[logical], lse=None, workspace=ws,
            workspace_bytes=wsb)

    # stacked issue: runs of consecutive physical layers, the logical layers cycling over them
    runs = []
    l = 0
    while l < NL:
        n = min(n_phys, NL - l)
        runs.append((l, n))
        l += n
    run_params = [params(0, l0) for l0, _ in runs]
    layer_params = {}

    def attn(stacked, ev=None, rotate=True):
        """The attention of one step: all logical layers."""
        if NL == 1:
            phys = (state["step"] % n_phys) if rotate else 0
            key = ("one", phys)
            if key not in layer_params:
                layer_params[key] = params(phys, 0)
            if ev:
                ms.memosight_attn_debug_events(ev[0].cuda_event, ev[1].cuda_event)
            ms.memosight_attn_step(layer_params[key])
            if ev:
                ms.memosight_attn_debug_events(None, None)
            return 1
        n_launch = 0
        if stacked:
            for i, (l0, n) in enumerate(runs):
                if ev:
                    ms.memosight_attn_debug_events(ev[i][0].cuda_event, ev[i][1].cuda_event)
                ms.memosight_attn_step_layers(run_params[i], n, lstride, q_ls, ks_ls, q_ls)
                n_launch += 1
        else:
            for lg in range(NL):
                key = ("layer", lg)
                if key not in layer_params:
                    layer_params[key] = params(lg % n_phys, lg)
                if ev:
                    ms.memosight_attn_debug_events(ev[lg][0].cuda_event, ev[lg][1].cuda_event)
                ms.memosight_attn_step(layer_params[key])
                n_launch += 1
        if ev:
            ms.memosight_attn_debug_events(None, None)
        return n_launch

    def rope():
        ms.memosight_rope_qk(q_all, ks_all, pos, NL * T, Hq, Hkv, D, cfg.rope_base)

    def accept():
        ms.memosight_accept(acc.logits, acc.ld_v, cfg.vocab, acc.row_off, B, T, acc.draft, am, nm, nk, aws, awb)

    def append(rotate=True):
        if NL == 1:
            phys = (state["step"] % n_phys) if rotate else 0
            ms.memosight_kv_append(inp.k_cache[phys], inp.v_cache[phys], stride, inp.n_slots, B, Hkv, D, inp.kv_off,
                                   inp.kv_len, None, ks_all[0], vs_all[0], inp.q_off, inp.n_cand, nk, nq, 1)
            return
        for lg in range(NL):
            # (layers that share a physical cache layer append to the same slots: the bytes moved are what counts)
            ms.memosight_kv_append(inp.k_cache[lg % n_phys], inp.v_cache[lg % n_phys], stride, inp.n_slots, B, Hkv, D,
                                   inp.kv_off, inp.kv_len, None, ks_all[lg], vs_all[lg], inp.q_off, inp.n_cand, nk, nq,
                                   1 if lg == NL - 1 else 0)

    def step(stacked=True, rotate=True):
        rope()
        attn(stacked, rotate=rotate)
        accept()
        append(rotate)
        state["step"] += 1

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t_host = time.perf_counter()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        host_ms = (time.perf_counter() - t_host) * 1e3
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n, host_ms / n

    lens_now = list(lens0)

    def advance(n):
        for b in range(B):
            lens_now[b] += keep[b] * n

    def kv_bytes_mean(n):
        """Algorithmic K/V bytes per step (all layers), averaged over the next n steps."""
        tot = 0
        for s in range(n):
            tot += sum(L + keep[b] * s for b, L in enumerate(lens_now))
        return tot / n * Hkv * D * 4 * NL

    for _ in range(W):
        step()
    advance(W)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    sampler = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))))
    sampler.start()
    # ---- round 1: whole steps
    kv_whole = kv_bytes_mean(K)
    step_ms, host_ms = timed(step, K)
    advance(K)
    clocks = sampler.finish()
    assert inp.kv_len.cpu().tolist() == lens_now, "cache lengths differ from the replayed schedule"
    assert nm.cpu().tolist() == [k - 1 for k in keep]
    # ---- the same K steps captured once in a CUDA graph, one replay timed (what the kernels cost when
    #      the host's launch work is gone; small configurations are bound by it otherwise)
    side = torch.cuda.Stream()
    gr = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(gr, stream=side):
        for _ in range(K):
            step()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    g0.record()
    gr.replay()
    g1.record()
    torch.cuda.synchronize()
    advance(K)
    assert inp.kv_len.cpu().tolist() == lens_now, "graph replay: cache lengths differ"
    graph_ms = g0.elapsed_time(g1) / K
    del gr
    # ---- round 2: the parts, each bracketed by events (this serialises the launches a little)
    n_ev = len(runs) if NL > 1 else 1
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
           for _ in range(K)]
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K)]
    for row in evs:
        for a_, b_ in row:
            a_.record()
            b_.record()
    for s_ in range(K):
        m = marks[s_]
        m[0].record()
        rope()
        m[1].record()
        attn(True)
        m[2].record()
        accept()
        m[3].record()
        append()
        m[4].record()
        state["step"] += 1
    torch.cuda.synchronize()
    advance(K)
    # ---- round 2b: the split-KV kernel alone (events recorded by the library right around it; no other
    #      event in the step, so that nothing but the kernel lies between the two)
    kv_parts = kv_bytes_mean(K)
    for s_ in range(K):
        rope()
        attn(True, ev=evs[s_] if NL > 1 else evs[s_][0])
        accept()
        append()
        state["step"] += 1
    torch.cuda.synchronize()
    advance(K)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    part = lambda i: float(np.mean([m[i].elapsed_time(m[i + 1]) for m in marks])) * 1e3
    split_ms = [sum(a_.elapsed_time(b_) for a_, b_ in row) for row in evs]        # per step, all launches
    attn_ms = float(np.mean(split_ms))
    step_local = T * (2 * Hq + 2 * Hkv) * D * 2 * NL
    algo = kv_parts + step_local
    achieved = algo / (attn_ms * 1e-3) / 1e9
    peak, peak_kind = peak_hbm()
    rows = nq * (Hq // Hkv)
    if D == 128 and rows <= 64:
        kernel = f"attn_umma_t_kernel<{(rows + 15) // 16 * 16}>"
    elif D == 64:
        kernel = f"attn_split_kernel<64,{1 if rows <= 16 else 2 if rows <= 32 else 4}>"
    else:
        kernel = "attn_umma_big_kernel"
    cold = n_phys > 1 or layer_bytes > 4 * 126e6
    roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak,
                "peak_source": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                "frac_of_nominal_8000": achieved / 8000.0, "avg_launch_ms": attn_ms / n_ev, "launches_per_step": n_ev,
                "algorithmic_bytes_per_launch": algo / n_ev, "traffic": None,
                "share_of_step_time": attn_ms / (part(0) + part(1) + part(2) + part(3)) * 1e3,
                "reads_from": "HBM" if cold else "L2 (the cache is not much larger than the 126 MB L2)"}
    # ---- round 3: layer by layer (long-CoT) or L2-warm (one copy of a small cache)
    per_layer, l2_warm = None, None
    if NL > 1:
        ev_l = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(NL)]
                for _ in range(K)]
        for row in ev_l:
            for a_, b_ in row:
                a_.record()
                b_.record()
        kv_l = kv_bytes_mean(K)
        t_ms, h_ms = timed(lambda: step(stacked=False), K)
        advance(K)
        # the same once more with events around every layer's split kernel
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        host_issue = []
        for s_ in range(min(K, 10)):
            rope()
            t_h = time.perf_counter()
            attn(False, ev=ev_l[s_])
            host_issue.append((time.perf_counter() - t_h) * 1e6 / NL)
            accept()
            append()
            state["step"] += 1
        torch.cuda.synchronize()
        advance(min(K, 10))
        dev_us = float(np.mean([a_.elapsed_time(b_) for row in ev_l[:min(K, 10)] for a_, b_ in row])) * 1e3
        ideal_us = kv_l / NL / (achieved * 1e9) * 1e6      # what a layer's bytes take at the stacked launch's rate
        per_layer = {"step_ms_layer_by_layer": t_ms, "step_ms_stacked": step_ms,
                     "split_kernel_us_per_layer": dev_us,
                     "device_fixed_us_per_layer_launch": dev_us - ideal_us,
                     "host_issue_us_per_layer_call": float(np.mean(host_issue)),
                     "note": "device fixed cost = a layer's own launch minus its bytes at the stacked launch's "
                             "bandwidth; host = wall time of one memosight_attn_step call through the Python binding"}
    elif n_phys > 1:
        e_w = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for a_, b_ in e_w:
            a_.record()
            b_.record()
        kv_w = kv_bytes_mean(K)
        for s_ in range(K):
            rope()
            attn(True, ev=e_w[s_], rotate=False)
            accept()
            append(rotate=False)
            state["step"] += 1
        torch.cuda.synchronize()
        advance(K)
        w_ms = float(np.mean([a_.elapsed_time(b_) for a_, b_ in e_w]))
        l2_warm = {"achieved": (kv_w + step_local) / (w_ms * 1e-3) / 1e9, "unit": "GB/s", "avg_launch_ms": w_ms,
                   "note": "the same cache copy every step: it stays in the L2, not an HBM figure"}
    # ---- the compaction event: every sequence ends a 512-token step (64 -> 8 + <o> for the tiny configuration)
    seg, mem = (64, 8) if name == "tiny" else (SEG_LEN, MEM_TOKENS)
    tail = mem + 1
    lens_dev = inp.kv_len.clone()
    can = all(L >= seg + tail for L in lens_now)
    comp_us, comp_bytes = 0.0, 0
    if can:
        seg_len = torch.full((B,), seg, dtype=torch.int32, device=dev)
        seg_start = (lens_dev - tail - seg).to(torch.int32)
        ts = []
        for _ in range(5):
            inp.kv_len.copy_(lens_dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ms.memosight_kv_compact(inp.k_cache, inp.v_cache, n_phys if NL > 1 else 1, lstride, stride, B, Hkv, D,
                                    inp.kv_off, inp.kv_len, seg_start, seg_len, None, 0, tail)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        lay = n_phys if NL > 1 else 1
        comp_us = float(np.median(ts)) * 1e3 * (NL / lay)
        comp_bytes = 2 * tail * Hkv * D * 2 * 2 * B * NL
        assert inp.kv_len.cpu().tolist() == [L - seg for L in lens_now]
        inp.kv_len.copy_(lens_dev)
    gen_per_step = float(np.mean(keep))
    parts = {"rope_us": part(0), "attn_us": part(1), "accept_us": part(2), "append_us": part(3),
             "compaction_event_us": comp_us, "compaction_event_bytes": comp_bytes,
             "compaction_event_gbs": (comp_bytes / (comp_us * 1e-6) / 1e9) if comp_us else None,
             "compaction_amortised_us_per_step": comp_us * gen_per_step / seg,
             "compaction_amortised_us_per_generated_token": comp_us / seg,
             "note": f"event = all {B} sequences evict a {seg}-token step and keep {mem} memory tokens + <o>, all "
                     f"{NL} layers" + (f" (measured on {n_phys} physical layers, scaled)" if NL > 1 else "") +
                     f"; once per {seg} generated tokens of a sequence, {gen_per_step:.2f} tokens per step"}
    line = {
        "metric": METRIC_CONFIG, "value": T / (step_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"{cfg0.name}: H_q={Hq} H_kv={Hkv} D={D}, batch {B}, compacted KV "
                               f"{cfg0.len_lo}..{cfg0.len_hi} (uniform from the seed; mean {np.mean(lens0):.0f}), "
                               f"{cfg0.n_cand} candidate + d={cfg0.d} foresight rows per block, vocab {cfg0.vocab}, "
                               f"{NL} logical layer(s) over {n_phys} physical cache layer(s)",
                   "name": name, "global_batch": B, "layers": NL, "physical_layers": n_phys, "rows": rows,
                   "n_cand": cfg0.n_cand, "d": cfg0.d,
                   "l2": ("every layer's cache is far larger than the 126 MB L2; no flush" if layer_bytes > 4 * 126e6 else
                          f"the cache of one layer ({layer_bytes / 1e6:.2f} MB) would sit in the L2: the steps rotate over "
                          f"{n_phys} copies ({n_phys * layer_bytes / 1e6:.0f} MB) so that reads come from HBM")},
        "kv_gb_per_step": kv_whole / 1e9, "host_issue_ms_per_step": host_ms,
        "graph": {"ms_per_step": graph_ms, "value": T / (graph_ms * 1e-3), "unit": UNIT,
                  "note": "K further steps captured once in a CUDA graph, one replay timed"},
        "attention_only_tokens_per_s": T / (attn_ms * 1e-3), "roofline": roofline, "parts": parts, "clocks": clocks,
        "gpu_launches": (1 + len(runs) + 1 + NL) * K if NL > 1 else 4 * K,
    }
    if per_layer:
        line["per_layer"] = per_layer
    if l2_warm:
        line["l2_warm"] = l2_warm
    if not args.no_cpu_baseline:
        del inp, acc, q_all, ks_all, vs_all, out_all
        torch.cuda.empty_cache()
        cb = config_cpu_baseline(cfg0, name)
        if name in ("tiny", "qwen7b"):
            import subprocess
            env = dict(os.environ, OMP_NUM_THREADS="1")
            o = subprocess.run([sys.executable, os.path.abspath(__file__), "--config", name, "--cpu-only"], env=env,
                               capture_output=True, text=True)
            if o.returncode == 0:
                one = json.loads(o.stdout.strip().splitlines()[-1])
                cb["single_thread_value"] = one["value"]
        line["cpu_baseline"] = cb
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- the loop of Algorithm 1

class DeviceToy:
    """synth.ToyModel evaluated on the device with tensor operations (the same integer hashes, so
    it predicts exactly what the host version predicts): stands in for the language model so that
    the decoding loop runs without the host in the data path.  Not part of the library."""

    def __init__(self, m, dev):
        self.m, self.dev = m, dev

    def _umod(self, h, n):
        # h holds the bits of an unsigned 64-bit hash in an int64 lane: its value modulo n
        r = torch.remainder(h, n)
        return torch.where(h < 0, torch.remainder(r + ((1 << 64) % n), n), r)

    def truth(self, b, pid, pid0):
        m = self.m
        key = b * 1000003 + pid
        t = self._umod(synth.hash64(key, m.seed, synth.STREAM_TOY_TOKEN), m.vocab - 5)
        t = torch.where(self._umod(synth.hash64(key, m.seed, synth.STREAM_TOY_DELIM), m.step_len) == 0,
                        torch.full_like(t, m.tok_delim), t)
        return torch.where(pid - pid0 >= m.eos_after, torch.full_like(t, m.tok_eos), t)

    def predict(self, b, tok, pid, pid0):
        m = self.m
        t = self.truth(b, pid + 1, pid0)
        miss = (tok == m.tok_f) & (self._umod(synth.hash64(b * 1000003 + pid, m.seed, synth.STREAM_TOY_HIT), 100)
                                   >= m.hit_pct)
        t = torch.where(miss, torch.remainder(t + 1, m.vocab - 5), t)
        return torch.where(tok == m.tok_m, self._umod(synth.hash64(pid, m.seed, synth.STREAM_TOY_TOKEN), m.vocab - 5), t)


class PlantedLogits:
    """fp32 [rows][V] seeded noise with one winner per row planted 40 above it; the winners move
    from step to step by undoing the last plant and making the next (four small index kernels)."""

    def __init__(self, rows, V, seed, dev):
        self.buf = synth.normal_f32(rows * V, seed, synth.STREAM_LOGITS, 2.0, device=dev).view(rows, V)
        self.rows = torch.arange(rows, device=dev)
        self.col = torch.zeros(rows, dtype=torch.int64, device=dev)
        self.noise = self.buf[self.rows, self.col].clone()

    def plant(self, col):
        self.buf[self.rows, self.col] = self.noise          # undo
        self.col.copy_(col)
        self.noise.copy_(self.buf[self.rows, self.col])
        self.buf[self.rows, self.col] = self.noise + 40.0


def run_loop(args, ms, dev):
    """Secondary workload: the whole inference loop of Algorithm 1 on device-resident state --
    Predict+Verify blocks until a step ends, then the compression block (memory tokens + <o>
    through the large-block kernel), append and eviction -- with a toy model as the logits source.
    Per iteration the host reads one 16-byte summary (rows, live sequences, sequences waiting for
    compression); everything else stays on the device.  Every iteration is one CUDA graph replay
    (a step graph or a compression graph, each ending with the plan of the next block)."""
    import ctypes as C
    assert int(os.environ.get("WORLD_SIZE", "1")) == 1
    Hq, Hkv, D, NL = 32, 8, 128, max(1, args.layers or 1)
    V, L0, max_mem, max_out = 128256, 1024, 64, 1500
    base = 5.0e5
    results = []
    grid = [(B, d, c) for B in ((args.batch,) if args.batch != 128 else (1, 64)) for c in (3, 5) for d in range(0, 5)]
    if args.d != 3:
        grid = [(B, d, c) for (B, d, c) in grid if d == args.d]
    for (B, d, c) in grid:
        m = synth.ToyModel(vocab=V, hit_pct=60, step_len=23, eos_after=1200, seed=0x70F0 + B)
        toy = DeviceToy(m, dev)
        pid0 = [L0 + 3 * b for b in range(B)]
        cap = L0 + 1400
        n_slots = B * cap
        stride, lstride = n_slots * D, Hkv * n_slots * D
        k_cache = synth.normal_bf16(NL * lstride, 11, synth.STREAM_KCACHE, device=dev).view(NL, Hkv, n_slots, D)
        v_cache = synth.normal_bf16(NL * lstride, 11, synth.STREAM_VCACHE, device=dev).view(NL, Hkv, n_slots, D)
        i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=dev)
        g_off = torch.tensor([b * cap for b in range(B)], dtype=torch.int64, device=dev)
        g_len, g_cap = i32([L0] * B), i32([cap] * B)
        first = [m.truth(b, pid0[b], pid0[b]) for b in range(B)]
        cand = torch.zeros((B, d + 1), dtype=torch.int32, device=dev)
        cand[:, 0] = i32(first)
        st_t = dict(kv_len=g_len, pos_next=i32(pid0), seg_start=i32([L0] * B), seg_n=i32([0] * B), seg_pid0=i32(pid0),
                    cand=cand, n_cand=i32([1] * B), flags=i32([0] * B),
                    out_tok=torch.zeros((B, max_out), dtype=torch.int32, device=dev), n_out=i32([0] * B))
        st = ms.decode_state(B, d, c, max_out, max_mem, m.tok_f, m.tok_m, m.tok_o, m.tok_delim, m.tok_eos, **st_t)
        nq_s, nq_c = 2 * d + 1, max_mem + 1
        Ts, Tc = B * nq_s, B * nq_c
        q_off, n_blk = torch.zeros(B + 1, dtype=torch.int32, device=dev), torch.zeros(B, dtype=torch.int32, device=dev)
        row_tok, pos_id, draft = (torch.zeros(Tc, dtype=torch.int32, device=dev) for _ in range(3))
        n_keep, seg_s, seg_l = (torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(3))
        summary = torch.zeros(4, dtype=torch.int32, device=dev)
        h_summary = torch.zeros(4, dtype=torch.int32).pin_memory()
        scratch = torch.empty(ms.memosight_decode_scratch_bytes(B), dtype=torch.uint8, device=dev)
        am, nm = torch.zeros(Tc + 1, dtype=torch.int32, device=dev), torch.zeros(B, dtype=torch.int32, device=dev)
        am_o = torch.zeros(B, dtype=torch.int32, device=dev)
        overflow = torch.zeros(1, dtype=torch.int32, device=dev)
        aws = torch.empty(ms.memosight_accept_workspace_bytes(max(Ts, B), V), dtype=torch.uint8, device=dev)
        # q / k / v of the blocks: fixed seeded tensors (what the attention computes does not steer the toy model)
        q = synth.normal_bf16(NL * Tc * Hq * D, 12, synth.STREAM_Q, device=dev).view(NL, Tc, Hq, D)
        ks = synth.normal_bf16(NL * Tc * Hkv * D, 12, synth.STREAM_KSTEP, device=dev).view(NL, Tc, Hkv, D)
        vs = synth.normal_bf16(NL * Tc * Hkv * D, 12, synth.STREAM_VSTEP, device=dev).view(NL, Tc, Hkv, D)
        out = torch.empty((NL, Tc, Hq, D), dtype=torch.bfloat16, device=dev)
        max_kv = cap
        wsb_s = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq_s)
        wsb_c = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq_c)
        ws_s = torch.empty(wsb_s, dtype=torch.uint8, device=dev)
        ws_c = torch.empty(wsb_c, dtype=torch.uint8, device=dev)
        lg_s, lg_c = PlantedLogits(Ts, V, 13, dev), PlantedLogits(B, V, 14, dev)
        pid0_t = torch.tensor(pid0, dtype=torch.int64, device=dev)
        rows_s = torch.arange(Ts, device=dev, dtype=torch.int32)
        row_off_c = torch.arange(B + 1, dtype=torch.int32, device=dev)
        draft_c = torch.full((B,), -1, dtype=torch.int32, device=dev)
        nm_c = torch.zeros(B, dtype=torch.int32, device=dev)
        n_iter_cap = 4000
        len_log = torch.zeros((n_iter_cap, B), dtype=torch.int32, device=dev)

        def attn_params(layer, ws, wsb, max_nq, T):
            return ms.attn_params(batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=k_cache[layer],
                                  v_cache=v_cache[layer], kv_head_stride=stride, n_slots=n_slots, kv_off=g_off,
                                  kv_len=g_len, max_kv_len=max_kv, max_nq=max_nq, q_off=q_off, n_cand=n_blk, anchor=None,
                                  total_rows=T, sm_scale=0.0, q=q[layer], k_step=ks[layer], v_step=vs[layer],
                                  out=out[layer], lse=None, workspace=ws, workspace_bytes=wsb)
        ap_s = [attn_params(l, ws_s, wsb_s, nq_s, Ts) for l in range(NL)]
        ap_c = [attn_params(l, ws_c, wsb_c, nq_c, Tc) for l in range(NL)]

        def plan():
            ms.memosight_decode_plan(st, q_off, n_blk, row_tok, pos_id, draft, summary, scratch)
            h_summary.copy_(summary, non_blocking=True)

        def step_body():
            # one Predict+Verify block of every live sequence (rows beyond q_off[B] hold stale, harmless data)
            for l in range(NL):
                ms.memosight_rope_qk(q[l], ks[l], pos_id, Ts, Hq, Hkv, D, base)
                ms.memosight_attn_step(ap_s[l])
            seq = torch.searchsorted(q_off[1:], rows_s, right=True).clamp_(max=B - 1).to(torch.int64)
            win = toy.predict(seq, row_tok[:Ts].to(torch.int64), pos_id[:Ts].to(torch.int64), pid0_t[seq])
            lg_s.plant(win)
            ms.memosight_accept(lg_s.buf, V, V, q_off, B, Ts, draft, am, nm, None, aws, aws.numel())
            ms.memosight_decode_commit(st, q_off, am, nm, n_keep)
            for l in range(NL):
                ms.memosight_kv_append(k_cache[l], v_cache[l], stride, n_slots, B, Hkv, D, g_off, g_len, g_cap, ks[l],
                                       vs[l], q_off, n_blk, n_keep, nq_s, l == NL - 1, overflow)
            plan()

        def compress_body():
            ms.memosight_decode_plan_compress(st, q_off, n_blk, row_tok, pos_id, n_keep, seg_s, seg_l, summary, scratch)
            for l in range(NL):
                ms.memosight_rope_qk(q[l], ks[l], pos_id, Tc, Hq, Hkv, D, base)
                ms.memosight_attn_step(ap_c[l])
            # the model's head is only needed on <o>, the last row of each block: one logits row per sequence
            last = (q_off[1:].to(torch.int64) - 1).clamp_(min=0)
            bs = torch.arange(B, device=dev, dtype=torch.int64)
            win = toy.predict(bs, row_tok[last].to(torch.int64), pos_id[last].to(torch.int64), pid0_t)
            lg_c.plant(win)
            ms.memosight_accept(lg_c.buf, V, V, row_off_c, B, B, draft_c, am_o, nm_c, None, aws, aws.numel())
            # to the block's last row, where commit_compress reads it (sequences without a block: a spare slot)
            am[torch.where(q_off[1:] > q_off[:-1], last, torch.full_like(last, Tc))] = am_o
            for l in range(NL):
                ms.memosight_kv_append(k_cache[l], v_cache[l], stride, n_slots, B, Hkv, D, g_off, g_len, g_cap, ks[l],
                                       vs[l], q_off, n_blk, n_keep, nq_c, l == NL - 1, overflow)
            ms.memosight_kv_compact(k_cache, v_cache, NL, lstride, stride, B, Hkv, D, g_off, g_len, seg_s, seg_l, None,
                                    0, max_mem + 1)
            ms.memosight_decode_commit_compress(st, q_off, am)
            plan()

        # warm both bodies up on a scratch copy of the state?  They mutate it, so instead: run the
        # first iterations eagerly (they are part of the decode), then capture and replay
        side = torch.cuda.Stream()
        graphs = {}

        def run(body, name, use_graph):
            if not use_graph:
                body()
                return
            if name not in graphs:
                g = torch.cuda.CUDAGraph()
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=side):
                    body()
                graphs[name] = g
            graphs[name].replay()

        plan()
        torch.cuda.synchronize()
        steps = comps = iters = 0
        eager_iters = {"step": 0, "compress": 0}
        t_start = None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_timed_steps = n_timed_comps = 0
        tokens_at_start = 0
        while True:
            T, live, pending, _ = h_summary.tolist()
            if T == 0 and pending == 0:
                break
            name = "compress" if pending else "step"
            use_graph = eager_iters[name] >= 2            # two eager runs of a body first (set-up, caches)
            if not use_graph:
                eager_iters[name] += 1
            elif t_start is None and all(v >= 2 for v in eager_iters.values()) and len(graphs) == 2:
                torch.cuda.synchronize()
                t_start = time.perf_counter()
                e0.record()
                tokens_at_start = int(st_t["n_out"].sum().item())
            run(compress_body if pending else step_body, name, use_graph)
            len_log[min(iters, n_iter_cap - 1)].copy_(g_len)
            torch.cuda.synchronize()                      # the 16-byte summary of the next block is on the host
            if t_start is not None:
                if pending:
                    n_timed_comps += 1
                else:
                    n_timed_steps += 1
            steps += 0 if pending else 1
            comps += 1 if pending else 0
            iters += 1
            assert iters < n_iter_cap
        e1.record()
        torch.cuda.synchronize()
        wall = time.perf_counter() - (t_start or time.perf_counter())
        assert int(overflow.item()) == 0, "a sequence outgrew its cache region"
        # the accepted tokens are what plain token-by-token greedy decoding with the same model gives
        n_out = st_t["n_out"].cpu().tolist()
        out_tok = st_t["out_tok"].cpu()
        for b in range(min(B, 4)):
            want, pid, tok = [], pid0[b], first[b]
            while len(want) < max_out:
                want.append(tok)
                if tok == m.tok_eos:
                    break
                if tok == m.tok_delim:
                    tok, pid = m.predict(b, m.tok_o, pid + 1, pid0[b]), pid + 2
                else:
                    tok, pid = m.predict(b, tok, pid, pid0[b]), pid + 1
            assert out_tok[b, :min(n_out[b], max_out)].tolist() == want[:min(n_out[b], max_out)], f"sequence {b} is not greedy"
        total_tokens = int(sum(min(n, max_out) for n in n_out))
        timed_tokens = total_tokens - tokens_at_start
        lens = len_log[:iters].float().mean(dim=1).cpu().tolist()
        pick = [lens[int(i * (len(lens) - 1) / 9)] for i in range(10)] if lens else []
        line = {
            "metric": "Predict+Verify steps/s of the whole inference loop (Algorithm 1) on device-resident state",
            "value": n_timed_steps / wall if wall > 0 else 0.0, "unit": "steps/s", "n_gpus": 1,
            "steps": n_timed_steps, "warmup": steps - n_timed_steps, "ms_per_step": wall / max(n_timed_steps, 1) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"loop: 8B-shape attention ({NL} layer(s)), batch {B}, d={d} foresight tokens, "
                                   f"compression ratio c={c}, prompt cache {L0}, toy model (60 % foresight hit rate, "
                                   f"reasoning steps of ~23 tokens, <eos> after 1200 positions), vocab {V}",
                       "global_batch": B, "d": d, "c": c, "layers": NL},
            "accepted_tokens_per_s": timed_tokens / wall if wall > 0 else 0.0,
            "tokens_per_step": timed_tokens / max(n_timed_steps, 1) / B,
            "compressions": comps, "timed_compressions": n_timed_comps, "iterations": iters,
            "device_ms_timed": e0.elapsed_time(e1) if t_start is not None else None,
            "mean_cache_length_over_time": [round(x, 1) for x in pick],
            "peak_mean_cache_length": max(lens) if lens else None,
            "uncompressed_length_at_end": L0 + float(np.mean([min(n, max_out) for n in n_out])),
            "note": "one CUDA graph replay and one 16-byte device-to-host read per iteration; wall-clock time",
        }
        results.append(line)
        print(json.dumps(line), flush=True)
        del k_cache, v_cache, q, ks, vs, out, lg_s, lg_c, graphs
        torch.cuda.empty_cache()
    print("| batch | d | c | steps/s | accepted tokens/s | tokens per step and sequence | ms per step | compressions | "
          "mean cache length start -> peak -> end | uncompressed length at the end |")
    print("|---:|---:|---:|---:|---:|---:|---:|---:|---|---:|")
    for j in results:
        c_ = j["config"]
        tr = j["mean_cache_length_over_time"]
        print(f"| {c_['global_batch']} | {c_['d']} | {c_['c']} | {j['value']:.0f} | {j['accepted_tokens_per_s']:.0f} | "
              f"{j['tokens_per_step']:.2f} | {j['ms_per_step']:.3f} | {j['compressions']} | "
              f"{tr[0]:.0f} -> {j['peak_mean_cache_length']:.0f} -> {tr[-1]:.0f} | {j['uncompressed_length_at_end']:.0f} |")


# --------------------------------------------------------------------------- the small HBM-bound kernels

def run_cacheops(args, ms, dev):
    """Secondary workload: the HBM-bound kernels around the attention, each timed alone on the
    long-CoT shapes -- the compaction event (512 -> 170 + <o>, every sequence, every layer), an
    eviction by keep list (every third of the last 3000 entries dropped: short runs; and a
    window-plus-prefix keep set: long runs), RoPE and append of the compression block's 171 tokens
    per sequence, and the split-KV merge of a small batch.  Bytes are the algorithmic ones: moved
    entries x 2 (read + write) for the cache operations, one read + one write of q and k for RoPE."""
    B = args.batch if args.batch != 128 else 64
    NL = args.layers or 4
    Hq, Hkv, D = 32, 8, 128
    reps = max(3, min(args.steps, 20))
    cfg = synth.StepConfig("cacheops", B, Hq, Hkv, D, 9000, 12000, 4, 4, 5e5, 100, n_layers=NL, seed=78)
    inp = synth.make_step_inputs(cfg, device=dev)
    stride, lstride = inp.n_slots * D, Hkv * inp.n_slots * D
    len0 = inp.kv_len.clone()
    peak, peak_kind = peak_hbm()

    def timeit(f, reset):
        for _ in range(2):
            reset()
            f()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            reset()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            f()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.median(ts))

    rows = []

    def report(name, kernel, ms_, nbytes, what):
        gbs = nbytes / (ms_ * 1e-3) / 1e9
        rows.append({"name": name, "kernel": kernel, "us": ms_ * 1e3, "algorithmic_bytes": nbytes, "achieved": gbs,
                     "unit": "GB/s", "frac": gbs / peak, "frac_of_nominal_8000": gbs / 8000.0, "what": what})

    reset = lambda: inp.kv_len.copy_(len0)
    # ---- compaction event
    tail = MEM_TOKENS + 1
    seg_start = (len0 - tail - SEG_LEN).to(torch.int32)
    seg_len = torch.full((B,), SEG_LEN, dtype=torch.int32, device=dev)
    t = timeit(lambda: ms.memosight_kv_compact(inp.k_cache, inp.v_cache, NL, lstride, stride, B, Hkv, D, inp.kv_off,
                                               inp.kv_len, seg_start, seg_len, None, 0, tail), reset)
    report("compaction event", "kv_compact_move_kernel", t, 2 * tail * Hkv * D * 2 * 2 * B * NL,
           f"{B} sequences x {NL} layers evict a {SEG_LEN}-token step, {tail} entries slide down")
    # ---- eviction by keep list
    lens = len0.cpu().tolist()
    for label, keep_fn in (("every third of the last 3000 dropped", lambda L: [i for i in range(L) if i < L - 3000 or i % 3]),
                           ("first 384 + last 4096 kept", lambda L: list(range(384)) + list(range(L - 4096, L)))):
        keep = [keep_fn(L) for L in lens]
        max_keep = max(len(k) for k in keep)
        ki = torch.zeros((B, max_keep), dtype=torch.int32)
        for b in range(B):
            ki[b, :len(keep[b])] = torch.tensor(keep[b], dtype=torch.int32)
        ki = ki.to(dev)
        nk = torch.tensor([len(k) for k in keep], dtype=torch.int32, device=dev)
        t = timeit(lambda: ms.memosight_kv_gather(inp.k_cache, inp.v_cache, NL, lstride, stride, B, Hkv, D, inp.kv_off,
                                                  inp.kv_len, ki, max_keep, nk, max_keep), reset)
        moved = sum(sum(1 for j, i in enumerate(k) if i != j) for k in keep)
        report(f"keep-list eviction ({label})", "kv_gather_kernel", t, moved * NL * 2 * Hkv * D * 2 * 2,
               f"{moved} entries per layer change their slot")
    reset()
    # ---- RoPE and append of the compression blocks
    nq = tail
    T = B * nq
    q = synth.normal_bf16(T * Hq * D, 5, synth.STREAM_Q, device=dev).view(T, Hq, D)
    k = synth.normal_bf16(T * Hkv * D, 5, synth.STREAM_KSTEP, device=dev).view(T, Hkv, D)
    pos = torch.from_numpy(np.concatenate([
        np.concatenate([ms.memosight_upl_pids(3 * L, SEG_LEN, 3)[:MEM_TOKENS], [ms.memosight_out_pid(3 * L, SEG_LEN)]])
        for L in lens]).astype(np.int32)).to(dev)
    t = timeit(lambda: ms.memosight_rope_qk(q, k, pos, T, Hq, Hkv, D, 5e5), lambda: None)
    report("RoPE of the compression blocks", "rope_qk_kernel", t, T * (Hq + Hkv) * D * 2 * 2,
           f"{T} tokens at UPL position IDs, in place")
    q_off = torch.arange(0, T + 1, nq, dtype=torch.int32, device=dev)
    n_c = torch.full((B,), nq, dtype=torch.int32, device=dev)
    # (the append keeps the lengths: bump_len = 0, so every repetition writes the same slots)
    t = timeit(lambda: ms.memosight_kv_append(inp.k_cache[0], inp.v_cache[0], stride, inp.n_slots, B, Hkv, D,
                                              inp.kv_off, inp.kv_len, None, k, k, q_off, n_c, n_c, nq, 0), lambda: None)
    report("append of the compression blocks (one layer)", "kv_append_kernel", t, T * Hkv * D * 2 * 2 * 2,
           f"{nq} rows per sequence, K and V")
    # ---- the merge of a small batch (every unit cut across many CTAs)
    Bs, d = 2, 7
    scfg = synth.sweep(Bs, d, 16384, True)
    sinp = synth.make_step_inputs(scfg, device=dev)
    Ts = Bs * scfg.n_q
    out = torch.empty((Ts, Hq, D), dtype=torch.bfloat16, device=dev)
    wsb = ms.memosight_attn_workspace_bytes(Bs, Hq, Hkv, D, 16384, scfg.n_q)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    ap = ms.attn_params(batch=Bs, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=sinp.k_cache[0],
                        v_cache=sinp.v_cache[0], kv_head_stride=sinp.n_slots * D, n_slots=sinp.n_slots,
                        kv_off=sinp.kv_off, kv_len=sinp.kv_len, max_kv_len=16384, max_nq=scfg.n_q, q_off=sinp.q_off,
                        n_cand=sinp.n_cand, anchor=None, total_rows=Ts, sm_scale=0.0, q=sinp.q, k_step=sinp.k_step,
                        v_step=sinp.v_step, out=out, lse=None, workspace=ws, workspace_bytes=wsb)
    ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    for e in ev:
        e.record()
    ms.memosight_attn_debug_events(ev[0].cuda_event, ev[1].cuda_event)
    t_all = timeit(lambda: ms.memosight_attn_step(ap), lambda: None)
    torch.cuda.synchronize()
    t_split = ev[0].elapsed_time(ev[1])
    ms.memosight_attn_debug_events(None, None)
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    rows_p = scfg.n_q * (Hq // Hkv)
    report("split-KV merge of a small batch (call minus split kernel)", "attn_merge_kernel", max(t_all - t_split, 1e-6),
           n_sm * rows_p * (D + 2) * 4 + Ts * Hq * D * 2,
           f"batch {Bs}, d={d}: {Bs * Hkv} units x {rows_p} rows, one partial per CTA ({n_sm}); latency-bound")
    line = {"metric": "GB/s of the HBM-bound kernels around the attention (algorithmic bytes / device time)",
            "unit": "GB/s", "n_gpus": 1, "steps": reps, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"cache operations on long-CoT shapes: batch {B}, {NL} layers, caches 9000..12000, "
                                   f"8B shape", "global_batch": B, "layers": NL},
            "peak": peak, "peak_source": f"{peak_kind} copy bandwidth", "kernels": rows}
    print(json.dumps(line), flush=True)
    print("| operation | kernel | µs | algorithmic MB | GB/s | of measured HBM | of 8 TB/s |")
    print("|---|---|---:|---:|---:|---:|---:|")
    for r in rows:
        print(f"| {r['name']} | {r['kernel']} | {r['us']:.1f} | {r['algorithmic_bytes'] / 1e6:.1f} | {r['achieved']:.0f} | "
              f"{r['frac']:.2f} | {r['frac_of_nominal_8000']:.2f} |")


def peak_tensor():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return float(j["bf16_tflops_sustained"]), float(j["bf16_tflops"]), "measured"
    except Exception:
        return 1400.0, 1590.0, "fallback"


def run_compress(args, ms, dev, world, rank):
    """Secondary workload: the compression event of long-CoT serving.  Every sequence has just
    finished a 512-token reasoning step; the 170 memory tokens + <o> are forwarded as one causal
    block against the cache (which still holds the verbose step), appended, and the step is
    evicted.  One "step" = that event for the whole batch, one layer; the cache length is put
    back before every event so that all events are the stated workload.  Compute-bound: the
    roofline is the bf16 tensor peak."""
    assert world == 1, "the compress workload is a single-GPU measurement"
    K, W = args.steps, max(args.warmup, 3)
    B = args.batch if args.batch != 128 else 64
    L0, nq, Hq, Hkv, D = args.kv_len, MEM_TOKENS + 1, 32, 8, 128
    growth = nq + SEG_LEN + 64
    cfg = synth.StepConfig("compress", B, Hq, Hkv, D, L0, L0, nq, 0, 5.0e5, 1024, headroom=growth, seed=0x5EED0004)
    inp = synth.make_step_inputs(cfg, device=dev)
    T = B * nq
    # a1: UPL position IDs of the memory tokens and the PID of <o>, per sequence (host integer helpers)
    pos = []
    for b in range(B):
        rho = inp.p0[b]
        pos.append(np.concatenate([ms.memosight_upl_pids(rho, SEG_LEN, 3)[:MEM_TOKENS],
                                   [ms.memosight_out_pid(rho, SEG_LEN)]]).astype(np.int32))
    pos = torch.from_numpy(np.concatenate(pos)).to(dev)
    q_work, ks_work = inp.q.clone(), inp.k_step.clone()
    out = torch.empty((T, Hq, D), dtype=torch.bfloat16, device=dev)
    max_kv = L0 + growth
    wsb = ms.memosight_attn_workspace_bytes(B, Hq, Hkv, D, max_kv, nq)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    stride = inp.n_slots * D
    keep = torch.full((B,), nq, dtype=torch.int32, device=dev)
    seg_len = torch.full((B,), SEG_LEN, dtype=torch.int32, device=dev)
    seg_start = torch.empty(B, dtype=torch.int32, device=dev)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a_, b_ in evs:
        a_.record()
        b_.record()

    len0 = inp.kv_len.clone()

    def step(ev=None):
        inp.kv_len.copy_(len0)                       # every event starts from the same cache of L0 entries;
        seg_start.copy_(inp.kv_len)                  # the finished step starts where the cache ended ...
        inp.kv_len.add_(SEG_LEN)                     # ... and its 512 entries are in the cache
        ms.memosight_rope_qk(q_work, ks_work, pos, T, Hq, Hkv, D, cfg.rope_base)
        if ev is not None:
            ms.memosight_attn_debug_events(ev[0].cuda_event, ev[1].cuda_event)
        ms.memosight_attn_step(
            batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
            kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len, max_kv_len=max_kv,
            max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None, total_rows=T, sm_scale=0.0, q=q_work,
            k_step=ks_work, v_step=inp.v_step, out=out, lse=None, workspace=ws, workspace_bytes=wsb)
        if ev is not None:
            ms.memosight_attn_debug_events(None, None)
        ms.memosight_kv_append(inp.k_cache[0], inp.v_cache[0], stride, inp.n_slots, B, Hkv, D, inp.kv_off,
                               inp.kv_len, None, ks_work, inp.v_step, inp.q_off, inp.n_cand, keep, nq, 1)
        ms.memosight_kv_compact(inp.k_cache, inp.v_cache, 1, Hkv * stride, stride, B, Hkv, D, inp.kv_off,
                                inp.kv_len, seg_start, seg_len, None, 0, nq)

    for _ in range(W):
        step()
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    sampler = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    e0.record()
    for s_ in range(K):
        step(evs[s_])
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.finish()
    elapsed_ms = e0.elapsed_time(e1)
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    assert inp.kv_len.cpu().tolist() == [L0 + nq] * B
    attn_ms = float(np.mean([a_.elapsed_time(b_) for a_, b_ in evs]))
    l_mid = L0 + SEG_LEN
    flops = 4.0 * B * Hq * D * nq * (l_mid + (nq + 1) / 2.0)       # visible keys: cache + causal half
    sustained, burst, kind = peak_tensor()
    achieved = flops / (attn_ms * 1e-3) / 1e12
    line = {
        "metric": "memory tokens/s (compression event: forward of 170 memory tokens + <o>, append, eviction of a "
                  "512-token step; 8B shape)", "value": T * K / (elapsed_ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": K, "warmup": W, "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"compression event, 8B-shape layer H_q={Hq} H_kv={Hkv} D={D}, batch {B}, cache "
                               f"{L0} + a {SEG_LEN}-token step (the same at every event), block of {nq} causal tokens, 1 layer",
                   "global_batch": B, "kv_len": L0, "block": nq,
                   "l2": "K/V of one sequence-layer (69 MB) is re-read by the 6 row tiles of a KV head, mostly "
                         "from L2; no flush"},
        "roofline": {"bound": "tensor", "kernel": "attn_umma_big_kernel", "achieved": achieved, "peak": sustained,
                     "peak_source": f"{kind} bf16 GEMM, sustained ({burst:.0f} burst)", "unit": "TFLOP/s",
                     "frac": achieved / sustained, "avg_launch_ms": attn_ms, "algorithmic_flops_per_launch": flops,
                     "traffic": None, "share_of_step_time": attn_ms * K / elapsed_ms},
        "clocks": clocks, "gpu_launches": 8 * K,
    }
    print(json.dumps(line), flush=True)


def run_e2e(ms, n_e2e, first, cfg, inp, acc, sched, seg_start, seg_len, ws, wsb, aws, awb, am, nm, nk, out, lse,
            pos, max_kv):
    """Same step through memosight_step_host: inputs from / results to pinned host memory each step."""
    import ctypes as C
    B, Hq, Hkv, D, nq = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_q
    T = B * nq
    h_q = inp.q.cpu().pin_memory()
    h_ks = inp.k_step.cpu().pin_memory()
    h_vs = inp.v_step.cpu().pin_memory()
    h_pos = pos.cpu().pin_memory()
    h_logits = acc.logits.cpu().pin_memory()
    h_draft = acc.draft.cpu().pin_memory()
    h_out = torch.empty((T, Hq, D), dtype=torch.bfloat16).pin_memory()
    h_am = torch.empty(T, dtype=torch.int32).pin_memory()
    h_nm = torch.empty(B, dtype=torch.int32).pin_memory()
    d_q, d_ks, d_vs = torch.empty_like(inp.q), torch.empty_like(inp.k_step), torch.empty_like(inp.v_step)
    d_pos, d_draft = torch.empty_like(pos), torch.empty_like(acc.draft)
    d_logits = torch.empty_like(acc.logits)
    # the cache keeps evolving from where the device-resident loop left it: rows `first`.. of the schedule
    stride = inp.n_slots * D
    p = ms.StepHostParams()
    p.struct_size = C.sizeof(ms.StepHostParams)
    p.attn = ms.attn_params(
        batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, k_cache=inp.k_cache[0], v_cache=inp.v_cache[0],
        kv_head_stride=stride, n_slots=inp.n_slots, kv_off=inp.kv_off, kv_len=inp.kv_len,
        max_kv_len=max_kv, max_nq=nq, q_off=inp.q_off, n_cand=inp.n_cand, anchor=None,
        total_rows=T, sm_scale=0.0, q=d_q, k_step=d_ks, v_step=d_vs, out=out, lse=lse, workspace=ws,
        workspace_bytes=wsb)
    p.h_q, p.h_k_step, p.h_v_step = h_q.data_ptr(), h_ks.data_ptr(), h_vs.data_ptr()
    p.h_pos_id, p.d_pos_id = h_pos.data_ptr(), d_pos.data_ptr()
    p.rope_base, p.rope_flags, p.vocab = cfg.rope_base, 0, cfg.vocab
    p.h_logits, p.ld_v, p.d_logits = h_logits.data_ptr(), acc.ld_v, d_logits.data_ptr()
    p.h_draft, p.d_draft = h_draft.data_ptr(), d_draft.data_ptr()
    p.d_argmax, p.d_n_match, p.d_n_keep = am.data_ptr(), nm.data_ptr(), nk.data_ptr()
    p.accept_workspace, p.accept_workspace_bytes = aws.data_ptr(), awb
    p.max_tail = MEM_TOKENS + 1
    p.h_out, p.h_argmax, p.h_n_match = h_out.data_ptr(), h_am.data_ptr(), h_nm.data_ptr()

    def host_step(s):
        p.d_seg_start, p.d_seg_len = seg_start[s].data_ptr(), seg_len[s].data_ptr()
        ms.memosight_step_host(p)
        torch.cuda.synchronize()          # the host reads the step's result before the next step

    for i in range(3):
        host_step(first + i)
    t0 = time.perf_counter()
    for i in range(n_e2e):
        host_step(first + 3 + i)
    dt = time.perf_counter() - t0
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    assert h_nm.tolist() == [k - 1 for k in sched.keep]
    assert inp.kv_len.cpu().tolist() == sched.final, "cache lengths differ from the replayed schedule"
    h2d = (h_q.numel() + h_ks.numel() + h_vs.numel()) * 2 + h_pos.numel() * 4 + h_logits.numel() * 4 \
        + h_draft.numel() * 4
    d2h = h_out.numel() * 2 + h_am.numel() * 4 + h_nm.numel() * 4
    return {"value": T * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "steps": n_e2e, "ms_per_step": dt / n_e2e * 1e3,
            "call": "memosight_step_host (pinned host buffers; the logits copy runs on the library's copy stream beside the "
                    "attention; host sync after every step)"}


if __name__ == "__main__":
    main()
