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
SEG_LEN, MEM_TOKENS = 512, 170          # one compaction: 512-token step -> 170 memory tokens + <o>
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes the split kernel moved per algorithmic byte in the ncu capture summarised in
# profiles/attn_umma_t_kernel_sweep_b32_L16384.md (batch 32; scaled by the bytes streamed).
NCU_TRAFFIC_PER_ALGO_BYTE = 1.011
KERNELS_PER_STEP = 9                    # rope 1, attention 2, accept 2, append 2, compaction 2


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
    ap.add_argument("--workload", default="step", choices=["step", "compress"],
                    help="step: the Predict+Verify step the headline metric is quoted on (default); "
                         "compress: the compression event (forward of the memory tokens + <o>, append, eviction)")
    ap.add_argument("--sweep", action="store_true",
                    help="the foresight/batch/cache-length sweep (8B shape): one device-resident run per point, "
                         "a table of KV bytes read, step tokens/s and HBM fraction on stdout")
    ap.add_argument("--graph", action="store_true",
                    help="after the timed region, also capture K further steps in one CUDA graph and time its "
                         "replay (adds a \"graph\" object; needs --no-e2e)")
    ap.add_argument("--uncompressed", action="store_true",
                    help="the cache is an uncompressed one (position IDs = cache indices); with --kv-len 49152 "
                         "it is the counterpart of the compacted 16K cache")
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
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
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
        "config": workload_config(cfg, args),
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
    print("| d | batch | cache | KV GB/step | step ms | step ms (CUDA graph) | attention µs | step tokens/s | "
          "step tokens/s (CUDA graph) | attention GB/s | of measured HBM | of 8 TB/s |")
    print("|---:|---:|---|---:|---:|---:|---:|---:|---:|---:|---:|---:|", flush=True)
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
                      f"{j['ms_per_step']:.3f} | {j['graph']['ms_per_step']:.3f} | {r['avg_launch_ms'] * 1e3:.1f} | "
                      f"{j['value']:.0f} | {j['graph']['value']:.0f} | {r['achieved']:.0f} | "
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
    K, W = args.steps, max(args.warmup, 3)
    cfg0 = synth.sweep(args.batch, args.d, args.kv_len, not args.uncompressed)
    n_e2e = 0 if args.no_e2e else max(1, min(args.e2e_steps, K))
    n_total = W + K
    if args.graph and n_e2e:
        raise SystemExit("--graph needs --no-e2e")
    n_sched = n_total + (3 + n_e2e if n_e2e else 0) + (K + 1 if args.graph else 0)
    growth = 3 * n_sched + SEG_LEN + 64
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
    e0.record()
    for s in range(K):
        step(W + s, ev_pairs[s])
    e1.record()
    barrier()
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

    # ---- end to end: the step's inputs and results live in pinned host memory
    e2e = None
    if not args.no_e2e and rank == 0:
        e2e = run_e2e(ms, n_e2e, n_total, cfg, inp, acc, sched, seg_start, seg_len, ws, wsb, aws, awb, am, nm,
                      nk, out, lse, pos, max_kv)
    if world > 1 and e2e is not None:
        e2e["note"] = "measured on rank 0 only, scaled by the number of ranks"
        e2e["value"] *= world

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
