"""The N>1 host logic of bench.py on CPU: two gloo ranks, max-over-ranks timing,
whole-job (weak scaling) throughput, per-rank seeds; and the reference arm's
rank rule (rank 0 prints, the others exit without work)."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 25.0            # rank 1 is the slow one
    value, elapsed = bench.whole_job_throughput(1000, local_ms, world)
    q.put((rank, value, elapsed))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_units():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, elapsed in got:
        assert elapsed == 25.0
        assert abs(value - 2 * 1000 / 0.025) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, elapsed = bench.whole_job_throughput(500, 4.0, 1)
    assert elapsed == 4.0 and value == 500 / 0.004


def test_schedule_replay_is_consistent():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2604_14889_b200 import synth
    # every sequence is compacted once per 128 steps: one per step at batch 128, one step in 16 at batch 8
    for B, n_steps in ((8, 300), (128, 140), (200, 210)):
        cfg = synth.sweep(B, 3, 4096, True)
        sch = bench.Schedule(cfg, [4096] * B, n_steps)
        assert all(1 <= k <= 3 for k in sch.keep)
        lens = [4096] * B
        events = 0
        for s in range(n_steps):
            assert sch.len_at[s] == lens
            lens = [l + k for l, k in zip(lens, sch.keep)]
            b = s % max(B, 128)
            if b < B:
                assert sch.seg_len[s].sum() == sch.seg_len[s, b] == 512
                assert sch.seg_start[s, b] == lens[b] - 171 - 512
                lens[b] -= 512
                events += 1
            else:
                assert sch.seg_len[s].sum() == 0
        assert events == sum(1 for s in range(n_steps) if s % max(B, 128) < B)
        assert sch.final == lens


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--kv-len", "1024", "--batch", "2"], env=env, capture_output=True,
                       text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
