"""GPU parity of every attention kernel behind memosight_attn_step, each forced in turn
through memosight_attn_set_path and compared with the CPU oracle on the same inputs:
the mma.sync kernel, the rows-on-lanes tcgen05 kernel, the keys-on-lanes tcgen05 kernel
and the general ALU kernel.  Covers the paths' private machinery: partial units cut
across CTAs (many tiles per CTA, buffer-ring wrap-around), the step-local mask, ragged
tails, and the rare branch that moves a row's reference maximum in mid-stream."""
import numpy as np
import pytest
import torch

from harness import assert_attn_close, check_attn, gpu_attn, oracle_attn, random_problem
from paper_2604_14889_b200 import binding as ms

pytestmark = pytest.mark.gpu

PATHS = {"mma_sync": ms.MS_ATTN_PATH_MMA_SYNC, "tcgen05_rows": ms.MS_ATTN_PATH_TCGEN05,
         "tcgen05_keys": ms.MS_ATTN_PATH_TCGEN05_KEYS, "general": ms.MS_ATTN_PATH_GENERAL}
FAST = ["mma_sync", "tcgen05_rows", "tcgen05_keys"]


@pytest.fixture
def force_path():
    def _set(name):
        ms.memosight_attn_set_path(PATHS[name])
    yield _set
    ms.memosight_attn_set_path(ms.MS_ATTN_PATH_AUTO)


def test_set_path_returns_previous_and_rejects_unknown():
    assert ms.memosight_attn_set_path(ms.MS_ATTN_PATH_TCGEN05) == ms.MS_ATTN_PATH_AUTO
    assert ms.memosight_attn_set_path(ms.MS_ATTN_PATH_AUTO) == ms.MS_ATTN_PATH_TCGEN05
    assert ms.lib().memosight_attn_set_path(99) == ms.MS_ERR_INVALID_ARG
    assert ms.memosight_attn_set_path(ms.MS_ATTN_PATH_AUTO) == ms.MS_ATTN_PATH_AUTO


@pytest.mark.parametrize("path", FAST)
@pytest.mark.parametrize("G,Hkv,nq", [(1, 3, 8), (4, 2, 6), (7, 1, 6), (8, 1, 8), (4, 2, 14), (2, 2, 16)])
def test_ragged_lengths_across_tile_edges(force_path, path, G, Hkv, nq):
    force_path(path)
    lens = [0, 1, 15, 16, 17, 127, 128, 129, 255, 256, 700, 1, 1500]
    B = len(lens)
    n_q = [1 + (3 * b) % nq for b in range(B)]
    n_q[5] = nq
    n_c = [(b * 5) % (n_q[b] + 1) for b in range(B)]
    check_attn(random_problem(B, G * Hkv, Hkv, 128, lens, n_q, n_c, seed=31 * G + nq, anchors=True),
               f"{path} ragged G={G} nq={nq}")


@pytest.mark.parametrize("path", FAST)
@pytest.mark.parametrize("tiles_per_cta", [2, 5, 7, 13])
def test_many_tiles_per_cta_wrap_the_buffer_rings(force_path, path, tiles_per_cta):
    # one KV head, one sequence: the 148 persistent CTAs get exactly `tiles_per_cta` tiles each,
    # every unit is cut across CTAs and merged, and the K/V rings wrap (5..12 buffers)
    force_path(path)
    n_ctas = torch.cuda.get_device_properties(0).multi_processor_count
    L = n_ctas * 128 * tiles_per_cta - 128
    check_attn(random_problem(1, 4, 1, 128, [L], [6], [3], seed=tiles_per_cta), f"{path} k={tiles_per_cta}")


@pytest.mark.parametrize("path", FAST)
def test_units_whole_and_partial_in_one_launch(force_path, path):
    force_path(path)
    lens = [2048 + 37 * i for i in range(48)]
    check_attn(random_problem(48, 32, 8, 128, lens, [14] * 48, [7] * 48, seed=12), f"{path} batch 48 rows 56")
    check_attn(random_problem(48, 32, 8, 128, lens, [2] * 48, [1] * 48, seed=13), f"{path} batch 48 rows 8")


@pytest.mark.parametrize("path", FAST + ["general"])
@pytest.mark.parametrize("D", [64, 128])
def test_head_dim_64_and_128(force_path, path, D):
    force_path(path)      # a path that does not cover the shape falls back to the automatic choice
    check_attn(random_problem(4, 8, 2, D, [513, 77, 128, 4000], [6] * 4, [3] * 4, seed=9 + D), f"{path} D={D}")


@pytest.mark.parametrize("path", FAST)
def test_peaked_scores_and_garbage_tail(force_path, path):
    force_path(path)
    check_attn(random_problem(4, 8, 2, 128, [513, 2000, 90, 128], [6] * 4, [3] * 4, seed=5, qscale=6.0),
               f"{path} peaked")
    P = random_problem(3, 8, 2, 128, [100, 257, 1], [6] * 3, [3] * 3, seed=13, headroom=140)
    want, want_lse = oracle_attn(P)
    for b in range(3):
        lo = int(P["kv_off"][b]) + P["lens"][b]
        P["k_cache"][:, lo:lo + 140] = float("nan")
        P["v_cache"][:, lo:lo + 140] = float("inf")
    out, lse = gpu_attn(P)
    assert_attn_close(out, lse, want, want_lse, f"{path} garbage tail")


def _plant_needle(P, b, kvh, pos, q_row, strength, in_step=False):
    """Key `pos` of sequence b becomes a multiple of one query row, scaled so that this row's
    score on it is `strength` nats (softmax scale 1/sqrt(D))."""
    q = P["q"][q_row[0], q_row[1]].float()
    k = (strength * np.sqrt(P["D"]) * q / q.norm() ** 2).to(torch.bfloat16)
    if in_step:
        P["k_step"][int(P["q_off"][b]) + pos, kvh] = k
    else:
        P["k_cache"][kvh, int(P["kv_off"][b]) + pos] = k


@pytest.mark.parametrize("path", FAST)
def test_reference_maximum_moves_in_mid_stream(force_path, path):
    # A key far into the cache outscores everything before it by > 2^48 (and a later one again by
    # as much): the kernels that exponentiate against a fixed row reference must rescale their
    # accumulators there.  Needles sit in the second tile, deep in the stream, in the last ragged
    # tile and among the block's own keys.
    force_path(path)
    L = [148 * 128 * 3 + 77, 900, 130]
    P = random_problem(3, 8, 2, 128, L, [6, 6, 6], [3, 3, 6], seed=77)
    r0 = [int(x) for x in P["q_off"][:3]]
    _plant_needle(P, 0, 0, 130, (r0[0] + 0, 0), 45.0)            # row 0 of head 0: grows once ...
    _plant_needle(P, 0, 0, 30000, (r0[0] + 0, 0), 90.0)          # ... and again, 45 nats higher
    _plant_needle(P, 0, 1, L[0] - 3, (r0[0] + 4, 5), 50.0)       # KV head 1, last (ragged) tile, foresight row
    _plant_needle(P, 1, 0, 899, (r0[1] + 2, 1), 100.0)          # 144 log2 units in one go: must rescale
    _plant_needle(P, 2, 1, 2, (r0[2] + 5, 6), 55.0, in_step=True)  # a candidate key seen by candidate row 5
    out, lse = check_attn(P, f"{path} moving reference")
    # the needle rows really are dominated by one key
    want, _ = oracle_attn(P)
    v_needle = P["v_cache"][0, int(P["kv_off"][0]) + 30000].double().numpy()
    assert np.abs(want[r0[0], 0] - v_needle).max() < 1e-6


@pytest.mark.parametrize("path", FAST)
def test_deterministic(force_path, path):
    force_path(path)
    P = random_problem(5, 32, 8, 128, [5000, 130, 2048, 3, 900], [6] * 5, [3] * 5, seed=12)
    a, la = gpu_attn(P)
    b, lb = gpu_attn(P)
    assert torch.equal(a, b) and torch.equal(la, lb)


def test_paths_agree_with_each_other(force_path):
    P = random_problem(6, 32, 8, 128, [3000, 130, 2048, 1, 900, 0], [8] * 6, [4] * 6, seed=21)
    outs = {}
    for path in FAST + ["general"]:
        force_path(path)
        outs[path], _ = gpu_attn(P)
    ref = outs["general"].float()
    for path in FAST:
        assert (outs[path].float() - ref).abs().max() <= 2e-2, path


@pytest.mark.parametrize("G,nq", [(7, 12), (8, 16), (8, 9)])
def test_forced_rows_path_never_outgrows_the_workspace(force_path, G, nq):
    # head_dim 128 with 65..128 packed rows: the automatic choice is the large-block kernel, whose
    # workspace is small; the rows-on-lanes kernel needs two partial slots per CTA.  Forced with
    # the workspace the library asks for, the call must fall back (and stay inside the workspace:
    # the harness checks a canary behind it); forced with a workspace large enough for it, the
    # rows-on-lanes kernel itself runs.  Both agree with the oracle.
    lens = [3000, 130, 0, 515]
    P = random_problem(4, G, 1, 128, lens, [nq, nq - 3, nq, 1], [nq // 2, 2, nq, 1], seed=G * 100 + nq, anchors=True)
    force_path("tcgen05_rows")
    check_attn(P, f"forced rows-on-lanes, default workspace G={G} nq={nq}")
    want, want_lse = oracle_attn(P)
    out, lse = gpu_attn(P, ws_min_bytes=64 << 20)
    assert_attn_close(out, lse, want, want_lse, f"forced rows-on-lanes, large workspace G={G} nq={nq}")


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    # The failure path of the bounded waits, without anything failing: one warp waits 3 ms on a
    # barrier at which nobody arrives; the wait gives up, the kernel returns, the status word says so
    # once, and the next attention call on the same workspace is served as usual.
    P = random_problem(2, 8, 2, 128, [300, 40], [6, 6], [3, 3], seed=2)
    ws_bytes = ms.memosight_attn_workspace_bytes(2, 8, 2, 128, 300, 6)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    assert ms.memosight_attn_status(ws) == ms.MS_OK
    ms.memosight_debug_wait_timeout(ws, 3000)
    assert ms.memosight_attn_status(ws) == ms.MS_ERR_DEVICE_TIMEOUT
    assert ms.memosight_attn_status(ws) == ms.MS_OK              # reported once, then cleared
    with pytest.raises(ms.MemosightError):
        ms.memosight_debug_wait_timeout(ws, 5_000_000)           # limits beyond a second are refused
    # the limit of the real kernels is a launch parameter too
    prev = ms.memosight_debug_set_wait_limit_us(2_000_000)
    try:
        assert ms.memosight_debug_set_wait_limit_us(0) == 2_000_000
        check_attn(P, "after a timed-out wait")
    finally:
        ms.memosight_debug_set_wait_limit_us(prev)
    assert ms.memosight_debug_set_wait_limit_us(0) == prev


def test_general_path_many_rows_and_clamped_lengths(force_path):
    # more than 65535 block rows in one call (head_dim 32 only has the general kernel)
    B, nq = 4200, 16
    lens = [(3 * b) % 7 for b in range(B)]
    P = random_problem(B, 2, 1, 32, lens, [nq] * B, [(b % (nq + 1)) for b in range(B)], seed=88, headroom=1)
    assert P["T"] > 65535
    check_attn(P, "general path, 67200 rows")
    # a device length above the host's bound is clamped to the bound, on this path as on the others:
    # the result is that of a cache of max_kv_len entries
    force_path("general")
    Q = random_problem(3, 8, 2, 128, [300, 40, 129], [6, 6, 6], [3, 3, 3], seed=89, headroom=64)
    want, want_lse = oracle_attn(Q)
    # (the harness passes max(lens) = 300 as max_kv_len and the tensor below as the device lengths)
    out, lse = gpu_attn(dict(Q, kv_len=torch.tensor([300 + 40, 40, 129], dtype=torch.int32)))
    assert_attn_close(out, lse, want, want_lse, "kv_len above max_kv_len is clamped")
