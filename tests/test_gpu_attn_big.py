"""GPU parity of the large-block attention (17..256 new tokens per sequence): the compression
pass of the method forwards the l memory tokens and <o> of a finished reasoning step as one
causal block against the compacted cache (Sec. 2.1.2; Algorithm 1).  Same call
(memosight_attn_step, max_nq > 16), same oracle, same tolerance as the step blocks."""
import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from harness import check_attn, gpu_attn, oracle_attn, random_problem
from paper_2604_14889_b200 import binding as ms

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,kw", [
    ("G4 one row tile and a bit", dict(B=1, Hq=4, Hkv=1, D=128, lens=[300], n_q_list=[40], n_c_list=[40], seed=1)),
    ("AMA(512,3)+1 tokens", dict(B=2, Hq=8, Hkv=2, D=128, lens=[1000, 77], n_q_list=[172, 33], n_c_list=[172, 20],
                                 seed=2, anchors=True)),
    ("G7: 18 tokens per row tile", dict(B=2, Hq=28, Hkv=4, D=128, lens=[513, 128], n_q_list=[50, 17],
                                        n_c_list=[50, 17], seed=3)),
    ("G1: two step-key tiles", dict(B=1, Hq=2, Hkv=2, D=128, lens=[700], n_q_list=[200], n_c_list=[200], seed=4)),
    ("G16: 8 tokens per row tile", dict(B=1, Hq=16, Hkv=1, D=128, lens=[257], n_q_list=[20], n_c_list=[12], seed=5,
                                        anchors=True)),
    ("empty cache", dict(B=1, Hq=8, Hkv=2, D=128, lens=[0], n_q_list=[172], n_c_list=[172], seed=6)),
    ("long cache, units cut across CTAs", dict(B=1, Hq=32, Hkv=8, D=128, lens=[20000], n_q_list=[172],
                                               n_c_list=[172], seed=7)),
    ("small, large, empty and maximal blocks", dict(B=4, Hq=8, Hkv=2, D=128, lens=[900, 5000, 0, 130],
                                                    n_q_list=[3, 172, 0, 256], n_c_list=[2, 172, 0, 100], seed=8,
                                                    anchors=True)),
    ("peaked scores", dict(B=2, Hq=8, Hkv=2, D=128, lens=[3000, 640], n_q_list=[100, 64], n_c_list=[100, 64], seed=9,
                           qscale=6.0)),
])
def test_large_blocks_match_oracle(name, kw):
    check_attn(random_problem(**kw), name)


def test_large_block_reference_moves_and_garbage_tail():
    P = random_problem(2, 8, 2, 128, [148 * 128 + 50, 300], [172, 40], [172, 40], seed=31, headroom=150)
    r0 = int(P["q_off"][0])
    q = P["q"][r0 + 100, 5].float()                       # token 100, head 5 -> KV head 1
    for pos, strength in ((200, 45.0), (9000, 100.0)):    # > 2^48 above everything before, twice
        P["k_cache"][1, int(P["kv_off"][0]) + pos] = (strength * np.sqrt(128) * q / q.norm() ** 2).to(torch.bfloat16)
    q2 = P["q"][r0 + 150, 0].float()                      # a step-local needle: key 140 seen by token 150
    P["k_step"][r0 + 140, 0] = (60.0 * np.sqrt(128) * q2 / q2.norm() ** 2).to(torch.bfloat16)
    want, want_lse = oracle_attn(P)
    for b in range(2):
        lo = int(P["kv_off"][b]) + P["lens"][b]
        P["k_cache"][:, lo:lo + 150] = float("nan")
        P["v_cache"][:, lo:lo + 150] = float("inf")
    out, lse = gpu_attn(P)
    from harness import assert_attn_close
    assert_attn_close(out, lse, want, want_lse, "needles + garbage tail")


def test_large_block_equals_the_same_tokens_as_small_blocks():
    # a causal block of 32 tokens gives, row for row, what two causal blocks of 16 give when the
    # first 16 tokens have been appended to the cache in between (ties the large-block kernel to
    # the step kernels and to kv_append)
    dev = "cuda"
    P = random_problem(1, 8, 2, 128, [500], [32], [32], seed=41, headroom=40)
    big, _ = gpu_attn(P)
    Hkv, D, stride = 2, 128, P["n_slots"] * 128
    kc, vc = P["k_cache"].to(dev).clone(), P["v_cache"].to(dev).clone()
    kv_len = P["kv_len"].to(dev).clone()
    first = dict(P, T=16, max_nq=16, q=P["q"][:16], k_step=P["k_step"][:16], v_step=P["v_step"][:16],
                 q_off=torch.tensor([0, 16], dtype=torch.int32), n_cand=torch.tensor([16], dtype=torch.int32))
    out1, _ = gpu_attn(first)
    ms.memosight_kv_append(kc, vc, stride, P["n_slots"], 1, Hkv, D, P["kv_off"].to(dev), kv_len, None,
                           P["k_step"][:16].to(dev),
                           P["v_step"][:16].to(dev), first["q_off"].to(dev), first["n_cand"].to(dev),
                           torch.tensor([16], dtype=torch.int32, device=dev), 16, 1)
    torch.cuda.synchronize()
    second = dict(first, k_cache=kc.cpu(), v_cache=vc.cpu(), kv_len=kv_len.cpu(), lens=[516], q=P["q"][16:],
                  k_step=P["k_step"][16:], v_step=P["v_step"][16:])
    out2, _ = gpu_attn(second)
    assert (big[:16].float() - out1.float()).abs().max() <= 2e-2
    assert (big[16:].float() - out2.float()).abs().max() <= 2e-2


def test_block_size_limits():
    P = random_problem(1, 8, 2, 128, [10], [16], [16], seed=1)
    assert ms.memosight_attn_workspace_bytes(1, 8, 2, 128, 10, 32769) == 0
    assert ms.memosight_attn_workspace_bytes(1, 8, 2, 128, 10, 256) > 0
    # head_dim 64 has no large-block tensor-core kernel: the general kernel serves it
    check_attn(random_problem(1, 4, 2, 64, [200], [40], [40], seed=2), "D=64 large block")


def test_prefill_sized_blocks():
    # Algorithm 1, Prefill: the prompt is one causal block; with an empty cache, and as a chunk
    # behind an already cached part, for two sequences of different length
    check_attn(random_problem(2, 8, 2, 128, [0, 0], [1500, 700], [1500, 700], seed=51), "prefill, empty cache")
    check_attn(random_problem(2, 8, 2, 128, [1000, 3], [1024, 257], [1024, 257], seed=52), "chunked prefill")


def test_long_blocks_whose_key_tiles_left_of_the_diagonal_still_need_the_mask():
    # A long block's key tiles left of the diagonal skip the mask only if all rows and keys there are
    # candidates with default anchors.  Here they are not: foresight rows behind the candidates
    # (they see the candidates up to their anchor and themselves, not each other), custom anchors.
    check_attn(random_problem(2, 8, 2, 128, [300, 0], [400, 300], [350, 300], seed=53),
               "foresight rows behind a long run of candidates")
    check_attn(random_problem(2, 8, 2, 128, [129, 0], [400, 300], [350, 260], seed=54, anchors=True),
               "long blocks with custom anchors")
    check_attn(random_problem(1, 4, 1, 128, [0], [640], [640], seed=55), "all candidates, G = 4, one head")


def test_rows_that_see_nothing_at_first_and_only_strongly_negative_scores_later():
    # Foresight rows with anchor 0 see themselves only.  In a long block with an empty cache such a
    # row finds no visible key in its item's first key tile; its one key comes tiles later -- and here
    # it scores 150 nats below zero, far beyond what an exponential against a placeholder reference
    # of 0 can represent.  The softmax over that single key is still exactly its V row.
    P = random_problem(1, 8, 2, 128, [0], [300], [120], seed=61, anchors=True)
    rows = [130, 201, 299]                       # foresight rows in the second and third key tile
    for i in rows:
        P["anchor"][i] = 0
        for kvh in range(2):
            q = P["q"][i, kvh * 4].float()      # first query head of the group: its score on key i is -150
            P["k_step"][i, kvh] = (-150.0 * np.sqrt(128) * q / q.norm() ** 2).to(torch.bfloat16)
    out, lse = check_attn(P, "unreferenced rows, strongly negative scores")
    for i in rows:
        for kvh in range(2):
            assert torch.equal(out[i, kvh * 4], P["v_step"][i, kvh]), "a single visible key: the output is its V row"
            assert abs(float(lse[i, kvh * 4]) + 150.0) < 1.0
    assert bool(torch.isfinite(out.float()).all())


def test_chunk_without_a_visible_key_beside_a_chunk_of_strongly_negative_scores():
    # The same rows, but the host's bound on the cache length is far above the (empty) cache, so the
    # launch cuts every unit into chunks and the two or three key tiles of a unit land in different
    # chunks.  A foresight row with anchor 0 then sees nothing at all in the chunk that holds the
    # block's first key tile and one key, 150 nats below zero, in a later chunk: the empty chunk's
    # partial must not take part in the merge (were it to carry a reference of 0, the real chunk's
    # weight 2^-216 would flush to zero and the row would come out as 0/0).
    P = random_problem(1, 8, 2, 128, [0], [300], [120], seed=62, anchors=True)
    P["max_kv_len"] = 30000
    rows = [130, 201, 299]
    for i in rows:
        P["anchor"][i] = 0
        for kvh in range(2):
            q = P["q"][i, kvh * 4].float()
            P["k_step"][i, kvh] = (-150.0 * np.sqrt(128) * q / q.norm() ** 2).to(torch.bfloat16)
    out, lse = check_attn(P, "chunked unit, an empty chunk beside strongly negative scores")
    for i in rows:
        for kvh in range(2):
            assert torch.equal(out[i, kvh * 4], P["v_step"][i, kvh])
            assert abs(float(lse[i, kvh * 4]) + 150.0) < 1.0
    assert bool(torch.isfinite(out.float()).all())
    # and a plain chunked block with short tiles in the right half of a tile only: the second
    # accumulator of an item may stay unwritten (every tile of the item has at most 64 valid keys)
    Q = random_problem(2, 8, 2, 128, [40, 64], [70, 100], [70, 100], seed=63)
    Q["max_kv_len"] = 30000
    check_attn(Q, "chunked units whose tiles hold at most 64 keys")
    check_attn(random_problem(2, 8, 2, 128, [40, 64], [40, 64], [40, 64], seed=64), "whole units of at most 64 keys per tile")


def test_more_units_than_ctas_cut_their_last_round():
    # 40 sequences x 2 KV heads x 2 row tiles = 160 units on 148 CTAs (fewer on a smaller part: the
    # case then still runs, uncut): the 12 units of the last round are cut into chunks, each leaves a
    # partial, and a second kernel merges them.  Ragged caches, so the chunks differ in length; a few
    # short blocks (one row tile) shift the unit numbering.
    rng = np.random.default_rng(71)
    lens = [int(x) for x in rng.integers(900, 3000, size=40)]
    n_q = [40] * 40
    n_q[3], n_q[17], n_q[39] = 33, 48, 64
    P = random_problem(40, 8, 2, 128, lens, n_q, n_q, seed=72)
    check_attn(P, "160 units: the last round cut into chunks")
    # and with foresight rows and custom anchors in the cut units
    Q = random_problem(40, 8, 2, 128, lens, n_q, [30] * 40, seed=73, anchors=True)
    check_attn(Q, "160 units, custom anchors")
