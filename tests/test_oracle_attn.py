"""Pins for the oracle's masked step attention: brute-force dense softmax with a
materialised mask, library SDPA special cases, closed forms and invariants."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from conftest import bits
from dense_check import dense_attention, to_f64, visibility_matrix


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g) * scale).to(torch.bfloat16)


def _problem(B, Hq, Hkv, D, lens, n_c, d, seed, headroom=3, qscale=1.0):
    """Random ragged problem in the layout the oracle takes."""
    offs, tot = [], 0
    for L in lens:
        offs.append(tot)
        tot += L + headroom
    n_q = n_c + d
    T = B * n_q
    P = dict(
        B=B, Hq=Hq, Hkv=Hkv, D=D, lens=lens, offs=offs, n_c=n_c, d=d, n_q=n_q, slots=tot,
        kc=_rand((Hkv, tot, D), seed), vc=_rand((Hkv, tot, D), seed + 1),
        q=_rand((T, Hq, D), seed + 2, qscale), ks=_rand((T, Hkv, D), seed + 3), vs=_rand((T, Hkv, D), seed + 4),
        q_off=np.arange(0, T + 1, n_q, dtype=np.int32), ncand=np.full(B, n_c, np.int32))
    return P


def _run(P, anchor=None, scale=None):
    return oracle.attn_step(bits(P["kc"]), bits(P["vc"]), P["slots"] * P["D"], np.array(P["offs"]),
                            np.array(P["lens"], np.int32), P["q_off"], P["ncand"], anchor,
                            bits(P["q"]), bits(P["ks"]), bits(P["vs"]), scale)


def _dense(P, anchor=None, scale=None):
    D, G = P["D"], P["Hq"] // P["Hkv"]
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    out = np.zeros((P["B"] * P["n_q"], P["Hq"], D))
    lse = np.zeros((P["B"] * P["n_q"], P["Hq"]))
    for b in range(P["B"]):
        L, o, r0 = P["lens"][b], P["offs"][b], b * P["n_q"]
        anc = None if anchor is None else [int(anchor[r0 + P["n_c"] + k]) for k in range(P["d"])]
        vis = visibility_matrix(L, P["n_c"], P["d"], anc)
        for h in range(P["Hq"]):
            kvh = h // G
            k_all = np.concatenate([to_f64(P["kc"][kvh, o:o + L]), to_f64(P["ks"][r0:r0 + P["n_q"], kvh])])
            v_all = np.concatenate([to_f64(P["vc"][kvh, o:o + L]), to_f64(P["vs"][r0:r0 + P["n_q"], kvh])])
            out[r0:r0 + P["n_q"], h], lse[r0:r0 + P["n_q"], h] = dense_attention(
                to_f64(P["q"][r0:r0 + P["n_q"], h]), k_all, v_all, vis, scale)
    return out, lse


def test_visibility_predicate_equals_materialised_rules():
    for n_c, d in itertools.product(range(0, 5), range(0, 5)):
        if n_c + d == 0:
            continue
        anchor_sets = [None] + [list(a) for a in itertools.product(range(n_c + 1), repeat=d)][:40]
        for anc in anchor_sets:
            vis = visibility_matrix(2, n_c, d, anc)[:, 2:]
            for i in range(n_c + d):
                a_i = i if i < n_c else (n_c if anc is None else anc[i - n_c])
                for j in range(n_c + d):
                    assert oracle.visible(i, j, n_c, a_i) == bool(vis[i, j]), (n_c, d, anc, i, j)


@pytest.mark.parametrize("n_c,d", [(1, 0), (1, 3), (3, 3), (4, 0), (0, 2), (2, 4), (4, 4)])
def test_equals_brute_force_dense_mask(n_c, d):
    P = _problem(B=3, Hq=4, Hkv=2, D=16, lens=[0, 7, 32], n_c=n_c, d=d, seed=100 + 10 * n_c + d)
    out, lse = _run(P)
    want, want_lse = _dense(P)
    assert np.allclose(out, want, rtol=1e-12, atol=1e-13)
    assert np.allclose(lse, want_lse, rtol=1e-12, atol=1e-13)


def test_equals_brute_force_with_all_anchor_choices():
    n_c, d = 3, 2
    P = _problem(B=2, Hq=6, Hkv=2, D=8, lens=[5, 11], n_c=n_c, d=d, seed=7)
    for a in itertools.product(range(n_c + 1), repeat=d):
        anchor = np.zeros(P["B"] * P["n_q"], np.int32)
        for b in range(P["B"]):
            anchor[b * P["n_q"] + n_c: (b + 1) * P["n_q"]] = a
        out, lse = _run(P, anchor)
        want, want_lse = _dense(P, anchor)
        assert np.allclose(out, want, rtol=1e-12, atol=1e-13)
        assert np.allclose(lse, want_lse, rtol=1e-12, atol=1e-13)


def test_plain_decode_equals_library_sdpa():
    # n_c=1, d=0: ordinary single-token decode; the token sees the cache and itself
    P = _problem(B=2, Hq=8, Hkv=2, D=32, lens=[19, 40], n_c=1, d=0, seed=21)
    out, _ = _run(P)
    G = 4
    for b in range(2):
        L, o = P["lens"][b], P["offs"][b]
        k = torch.cat([P["kc"][:, o:o + L], P["ks"][b:b + 1].transpose(0, 1)], dim=1).double()
        v = torch.cat([P["vc"][:, o:o + L], P["vs"][b:b + 1].transpose(0, 1)], dim=1).double()
        k = k.repeat_interleave(G, dim=0)[None]                      # [1][Hq][L+1][D]
        v = v.repeat_interleave(G, dim=0)[None]
        qq = P["q"][b].double()[None, :, None, :]                   # [1][Hq][1][D]
        want = torch.nn.functional.scaled_dot_product_attention(qq, k, v)[0, :, 0]
        assert np.allclose(out[b], want.numpy(), rtol=1e-10, atol=1e-12)


def test_verify_only_equals_library_causal_chunk():
    # d=0: a causal chunk of n_c tokens behind the cache (SDPA with an explicit mask)
    n_c = 5
    P = _problem(B=1, Hq=4, Hkv=4, D=32, lens=[23], n_c=n_c, d=0, seed=33)
    out, _ = _run(P)
    L = 23
    k = torch.cat([P["kc"][:, :L], P["ks"].transpose(0, 1)], dim=1).double()[None]
    v = torch.cat([P["vc"][:, :L], P["vs"].transpose(0, 1)], dim=1).double()[None]
    qq = P["q"].double().transpose(0, 1)[None]                       # [1][H][n_c][D]
    mask = torch.ones(n_c, L + n_c, dtype=torch.bool)
    mask[:, L:] = torch.tril(torch.ones(n_c, n_c, dtype=torch.bool))
    want = torch.nn.functional.scaled_dot_product_attention(qq, k, v, attn_mask=mask)[0].transpose(0, 1)
    assert np.allclose(out, want.numpy(), rtol=1e-10, atol=1e-12)


def test_custom_scale_is_used():
    P = _problem(B=1, Hq=2, Hkv=1, D=16, lens=[9], n_c=2, d=1, seed=5)
    out, lse = _run(P, scale=0.3)
    want, want_lse = _dense(P, scale=0.3)
    assert np.allclose(out, want, rtol=1e-12) and np.allclose(lse, want_lse, rtol=1e-12)
    assert not np.allclose(out, _run(P)[0], rtol=1e-3)


def test_closed_forms():
    P = _problem(B=1, Hq=4, Hkv=2, D=16, lens=[13], n_c=3, d=2, seed=9)
    # (a) all V rows equal -> output is that row, whatever the scores
    row = _rand((16,), 77)
    P["vc"][:] = row
    P["vs"][:] = row
    out, _ = _run(P)
    assert np.allclose(out, np.broadcast_to(to_f64(row), out.shape), rtol=1e-12, atol=1e-14)
    # (b) all K rows equal -> uniform weights: mean of the visible V rows, lse = s + ln(count)
    P = _problem(B=1, Hq=4, Hkv=2, D=16, lens=[13], n_c=3, d=2, seed=9)
    krow = _rand((16,), 78)
    P["kc"][:] = krow
    P["ks"][:] = krow
    out, lse = _run(P)
    for i in range(5):
        vis_local = [j for j in range(5) if (j == i) or (j < 3 and j < (i if i < 3 else 3))]
        for h in range(4):
            kvh = h // 2
            vv = np.concatenate([to_f64(P["vc"][kvh, :13]), to_f64(P["vs"][vis_local, kvh])])
            assert np.allclose(out[i, h], vv.mean(axis=0), rtol=1e-12, atol=1e-14)
            s = float(to_f64(P["q"][i, h]) @ to_f64(krow)) / 4.0
            assert np.isclose(lse[i, h], s + np.log(13 + len(vis_local)), rtol=1e-12)


def test_needle_dominates():
    P = _problem(B=1, Hq=2, Hkv=1, D=32, lens=[50], n_c=2, d=2, seed=13)
    # key 17 is 3x the query of row 0/head 0: its score exceeds every other by > 30
    P["kc"][0, 17] = (P["q"][0, 0].float() * 3.0).to(torch.bfloat16)
    P["q"][0, 0] = (P["q"][0, 0].float() * 3.0).to(torch.bfloat16)
    out, _ = _run(P)
    assert np.allclose(out[0, 0], to_f64(P["vc"][0, 17]), atol=1e-6)


def test_invariants_foresight_isolation_and_causality():
    n_c, d = 3, 3
    P = _problem(B=2, Hq=4, Hkv=2, D=16, lens=[6, 20], n_c=n_c, d=d, seed=55)
    base, base_lse = _run(P)
    n_q = n_c + d
    for b in range(2):
        for k in range(d):                        # perturb foresight token k of sequence b
            Q = {key: (val.clone() if torch.is_tensor(val) else val) for key, val in P.items()}
            r = b * n_q + n_c + k
            Q["q"][r] += 1.0
            Q["ks"][r] += 1.0
            Q["vs"][r] -= 2.0
            out, lse = _run(Q)
            same = np.ones(2 * n_q, bool)
            same[r] = False
            assert np.array_equal(out[same], base[same]) and np.array_equal(lse[same], base_lse[same])
            assert not np.allclose(out[r], base[r])
        for i in range(n_c):                      # perturb candidate i: rows before it unchanged
            Q = {key: (val.clone() if torch.is_tensor(val) else val) for key, val in P.items()}
            r = b * n_q + i
            Q["ks"][r] += 1.0
            Q["vs"][r] -= 2.0
            out, _ = _run(Q)
            untouched = [b2 * n_q + j for b2 in range(2) for j in range(n_q) if b2 != b or j < i]
            assert np.array_equal(out[untouched], base[untouched])
            later = [b * n_q + j for j in range(i, n_q)]
            assert all(not np.allclose(out[j], base[j]) for j in later)


def test_lse_merge_of_any_key_partition_equals_unsplit():
    # softmax is associative under a log-sum-exp merge: split the cache in two, run the oracle on
    # each part (the step-local keys ride with the second part), merge -> the unsplit answer
    P = _problem(B=1, Hq=2, Hkv=1, D=16, lens=[29], n_c=1, d=0, seed=91, headroom=0)
    full, full_lse = _run(P)
    for cut in (1, 8, 28):
        A = dict(P)
        A["lens"] = [cut - 1]                    # first part: cut-1 cache keys + "itself" replaced below
        # part 1: keys [0, cut) only: emulate by making the step key a copy of cache key cut-1
        A["ks"] = P["kc"][:, cut - 1][None].clone()
        A["vs"] = P["vc"][:, cut - 1][None].clone()
        o1, l1 = _run(A)
        Bp = dict(P)
        Bp["kc"], Bp["vc"] = P["kc"][:, cut:].contiguous(), P["vc"][:, cut:].contiguous()
        Bp["lens"], Bp["slots"] = [29 - cut], 29 - cut
        o2, l2 = _run(Bp)
        m = np.maximum(l1, l2)
        w1, w2 = np.exp(l1 - m), np.exp(l2 - m)
        merged = (o1 * w1[..., None] + o2 * w2[..., None]) / (w1 + w2)[..., None]
        assert np.allclose(merged, full, rtol=1e-11, atol=1e-13)
        assert np.allclose(m + np.log(w1 + w2), full_lse, rtol=1e-12)


def test_gqa_head_mapping_is_consecutive_groups():
    # with G=3, query heads 0-2 read KV head 0 and 3-5 read KV head 1: give the
    # two KV heads different constant V rows and read the mapping off the output
    P = _problem(B=1, Hq=6, Hkv=2, D=8, lens=[4], n_c=1, d=0, seed=3)
    P["vc"][0], P["vc"][1] = 1.0, 2.0
    P["vs"][:, 0], P["vs"][:, 1] = 1.0, 2.0
    out, _ = _run(P)
    assert np.allclose(out[0, :3], 1.0) and np.allclose(out[0, 3:], 2.0)
