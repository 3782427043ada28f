"""Pins for the oracle's KV compaction, append and greedy accept."""
import json
import os

import numpy as np
import torch

import oracle
from conftest import bits, from_bits
from dense_check import dense_attention, to_f64, visibility_matrix

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_examples.json")))


def _cache(n_layers, Hkv, slots, D, seed):
    rng = np.random.default_rng(seed)
    k = rng.integers(0, 0x7F00, size=(n_layers, Hkv, slots, D), dtype=np.uint16)
    v = rng.integers(0, 0x7F00, size=(n_layers, Hkv, slots, D), dtype=np.uint16)
    return k, v


def test_compaction_against_list_surgery():
    n_layers, Hkv, D = 2, 3, 4
    lens, offs = [10, 0, 25, 7], [0, 12, 13, 40]
    slots = 50
    cases = [
        ([3, 0, 5, 0], [4, 0, 17, 7]),      # tail > n, skip, tail < n, everything evicted
        ([0, 0, 24, 6], [1, 0, 1, 0]),      # first entry, skip, last entry, n = 0
        ([9, 0, 0, 2], [1, 0, 25, 3]),
    ]
    for seg_start, seg_len in cases:
        k, v = _cache(n_layers, Hkv, slots, D, 1)
        k0, v0 = k.copy(), v.copy()
        kv_len = np.array(lens, np.int32)
        src = oracle.kv_compact(k, v, n_layers, Hkv * slots * D, slots * D, Hkv, D, np.array(offs),
                                kv_len, seg_start, seg_len, idx_stride=32)
        for b in range(4):
            L, s, n, o = lens[b], seg_start[b], seg_len[b], offs[b]
            keep = list(range(L))
            del keep[s:s + n]                                     # the definition: drop the span
            assert kv_len[b] == L - n == len(keep)
            assert src[b, :len(keep)].tolist() == keep
            assert np.all(src[b, len(keep):] == -1)
            assert np.all(np.diff(src[b, :len(keep)]) > 0)        # order preserved
            for arr, arr0 in ((k, k0), (v, v0)):
                assert np.array_equal(arr[:, :, o:o + len(keep)], arr0[:, :, [o + j for j in keep]])
                assert np.array_equal(arr[:, :, o:o + s], arr0[:, :, o:o + s])   # prefix untouched
        # slots that belong to nobody are never written
        assert np.array_equal(k[:, :, 47:], k0[:, :, 47:])
        assert np.array_equal(k[:, :, 10:12], k0[:, :, 10:12])


def test_compaction_paper_shape_memory_tokens_take_the_steps_place():
    # Sec. 2.1.2 / Algorithm 1: [prefix | step R (n tokens) | l memory tokens, <o>] -> [prefix | M, <o>]
    n, c = 64, 8
    l = oracle.ama(n, c)
    assert l == 8
    prefix = 192
    L = prefix + n + l + 1
    k, v = _cache(1, 2, L, 4, 2)
    k0 = k.copy()
    kv_len = np.array([L], np.int32)
    src = oracle.kv_compact(k, v, 1, 2 * L * 4, L * 4, 2, 4, np.array([0]), kv_len, [prefix], [n], idx_stride=L)
    assert kv_len[0] == prefix + l + 1 == 201
    assert src[0, :201].tolist() == list(range(192)) + list(range(256, 265))
    assert np.array_equal(k[0, :, 192:201], k0[0, :, 256:265])


def test_attention_after_compaction_equals_attention_with_step_masked():
    # ties compaction to the mask rule of Sec. 2.3: evicting a verbose step from the cache is
    # the same as masking it out
    rng = torch.Generator().manual_seed(4)
    Hkv, D, L, s, n = 2, 8, 30, 11, 9
    kc = torch.randn((Hkv, L, D), generator=rng).to(torch.bfloat16)
    vc = torch.randn((Hkv, L, D), generator=rng).to(torch.bfloat16)
    q = torch.randn((4, 4, D), generator=rng).to(torch.bfloat16)
    ks = torch.randn((4, Hkv, D), generator=rng).to(torch.bfloat16)
    vs = torch.randn((4, Hkv, D), generator=rng).to(torch.bfloat16)
    kb, vb = bits(kc)[None].copy(), bits(vc)[None].copy()
    kv_len = np.array([L], np.int32)
    oracle.kv_compact(kb, vb, 1, Hkv * L * D, L * D, Hkv, D, np.array([0]), kv_len, [s], [n])
    out, lse = oracle.attn_step(kb[0], vb[0], L * D, [0], kv_len, [0, 4], [2], None, bits(q), bits(ks), bits(vs))
    vis = visibility_matrix(L, 2, 2, None, hidden_cache=list(range(s, s + n)))
    for h in range(4):
        kvh = h // 2
        k_all = np.concatenate([to_f64(kc[kvh]), to_f64(ks[:, kvh])])
        v_all = np.concatenate([to_f64(vc[kvh]), to_f64(vs[:, kvh])])
        want, want_lse = dense_attention(to_f64(q[:, h]), k_all, v_all, vis, 1 / np.sqrt(D))
        assert np.allclose(out[:, h], want, rtol=1e-12, atol=1e-14)
        assert np.allclose(lse[:, h], want_lse, rtol=1e-12)


def test_append_copies_only_accepted_candidates():
    Hkv, D, slots = 2, 4, 40
    k, v = _cache(1, Hkv, slots, D, 5)
    k, v = k[0], v[0]
    k0, v0 = k.copy(), v.copy()
    rng = np.random.default_rng(6)
    ks = rng.integers(0, 0x7F00, size=(9, Hkv, D), dtype=np.uint16)
    vs = rng.integers(0, 0x7F00, size=(9, Hkv, D), dtype=np.uint16)
    kv_len = np.array([10, 5], np.int32)
    offs = np.array([0, 20])
    q_off = np.array([0, 5, 9], np.int32)         # blocks of 5 (3 cand) and 4 (2 cand)
    oracle.kv_append(k, v, slots * D, Hkv, D, offs, kv_len, ks, vs, q_off, [3, 2], [2, 0])
    assert kv_len.tolist() == [12, 5]
    for h in range(Hkv):
        assert np.array_equal(k[h, 10:12], ks[0:2, h]) and np.array_equal(v[h, 10:12], vs[0:2, h])
    touched = np.zeros(slots, bool)
    touched[10:12] = True
    assert np.array_equal(k[:, ~touched], k0[:, ~touched]) and np.array_equal(v[:, ~touched], v0[:, ~touched])
    # a foresight row can never be appended
    try:
        oracle.kv_append(k, v, slots * D, Hkv, D, offs, kv_len, ks, vs, q_off, [3, 2], [4, 0])
        raise AssertionError("n_keep > n_cand must be rejected")
    except ValueError:
        pass
    # bump=False leaves the lengths (used for all but the last layer)
    oracle.kv_append(k, v, slots * D, Hkv, D, offs, kv_len, ks, vs, q_off, [3, 2], [1, 1], bump=False)
    assert kv_len.tolist() == [12, 5]


# ----------------------------------------------------------------------------- accept

def _logits_with_argmax(argmaxes, V=16, seed=0):
    rng = np.random.default_rng(seed)
    lg = rng.normal(size=(len(argmaxes), V)).astype(np.float32)
    for r, a in enumerate(argmaxes):
        lg[r, a] = 10.0
    return lg


def test_accept_paper_figure_case():
    # Fig. 1 (d=3): the verify block holds the 4 drafts r^3..r^6 as candidates; row i predicts the
    # token after candidate i and is compared with candidate i+1.  r_3 (always valid: it came from
    # the plain next-token prediction) and r_4 are accepted, the draft for r_5 is wrong.
    ex = GOLD["accept"][0]
    r3, r4, r5_draft, r6_draft, r5_true = 3, 4, 55, 6, 5
    cands = [r3, r4, r5_draft, r6_draft]
    draft = cands[1:] + [-1]
    lg = _logits_with_argmax([r4, r5_true, 9, 9])
    am, nm = oracle.accept(lg, 16, [0, 4], draft)
    assert am.tolist() == [r4, r5_true, 9, 9]
    assert nm.tolist() == [1]
    assert nm[0] + 1 == ex["n_accepted_drafts"], ex["cite"]        # c_0 .. c_{n_match} become permanent


def test_accept_hand_worked_cases():
    def run(argmaxes, draft):
        am, nm = oracle.accept(_logits_with_argmax(argmaxes), 16, [0, len(draft)], draft)
        assert am.tolist() == argmaxes
        return int(nm[0])
    assert run([5, 7, 2, 9], [5, 7, 2, -1]) == 3             # everything matches: n_c - 1
    assert run([5, 7, 2, 9], [4, 7, 2, -1]) == 0             # first row wrong
    assert run([5, 7, 2, 9], [5, 7, 9, 9]) == 2              # a match after a mismatch does not count
    assert run([5, 7, 2, 9], [5, -1, 2, 9]) == 1             # the -1 sentinel ends the comparison
    assert run([5, 7, 2, 9], [-1, -1, -1, -1]) == 0
    # several sequences, ragged blocks
    lg = _logits_with_argmax([1, 2, 3, 4, 5, 6, 7])
    am, nm = oracle.accept(lg, 16, [0, 3, 3, 7], [1, 2, -1, 4, 0, 6, -1])
    assert nm.tolist() == [2, 0, 1]


def test_argmax_ties_nan_inf_and_library():
    rng = np.random.default_rng(3)
    lg = rng.normal(size=(40, 257)).astype(np.float32)
    lg[1, [9, 100]] = 50.0                                       # tie: lower index
    lg[2, [256, 0]] = 50.0
    lg[3, 77] = np.inf
    lg[4, :] = -np.inf
    lg[5, [30, 200]] = np.nan                                    # NaN beats everything, first wins
    lg[5, 10] = np.inf
    lg[6, :] = 0.0
    lg[6, 5] = -0.0                                              # -0 == +0: still a tie -> index 0
    lg[7, 256] = 99.0
    am, _ = oracle.accept(lg, 257, [0, 40], [-1] * 40)
    assert am[1] == 9 and am[2] == 0 and am[3] == 77 and am[4] == 0 and am[5] == 30 and am[6] == 0 and am[7] == 256
    assert np.array_equal(am, np.argmax(lg, axis=1).astype(np.int32))    # numpy's convention
    # padded rows: columns >= V are ignored
    lg2 = np.concatenate([lg, np.full((40, 3), 1000.0, np.float32)], axis=1)
    am2, _ = oracle.accept(lg2, 257, [0, 40], [-1] * 40)
    assert np.array_equal(am2, am)


def test_gather_by_keep_list_is_numpy_take_and_generalises_compaction():
    n_layers, Hkv, D, slots = 2, 3, 4, 60
    lens, offs = [10, 0, 25, 7], [0, 12, 13, 40]
    rng = np.random.default_rng(3)
    keeps = [sorted(rng.choice(L, size=rng.integers(0, L + 1), replace=False).tolist()) if L else [] for L in lens]
    keeps[3] = list(range(7))                                   # keep everything: identity
    idx = np.full((4, 32), -1, np.int32)
    for b, kp in enumerate(keeps):
        idx[b, :len(kp)] = kp
    k, v = _cache(n_layers, Hkv, slots, D, 2)
    k0, v0 = k.copy(), v.copy()
    kv_len = np.array(lens, np.int32)
    oracle.kv_gather(k, v, n_layers, Hkv * slots * D, slots * D, Hkv, D, np.array(offs), kv_len, idx,
                     [len(kp) for kp in keeps])
    for b, kp in enumerate(keeps):
        assert kv_len[b] == len(kp)
        for arr, arr0 in ((k, k0), (v, v0)):
            want = np.take(arr0[:, :, offs[b]:offs[b] + lens[b]], np.array(kp, dtype=np.int64), axis=2)
            assert np.array_equal(arr[:, :, offs[b]:offs[b] + len(kp)], want)
    assert np.array_equal(k[:, :, 47:], k0[:, :, 47:])           # nobody's slots stay untouched
    # the paper's eviction is the keep list "everything but the step": same result as kv_compact
    k1, v1 = k0.copy(), v0.copy()
    k2, v2 = k0.copy(), v0.copy()
    len1, len2 = np.array(lens, np.int32), np.array(lens, np.int32)
    seg_start, seg_len = [3, 0, 5, 2], [4, 0, 17, 3]
    src = oracle.kv_compact(k1, v1, n_layers, Hkv * slots * D, slots * D, Hkv, D, np.array(offs), len1,
                            seg_start, seg_len, idx_stride=32)
    oracle.kv_gather(k2, v2, n_layers, Hkv * slots * D, slots * D, Hkv, D, np.array(offs), len2, src, len1)
    assert np.array_equal(len1, len2)
    for b in range(4):
        sl = slice(offs[b], offs[b] + int(len1[b]))
        assert np.array_equal(k1[:, :, sl], k2[:, :, sl]) and np.array_equal(v1[:, :, sl], v2[:, :, sl])


def test_gather_rejects_bad_keep_lists():
    k, v = _cache(1, 1, 10, 4, 5)
    for bad in ([[2, 1]], [[0, 0]], [[9, 10]], [[-1, 3]]):
        idx = np.array(bad, np.int32)
        try:
            oracle.kv_gather(k.copy(), v.copy(), 1, 40, 40, 1, 4, np.array([0]), np.array([10], np.int32), idx, [2])
        except Exception:
            continue
        raise AssertionError(f"keep list {bad} was accepted")
