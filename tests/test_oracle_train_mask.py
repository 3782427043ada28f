"""Pins for the training-time attention mask of the oracle (Sec. 2.3 "Attention Mask
Strategy") over an augmented sequence (Sec. 2.2): prompt, then per reasoning step a foresight
token before every reasoning token, the step's memory tokens and its output token."""
import numpy as np
import torch

import oracle
from conftest import bits
from dense_check import dense_attention, to_f64

P, R, F, M, O = oracle.KIND_PROMPT, oracle.KIND_REASON, oracle.KIND_FORESIGHT, oracle.KIND_MEMORY, oracle.KIND_OUTPUT


def augmented_sequence(n_prompt, step_lens, c):
    """Token kinds and step ids of S = P, then for each step: (<f> r)*, <m>*ceil(n/c), <o>."""
    kind, step = [P] * n_prompt, [-1] * n_prompt
    for i, n in enumerate(step_lens):
        for _ in range(n):
            kind += [F, R]
            step += [i, i]
        l = oracle.ama(n, c)
        kind += [M] * l + [O]
        step += [i] * (l + 1)
    return np.array(kind, np.uint8), np.array(step, np.int32)


def prose_matrix(kind, step):
    """The mask built from the prose with whole-matrix operations (not the oracle's predicate):
    causal; a foresight column is hidden from everybody else; a verbose reasoning column is hidden
    from every query outside its step."""
    N = len(kind)
    vis = np.tril(np.ones((N, N), dtype=bool))
    vis[:, kind == F] = False
    verbose = kind == R
    other_step = step[:, None] != step[None, :]
    vis &= ~(verbose[None, :] & other_step)
    vis[np.arange(N), np.arange(N)] = True
    return vis


def _rand(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16)


def _run(kind, step, q, k, v, Hq, Hkv, D):
    T = len(kind)
    empty = np.zeros((Hkv, 1, D), np.uint16)
    return oracle.attn_step(empty, empty, D, [0], np.array([0], np.int32), np.array([0, T], np.int32),
                            np.array([T], np.int32), None, bits(q), bits(k), bits(v), tok_kind=kind, tok_step=step)


def test_predicate_equals_prose_matrix():
    kind, step = augmented_sequence(5, [3, 1, 4], 2)
    N = len(kind)
    want = prose_matrix(kind, step)
    got = np.array([[bool(oracle.lib().ms_oracle_visible_train(i, j, int(kind[j]), int(step[i]), int(step[j])))
                     for j in range(N)] for i in range(N)])
    assert np.array_equal(got, want)
    # spot checks straight from the text: a reasoning token of step 2 sees the prompt, all memory and
    # output tokens before it, the reasoning tokens of its own step before it -- and nothing else
    i = int(np.flatnonzero((kind == R) & (step == 2))[2])
    seen = np.flatnonzero(want[i])
    assert set(kind[seen[:-1]]) <= {P, M, O, R} and all(step[j] == 2 for j in seen if kind[j] == R)
    assert all(j in seen for j in range(5)) and not any(kind[j] == F for j in seen[:-1])


def test_attention_against_dense_softmax_with_the_prose_mask():
    Hq, Hkv, D = 4, 2, 16
    kind, step = augmented_sequence(4, [3, 2, 5], 2)
    T = len(kind)
    q, k, v = _rand((T, Hq, D), 1), _rand((T, Hkv, D), 2), _rand((T, Hkv, D), 3)
    out, lse = _run(kind, step, q, k, v, Hq, Hkv, D)
    vis = prose_matrix(kind, step)
    for h in range(Hq):
        want, want_lse = dense_attention(to_f64(q[:, h]), to_f64(k[:, h // 2]), to_f64(v[:, h // 2]), vis, D ** -0.5)
        assert np.allclose(out[:, h], want, rtol=1e-12, atol=1e-13) and np.allclose(lse[:, h], want_lse, rtol=1e-12)


def test_foresight_tokens_and_old_steps_leave_no_trace():
    Hq, Hkv, D = 2, 1, 8
    kind, step = augmented_sequence(3, [4, 3, 2], 3)
    T = len(kind)
    q, k, v = _rand((T, Hq, D), 4), _rand((T, Hkv, D), 5), _rand((T, Hkv, D), 6)
    base, _ = _run(kind, step, q, k, v, Hq, Hkv, D)
    # (a) perturbing a foresight token changes its own row only
    f_rows = np.flatnonzero(kind == F)
    k2, v2 = k.clone(), v.clone()
    k2[f_rows] += 3.0
    v2[f_rows] -= 2.0
    out, _ = _run(kind, step, q, k2, v2, Hq, Hkv, D)
    others = np.setdiff1d(np.arange(T), f_rows)
    assert np.array_equal(out[others], base[others]) and not np.array_equal(out[f_rows], base[f_rows])
    # (b) the verbose tokens of step 0 are invisible to every later step
    r0 = np.flatnonzero((kind == R) & (step == 0))
    k3, v3 = k.clone(), v.clone()
    k3[r0] *= -1.0
    v3[r0] += 5.0
    out, _ = _run(kind, step, q, k3, v3, Hq, Hkv, D)
    later = np.flatnonzero(step >= 1)
    assert np.array_equal(out[later], base[later])
    own = np.flatnonzero((step == 0) & (kind != F))[1:]
    assert not np.array_equal(out[own], base[own])


def test_training_mask_equals_inference_over_the_compacted_cache():
    # What a token sees under the training mask is exactly what it sees at inference, where the
    # verbose steps have been evicted and foresight tokens were never cached (Sec. 2.1, Sec. 2.3):
    # memory tokens and <o> of step i = one causal block against [prompt, M_<i, o_<i, R_i];
    # a foresight token = a block of its own against [prompt, M_<i, o_<i, r_<t].
    Hq, Hkv, D = 4, 2, 16
    kind, step = augmented_sequence(4, [3, 4, 2], 2)
    T = len(kind)
    q, k, v = _rand((T, Hq, D), 7), _rand((T, Hkv, D), 8), _rand((T, Hkv, D), 9)
    train, train_lse = _run(kind, step, q, k, v, Hq, Hkv, D)
    kb, vb, qb = bits(k), bits(v), bits(q)

    def infer(cache_rows, block_rows, n_c):
        L, n = len(cache_rows), len(block_rows)
        kc = np.ascontiguousarray(kb[cache_rows].transpose(1, 0, 2)) if L else np.zeros((Hkv, 1, D), np.uint16)
        vc = np.ascontiguousarray(vb[cache_rows].transpose(1, 0, 2)) if L else np.zeros((Hkv, 1, D), np.uint16)
        return oracle.attn_step(kc, vc, max(L, 1) * D, [0], np.array([L], np.int32), np.array([0, n], np.int32),
                                np.array([n_c], np.int32), None, qb[block_rows], kb[block_rows], vb[block_rows])

    for i in range(3):
        kept = [j for j in range(T) if kind[j] == P or (kind[j] in (M, O) and step[j] < i)]
        r_i = [j for j in range(T) if kind[j] == R and step[j] == i]
        blk = [j for j in range(T) if kind[j] in (M, O) and step[j] == i]
        out, lse = infer(kept + r_i, blk, len(blk))
        assert np.allclose(out, train[blk], rtol=1e-12, atol=1e-13) and np.allclose(lse, train_lse[blk], rtol=1e-12)
        for t, r in enumerate(r_i):
            f = r - 1                                  # the foresight token in front of r_t
            assert kind[f] == F
            out, _ = infer(kept + r_i[:t], [f], 0)     # a lone foresight token: d = 1, no candidates
            assert np.allclose(out, train[[f]], rtol=1e-12, atol=1e-13)
            out, _ = infer(kept + r_i[:t], [r], 1)     # the regular token itself
            assert np.allclose(out, train[[r]], rtol=1e-12, atol=1e-13)
