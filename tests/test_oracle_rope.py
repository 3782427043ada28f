"""Pins for the oracle's RoPE: identities, the relative-position property, a
plain 2-D rotation, and the rotate-half formula evaluated with torch in fp64."""
import numpy as np
import torch

import oracle
from conftest import bits, from_bits


def _rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16)


def _torch_rope_fp64(x, pos, base, interleaved=False, half_units=False, inv_freq=None):
    """Library-style statement: x*cos + rotate_half(x)*sin, fp64, then bf16."""
    T, H, D = x.shape
    xf = x.double()
    inv = torch.tensor(inv_freq, dtype=torch.float64) if inv_freq is not None else \
        base ** (-torch.arange(0, D, 2, dtype=torch.float64) / D)
    p = pos.double() * (0.5 if half_units else 1.0)
    ang = p[:, None] * inv[None, :]                      # [T][D/2]
    if interleaved:
        cos = torch.repeat_interleave(ang.cos(), 2, dim=1)[:, None, :]
        sin = torch.repeat_interleave(ang.sin(), 2, dim=1)[:, None, :]
        rot = torch.stack([-xf[..., 1::2], xf[..., 0::2]], dim=-1).reshape(T, H, D)
    else:
        cos = torch.cat([ang.cos(), ang.cos()], dim=1)[:, None, :]
        sin = torch.cat([ang.sin(), ang.sin()], dim=1)[:, None, :]
        rot = torch.cat([-xf[..., D // 2:], xf[..., :D // 2]], dim=-1)
    return xf * cos + rot * sin


def test_position_zero_is_identity():
    x = _rand_bf16((5, 3, 64), 0)
    out = oracle.rope(bits(x), np.zeros(5, np.int32), 1e4)
    assert np.array_equal(out, bits(x))


def test_d2_is_a_plane_rotation():
    # D=2: a single pair, frequency base^0 = 1: rotation by exactly `pos` radians
    x = torch.tensor([[[1.0, 0.0]], [[0.0, 2.0]], [[-3.0, 4.0]]]).to(torch.bfloat16)
    pos = np.array([1, 2, 5], np.int32)
    got = oracle.bf16_to_f64(oracle.rope(bits(x), pos, 12345.0))
    for t in range(3):
        a, b = x[t, 0].double().tolist()
        c, s = np.cos(pos[t]), np.sin(pos[t])
        want = oracle.bf16_to_f64(oracle.f64_to_bf16(np.array([a * c - b * s, a * s + b * c])))
        assert np.array_equal(got[t, 0], want)


def test_matches_rotate_half_formula_fp64():
    for D, base in ((64, 1e4), (128, 1e6), (128, 5e5)):
        x = _rand_bf16((9, 4, D), D)
        pos = torch.tensor([0, 1, 2, 3, 17, 4096, 49152, 98304, 150000], dtype=torch.int32)
        want = _torch_rope_fp64(x, pos, base)
        got = oracle.bf16_to_f64(oracle.rope(bits(x), pos.numpy(), base))
        # the oracle rounds to bf16 once; the library formula stays fp64
        err = np.abs(got - want.numpy())
        assert np.all(err <= np.abs(want.numpy()) * 2.0**-8 + 1e-30)
        # and after one rounding they agree except (rarely) at rounding boundaries
        want_b = bits(want.to(torch.bfloat16))
        assert np.mean(want_b != oracle.rope(bits(x), pos.numpy(), base)) < 1e-3


def test_interleaved_and_half_units_and_inv_freq():
    x = _rand_bf16((6, 2, 64), 3)
    pos = torch.tensor([3, 8, 11, 250, 7001, 12], dtype=torch.int32)
    want = _torch_rope_fp64(x, pos, 1e4, interleaved=True)
    got = oracle.bf16_to_f64(oracle.rope(bits(x), pos.numpy(), 1e4, flags=oracle.ROPE_INTERLEAVED))
    assert np.all(np.abs(got - want.numpy()) <= np.abs(want.numpy()) * 2.0**-8 + 1e-30)
    want = _torch_rope_fp64(x, pos, 1e4, half_units=True)
    got = oracle.bf16_to_f64(oracle.rope(bits(x), pos.numpy(), 1e4, flags=oracle.POS_HALF_UNITS))
    assert np.all(np.abs(got - want.numpy()) <= np.abs(want.numpy()) * 2.0**-8 + 1e-30)
    # position 2p in half units == position p in whole units, bit for bit
    a = oracle.rope(bits(x), 2 * pos.numpy(), 1e4, flags=oracle.POS_HALF_UNITS)
    b = oracle.rope(bits(x), pos.numpy(), 1e4)
    assert np.array_equal(a, b)
    inv = (np.linspace(1.0, 1e-3, 32)).tolist()
    want = _torch_rope_fp64(x, pos, 0.0, inv_freq=inv)
    got = oracle.bf16_to_f64(oracle.rope(bits(x), pos.numpy(), 0.0, inv_freq=np.array(inv)))
    assert np.all(np.abs(got - want.numpy()) <= np.abs(want.numpy()) * 2.0**-8 + 1e-30)


def test_norm_preserved_and_scores_depend_on_relative_position():
    D = 128
    q = _rand_bf16((1, 1, D), 10)
    k = _rand_bf16((1, 1, D), 11)
    qn = float((q.double() ** 2).sum())

    def dot(pq, pk):
        rq = oracle.bf16_to_f64(oracle.rope(bits(q), np.array([pq], np.int32), 1e4))
        rk = oracle.bf16_to_f64(oracle.rope(bits(k), np.array([pk], np.int32), 1e4))
        return float((rq * rk).sum()), float((rq ** 2).sum())

    base_dot, n0 = dot(5, 2)
    assert abs(n0 - qn) / qn < 5e-3                       # rotation keeps the norm (bf16 rounding)
    for shift in (1, 40, 777):
        d2, n2 = dot(5 + shift, 2 + shift)
        assert abs(d2 - base_dot) < 0.25                  # bf16 rounding noise on |q||k| ~ 128
        assert abs(n2 - qn) / qn < 5e-3
    assert abs(dot(9, 2)[0] - base_dot) > 0.5             # a different offset does change it
