"""The seeded input generator: reproducible, sliceable, roughly normal."""
import numpy as np
import torch

from paper_2604_14889_b200 import synth


def test_normal_bf16_is_reproducible_and_sliceable():
    a = synth.normal_bf16(5000, 11, synth.STREAM_KCACHE)
    b = synth.normal_bf16(5000, 11, synth.STREAM_KCACHE, chunk=777)
    assert torch.equal(a, b)
    c = synth.normal_bf16(1000, 11, synth.STREAM_KCACHE, offset=1234)
    assert torch.equal(a[1234:2234], c)
    assert not torch.equal(a, synth.normal_bf16(5000, 12, synth.STREAM_KCACHE))
    assert not torch.equal(a, synth.normal_bf16(5000, 11, synth.STREAM_VCACHE))


def test_moments():
    x = synth.normal_bf16(400000, 1, 2).float()
    assert abs(float(x.mean())) < 0.01 and abs(float(x.std()) - 1.0) < 0.01
    y = synth.normal_f32(400000, 1, 6, sigma=2.0)
    assert abs(float(y.mean())) < 0.02 and abs(float(y.std()) - 2.0) < 0.02
    assert y.unique().numel() > 390000          # fp32 logits: ties are rare


def test_hash_scalar_matches_tensor_hash():
    idx = torch.arange(0, 50, dtype=torch.int64)
    h = synth.hash64(idx, 5, 7)
    for i in range(50):
        want = synth.hash_scalar(i, 5, 7)
        assert (int(h[i]) & ((1 << 64) - 1)) == want


def test_make_step_inputs_layout_and_regeneration():
    cfg = synth.StepConfig("t", 3, 4, 2, 64, 10, 40, 2, 2, 1e4, 100, n_layers=2, headroom=5, seed=9)
    s = synth.make_step_inputs(cfg)
    assert s.k_cache.shape == (2, 2, s.n_slots, 64)
    assert s.kv_off.tolist() == s.offs and s.kv_len.tolist() == s.lens
    assert all(10 <= L <= 40 for L in s.lens)
    assert s.q_off.tolist() == [0, 4, 8, 12]
    unit = synth.regenerate_cache_unit(cfg, s.n_slots, 1, 1, s.offs[2], s.lens[2], "v")
    assert torch.equal(unit, s.v_cache[1, 1, s.offs[2]:s.offs[2] + s.lens[2]])


def test_accept_inputs_cover_all_prefix_lengths():
    cfg = synth.StepConfig("t", 40, 4, 2, 64, 8, 8, 4, 2, 1e4, 500, seed=3)
    a = synth.make_accept_inputs(cfg)
    d = a.draft.view(40, 6)
    assert torch.all(d[:, 3:] == -1) and torch.all(d[:, :3] >= 0)
    assert float(a.logits.max()) == 40.0
