"""Several calls finish their work in the tail of their main kernel when a bank of
last-block-done counters is to be had (the merge of cut attention units, pass 2 of the accept,
the new lengths of append / compaction / keep-list eviction) and fall back to a second launch
when none is.  Here no bank is handed out at all (memosight_debug_set_bank_limit(0)), so every
call takes its two-launch form; the results must be what the oracle gives, exactly as with the
banks -- and the very same problems are run once more with the banks back on."""
import numpy as np
import pytest
import torch

from harness import check_attn, random_problem
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth
import test_gpu_parity as tp

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["two launches", "one launch"])
def banks(request):
    prev = ms.memosight_debug_set_bank_limit(-1)
    if request.param == "two launches":
        ms.memosight_debug_set_bank_limit(0)
    yield request.param
    ms.memosight_debug_set_bank_limit(prev)
    assert ms.memosight_debug_set_bank_limit(-1) == prev


def test_attention_with_many_units_merges_either_way(banks):
    # 320 units on 148 CTAs: with a bank the cut units are merged inside the split kernel, without one by
    # the merge kernel behind it
    lens = [300 + 41 * (b % 9) for b in range(40)]
    check_attn(random_problem(40, 32, 8, 128, lens, [6] * 40, [3] * 40, seed=71), f"40 x 8 units, {banks}")


def test_accept_compaction_gather_and_large_append_either_way(banks):
    cfg = synth.StepConfig("acc", 37, 4, 2, 64, 8, 8, 5, 3, 1e4, 20011, seed=5)
    a = synth.make_accept_inputs(cfg)
    am, nm = tp._accept_both(a.logits, cfg.vocab, a.row_off.tolist(), a.draft.tolist())
    assert am.tolist() == a.target
    c = synth.StepConfig("c4", 3, 32, 8, 128, 900, 1200, 4, 4, 5e5, 100, n_layers=2, seed=78)
    inp = synth.make_step_inputs(c)
    tp._compact_both(inp, [L - 171 - 512 for L in inp.lens], [512] * 3, 1200)
    g = synth.StepConfig("g", 3, 8, 2, 128, 300, 700, 3, 3, 1e4, 100, n_layers=2, headroom=32, seed=91)
    ginp = synth.make_step_inputs(g)
    keeps = [[i for i in range(L) if i < 10 or i % 3] for L in ginp.lens]
    tp._gather_both(ginp, keeps, max(len(k) for k in keeps) + 5)
    # an append of 40-row blocks: several CTAs per sequence, the lengths bumped by whoever counts last
    # (or by the bump kernel)
    import oracle
    from conftest import bits
    ac = synth.StepConfig("ap", 4, 8, 2, 128, 10, 90, 40, 0, 1e4, 100, headroom=48, seed=92)
    ainp = synth.make_step_inputs(ac)
    n_keep = [40, 17, 0, 33]
    kb, vb = bits(ainp.k_cache[0]), bits(ainp.v_cache[0])
    kv_len = ainp.kv_len.numpy().copy()
    oracle.kv_append(kb, vb, ainp.n_slots * 128, 2, 128, ainp.kv_off.numpy(), kv_len, bits(ainp.k_step),
                     bits(ainp.v_step), ainp.q_off.numpy(), ainp.n_cand.numpy(), n_keep)
    dev = "cuda"
    gk, gv, g_len = ainp.k_cache[0].to(dev).clone(), ainp.v_cache[0].to(dev).clone(), ainp.kv_len.to(dev).clone()
    ms.memosight_kv_append(gk, gv, ainp.n_slots * 128, ainp.n_slots, 4, 2, 128, ainp.kv_off.to(dev), g_len, None,
                           ainp.k_step.to(dev), ainp.v_step.to(dev), ainp.q_off.to(dev), ainp.n_cand.to(dev),
                           torch.tensor(n_keep, dtype=torch.int32, device=dev), 40, 1)
    torch.cuda.synchronize()
    assert np.array_equal(g_len.cpu().numpy(), kv_len)
    assert np.array_equal(bits(gk), kb) and np.array_equal(bits(gv), vb)
