"""memosight_accept_static: the accept call for callers that cannot allocate device
memory (a frozen serving allocator, a plug-in without an allocator handle).  Its
scratch is a fixed array inside the library, shared by every call and never cleared,
so the check is made on two calls in a row with different inputs: both must equal what
memosight_accept (caller workspace) returns, bit for bit -- stale contents of the shared
array must not matter -- and what the CPU oracle's accept returns for the same logits, so that
a mistake the two launch paths had in common would not pass either.  Collected last on purpose:
a failure here cannot hide another test's result in a run that stops at the first failure."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_14889_b200 import binding as ms
from paper_2604_14889_b200 import synth

DEV = "cuda"


def _both(cfg, plant, pad):
    a = synth.make_accept_inputs(cfg, device=DEV, plant=plant, pad=pad)
    B, T = cfg.batch, cfg.batch * cfg.n_q
    ref = [torch.full((n,), -5, dtype=torch.int32, device=DEV) for n in (T, B, B)]
    wsb = ms.memosight_accept_workspace_bytes(T, cfg.vocab)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    ms.memosight_accept(a.logits, a.ld_v, cfg.vocab, a.row_off, B, T, a.draft, *ref, ws, wsb)
    got = [torch.full((n,), -6, dtype=torch.int32, device=DEV) for n in (T, B, B)]
    ms.memosight_accept_static(a.logits, a.ld_v, cfg.vocab, a.row_off, B, T, a.draft, *got)
    torch.cuda.synchronize()
    for g, r in zip(got, ref):
        assert torch.equal(g, r)
    want_am, want_nm = oracle.accept(a.logits.cpu().numpy(), cfg.vocab, a.row_off.cpu().numpy(), a.draft.cpu().numpy())
    assert np.array_equal(got[0].cpu().numpy(), want_am)
    assert np.array_equal(got[1].cpu().numpy(), want_nm)
    assert np.array_equal(got[2].cpu().numpy(), want_nm + 1)
    return a, got


@pytest.mark.gpu
def test_static_accept_equals_workspace_accept_on_two_calls_in_a_row():
    # call 1: planted winners, large vocabulary (19 chunks per row, vector loads)
    cfg1 = synth.StepConfig("na1", 24, 4, 2, 64, 8, 8, 3, 3, 1e4, 151936, seed=41)
    a1, got1 = _both(cfg1, plant=True, pad=0)
    assert got1[0].cpu().tolist() == a1.target
    # call 2, right behind it: other shape, unplanted rows, unaligned rows (scalar loads); the
    # shared array still holds call 1's candidates
    cfg2 = synth.StepConfig("na2", 7, 4, 2, 64, 8, 8, 4, 1, 1e4, 20011, seed=42)
    _both(cfg2, plant=False, pad=1)
    # and once more with the first problem: nothing of call 2 may leak into it
    _, got3 = _both(cfg1, plant=True, pad=0)
    assert got3[0].cpu().tolist() == a1.target


@pytest.mark.gpu
def test_static_accept_rejects_sizes_beyond_its_fixed_array():
    # 3450 rows x 19 chunks = 65 550 candidates > 65 536: refused on the host, nothing is launched
    T, V = 3450, 151936
    assert T * ((V + 8191) // 8192) > ms.MS_ACCEPT_STATIC_MAX_PARTIALS
    dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
    with pytest.raises(ms.MemosightError) as e:
        ms.memosight_accept_static(dummy, V, V, dummy, 1, T, dummy, dummy, dummy, dummy)
    assert e.value.status == ms.MS_ERR_UNSUPPORTED_SHAPE
    # the largest size that fits is accepted by the size check (rows of a 1-chunk vocabulary)
    cfg = synth.StepConfig("na3", 512, 4, 2, 64, 8, 8, 2, 2, 1e4, 4096, seed=43)
    _both(cfg, plant=True, pad=0)
