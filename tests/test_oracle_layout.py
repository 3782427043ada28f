"""Pins for the oracle's integer position layout (AMA, UPL, <o>, foresight PIDs)
and its bf16 rounding: values the paper prints, closed forms and invariants."""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle
from conftest import bits

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_examples.json")))


def test_ama_paper_examples():
    for ex in GOLD["ama"]:
        assert oracle.ama(ex["n"], ex["c"]) == ex["l"], ex["cite"]


def test_ama_closed_form():
    # l = ceil(n/c), checked against exact rational arithmetic
    for n in range(0, 200):
        for c in range(1, 20):
            assert oracle.ama(n, c) == math.ceil(n / c) == -(-n // c)
    assert oracle.ama(512, 3) == 171
    assert oracle.ama(1, 9) == 1
    with pytest.raises(ValueError):
        oracle.ama(5, 0)


def test_upl_paper_example():
    for ex in GOLD["upl"]:
        assert oracle.upl_pids(ex["rho_first"], ex["n"], ex["c"]).tolist() == ex["pids"], ex["cite"]
    for ex in GOLD["out_pid"]:
        assert oracle.out_pid(ex["rho_first"], ex["n"]) == ex["pid"], ex["cite"]


def test_upl_derived_from_definition():
    # n=10, c=5, PIDs 11..20: groups 11..15 and 16..20 -> centres 13, 18
    assert oracle.upl_pids(11, 10, 5).tolist() == [13, 18]
    # n=7, c=3, PIDs 0..6: groups 0..2, 3..5, 6 -> centres 1, 4, 6
    assert oracle.upl_pids(0, 7, 3).tolist() == [1, 4, 6]
    # exact half-unit centres: group 0..3 has centre 1.5 -> 3 half units
    assert oracle.upl_pids(0, 4, 4, half_units=True).tolist() == [3]
    assert oracle.upl_pids(0, 4, 4).tolist() == [1]          # floor reading of the half-integer


def test_upl_invariants():
    for rho in (0, 5, 1000):
        for n in range(1, 60):
            for c in range(1, 12):
                p = oracle.upl_pids(rho, n, c)
                ph = oracle.upl_pids(rho, n, c, half_units=True)
                l = oracle.ama(n, c)
                assert len(p) == l == len(ph)
                assert np.all(np.diff(p) > 0)                       # strictly increasing
                for g in range(l):
                    lo, hi = rho + g * c, rho + min((g + 1) * c, n) - 1
                    assert lo <= p[g] <= hi                          # inside its own group
                    assert ph[g] == lo + hi                          # exact centre * 2
                    assert p[g] == ph[g] // 2
                # uniform spacing c between full groups
                if l > 2:
                    assert np.all(np.diff(p[:-1]) == c)
                assert oracle.out_pid(rho, n) == rho + n


def test_monotone_pids_ablation():
    assert oracle.monotone_pids(10, 7, 3).tolist() == [17, 18, 19]


def test_fixed_budget_pids_ablation():
    # the "w/o AMA" variant: 9 memory tokens per step whatever its length (App. B.3)
    for rho, n in ((0, 9), (100, 56), (7, 512), (3, 10), (50, 4), (0, 1)):
        p = oracle.budget_pids(rho, n, 9)
        assert len(p) == 9
        assert np.all(np.diff(p) >= 0) and p[0] >= rho and p[-1] <= rho + n - 1    # ordered, inside the step
        if n >= 9:
            assert np.all(np.diff(p) >= 1)                                          # distinct when there is room
            edges = [g * n // 9 for g in range(10)]
            for g in range(9):
                assert rho + edges[g] <= p[g] <= rho + edges[g + 1] - 1             # inside its own group
    # with a budget that divides the step it is UPL with c = n / l
    assert oracle.budget_pids(11, 45, 9).tolist() == oracle.upl_pids(11, 45, 5).tolist()
    assert oracle.budget_pids(0, 9, 9).tolist() == list(range(9))


def test_foresight_pid_paper_examples():
    for ex in GOLD["foresight_pid"]:
        got = oracle.step_pids(ex["p0"], ex["n_c"], ex["d"], ex.get("anchor")).tolist()
        assert got == ex["pids"], ex["cite"]


def test_step_pids_general():
    # candidates consecutive; foresight k sits k after the last regular token it sees
    for p0 in (0, 7, 30000):
        for n_c in range(0, 6):
            for d in range(0, 6):
                pid = oracle.step_pids(p0, n_c, d)
                assert pid[:n_c].tolist() == list(range(p0, p0 + n_c))
                assert pid[n_c:].tolist() == [p0 + n_c - 1 + k for k in range(1, d + 1)]
                # the PID immediately preceding the target: target of f_k is the (k+1)-th token
                # after the last regular one, i.e. PID p_last + k + 1
                for k in range(1, d + 1):
                    assert pid[n_c + k - 1] + 1 == (p0 + n_c - 1) + k + 1
    # training layout (Sec. 2.2): <f> before r_t with offset d' holds rho_{t+d'-1};
    # it sees r_1..r_{t-1}: block = candidates r_1..r_{t-1}, anchor t-1, k = d'
    rho1 = 11
    for t in range(1, 6):
        for dp in range(1, 4):
            anchor = [t - 1] * dp
            pid = oracle.step_pids(rho1, t - 1, dp, anchor)
            assert pid[(t - 1) + dp - 1] == rho1 + (t + dp - 1) - 1


def test_draft_count_statement():
    for ex in GOLD["draft_count"]:
        # one NTP draft from the current token + one per foresight token
        assert 1 + ex["d"] == ex["drafts"]


def test_bf16_rounding_matches_library_on_floats():
    # torch's fp32 -> bf16 cast is round-to-nearest-even; for inputs that are
    # exactly fp32 the oracle's fp64 -> bf16 must agree bit for bit
    g = torch.Generator().manual_seed(1)
    x = torch.randn(200000, generator=g) * torch.exp(torch.randn(200000, generator=g) * 8)
    x = torch.cat([x, torch.tensor([0.0, -0.0, 1.0, -1.0, 3.3895e38, 1e-40, -1e-45, float("inf")])])
    want = bits(x.to(torch.bfloat16))
    got = oracle.f64_to_bf16(x.double().numpy())
    assert np.array_equal(want, got)


def test_bf16_rounding_single_step_from_fp64():
    # 1 + 2^-8 is exactly half way between bf16 neighbours 1 and 1+2^-7: ties to even -> 1.
    # 1 + 2^-8 + 2^-40 is above the tie (an fp32 detour would lose the 2^-40 and mis-round).
    one = 0x3F80
    assert oracle.f64_to_bf16(np.array([1.0 + 2.0**-8]))[0] == one
    assert oracle.f64_to_bf16(np.array([1.0 + 2.0**-8 + 2.0**-40]))[0] == one + 1
    assert oracle.f64_to_bf16(np.array([1.0 + 3 * 2.0**-8]))[0] == one + 2     # tie -> even (up)
    assert oracle.f64_to_bf16(np.array([-(1.0 + 2.0**-8 + 2.0**-40)]))[0] == (one + 1) | 0x8000
    back = oracle.bf16_to_f64(np.arange(0, 0x7F80, 7, dtype=np.uint16))
    assert np.array_equal(oracle.f64_to_bf16(back), np.arange(0, 0x7F80, 7, dtype=np.uint16))
