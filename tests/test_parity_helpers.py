"""CPU checks of the tolerance-aware end-to-end comparisons the GPU tests rely on: they must
accept differences that lie inside the score tolerance, report them, and reject anything else.
The "other side" here is the oracle itself run on perturbed scores -- no GPU involved."""
import numpy as np
import pytest

import parity as Pz


def _scores(seed, L=3, Hkv=2, N=400):
    rng = np.random.default_rng(seed)
    return rng.random((L, Hkv, N)) ** 4 + 1e-6


def test_identical_sides_report_nothing(oracle):
    S = _scores(0)
    d = Pz.oracle_downstream(S, oracle.AGG_MEAN, budget=300)
    rep = Pz.end_to_end_report(S, d["idx"])
    assert rep["order_violations"] == 0 and rep["n_diff"] == 0 and rep["max_gap_at_diff"] == 0.0
    assert 0 < rep["tie_margin"] < 1
    a = Pz.assert_allocation_e2e(d["composite"], d["n_keep"], d["n_keep"], 300, strict=True)
    assert a["sum_abs_dn"] == 0 and a["layers_differing"] == [] and a["boundary_margin"] >= 0


def test_perturbation_inside_the_tolerance_is_accepted_and_reported(oracle):
    S = _scores(1, N=3000)
    rng = np.random.default_rng(2)
    S_other = S * (1 + rng.uniform(-0.9e-3, 0.9e-3, S.shape))        # a side that is within rtol
    d = Pz.oracle_downstream(S, oracle.AGG_MEAN, budget=4000)
    o = Pz.oracle_downstream(S_other, oracle.AGG_MEAN, budget=4000)
    rep = Pz.end_to_end_report(S, o["idx"])
    assert rep["n_diff"] > 0, "dense scores: a 1e-3 perturbation must reorder some neighbours"
    assert rep["order_violations"] == 0 and rep["max_gap_at_diff"] < 2e-3
    a = Pz.assert_allocation_e2e(d["composite"], d["n_keep"], o["n_keep"], 4000)
    assert a["max_gap_at_diff"] < 2e-3


def test_a_wrong_order_or_allocation_is_rejected(oracle):
    S = _scores(3)
    d = Pz.oracle_downstream(S, oracle.AGG_MEAN, budget=300)
    bad = d["idx"].copy()
    bad[0, 0, [0, 200]] = bad[0, 0, [200, 0]]                       # best token swapped far down
    rep = Pz.end_to_end_report(S, bad)
    assert rep["order_violations"] > 0 and rep["max_gap_at_diff"] > 2e-3
    n_bad = d["n_keep"].copy()
    take = min(40, int(n_bad[0]))
    n_bad[0] -= take; n_bad[1] += take                               # budget moved between layers
    with pytest.raises(AssertionError):
        Pz.assert_allocation_e2e(d["composite"], d["n_keep"], n_bad, 300)
    with pytest.raises(AssertionError):                              # strict: even a one-slot move
        n1 = d["n_keep"].copy(); n1[0] -= 1; n1[1] += 1
        Pz.assert_allocation_e2e(d["composite"], d["n_keep"], n1, 300, strict=True)


def test_exact_ties_are_the_only_difference_the_strict_report_lets_through(oracle):
    S = _scores(4, L=1, Hkv=1, N=50)
    S[0, 0, 10] = S[0, 0, 20]                                        # an exact tie in double
    idx, _ = oracle.rank(S[0, 0])
    other = idx.copy()
    i10, i20 = int(np.where(idx == 10)[0][0]), int(np.where(idx == 20)[0][0])
    other[[i10, i20]] = other[[i20, i10]]                            # the tie broken the other way
    r = Pz.exact_tie_report(S, other[None, None])
    assert r["n_diff"] == 2 and r["n_diff_not_exact_tie"] == 0
    other2 = idx.copy(); other2[[0, 1]] = other2[[1, 0]]              # a real inversion
    r = Pz.exact_tie_report(S, other2[None, None])
    assert r["n_diff_not_exact_tie"] == 2
