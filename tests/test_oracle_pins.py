"""Pins for the CPU oracle: every step is checked against something other than itself --
closed forms in exact rational arithmetic, invariants the definitions force, special cases
that collapse to a library routine, and brute force on tiny inputs.  CPU only."""
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

MAX, MEAN = 0, 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# --------------------------------------------------------------------------------------
# Step 1: attention rows (Eq. 3)
# --------------------------------------------------------------------------------------

def test_softmax_special_case_matches_library_softmax(oracle):
    """L = Hkv = G = w = 1 without mask: S = softmax(q K^T / sqrt(d)), twice that with Eq. 16."""
    r = _rng(1)
    d, N = 16, 37
    q = r.standard_normal((1, 1, d)).astype(np.float32)
    k = r.standard_normal((1, N, d)).astype(np.float32)
    scale = 1.0 / math.sqrt(d)
    ref = torch.softmax(torch.from_numpy(k[0].astype(np.float64)) @ torch.from_numpy(q[0, 0].astype(np.float64)) * scale, dim=0).numpy()
    S1 = oracle.score_layer(q, k, scale, q_pos0=N, augment=False)
    S2 = oracle.score_layer(q, k, scale, q_pos0=N, augment=True)
    np.testing.assert_allclose(S1[0], ref, rtol=1e-13, atol=0)
    np.testing.assert_allclose(S2[0], 2 * ref, rtol=1e-13, atol=0)


def test_rows_sum_to_one_through_mean_pooling(oracle):
    """Each attention row sums to 1, so with average pooling over rows and G = 1 the scores of a
    head sum to 1 (2 with the head-mean term, which adds the mean of rows that each sum to 1)."""
    r = _rng(2)
    Hq = Hkv = 3
    w, d, N = 5, 8, 64
    q = r.standard_normal((Hq, w, d)).astype(np.float32) * 2
    k = r.standard_normal((Hkv, N, d)).astype(np.float32) * 2
    for q_pos0 in (N - w, 10, N + 3):
        S = oracle.score_layer(q, k, 0.7, q_pos0, agg_task=MEAN, agg_group=MEAN, augment=False)
        np.testing.assert_allclose(S.sum(axis=1), np.ones(Hkv), rtol=1e-12)
        S = oracle.score_layer(q, k, 0.7, q_pos0, agg_task=MEAN, agg_group=MEAN, augment=True)
        np.testing.assert_allclose(S.sum(axis=1), 2 * np.ones(Hkv), rtol=1e-12)


def test_attention_rows_are_distributions_with_causal_support(oracle):
    r = _rng(3)
    w, d, N, q_pos0 = 6, 4, 20, 11
    A = oracle.attention_rows(r.standard_normal((w, d)), r.standard_normal((N, d)), 0.5, q_pos0)
    for m in range(w):
        vis = min(N, q_pos0 + m + 1)
        assert np.all(A[m, :vis] > 0) and np.all(A[m, vis:] == 0)
        assert abs(A[m].sum() - 1) < 1e-13


def test_identical_keys_closed_form(oracle):
    """All keys equal => every visible key of row m gets 1 / (#visible) = 1 / (q_pos0 + m + 1).
    Max-pooling over rows then gives 1 / (max(c, q_pos0) + 1); average pooling gives the
    mean over the rows that see c.  Evaluated in exact rational arithmetic."""
    r = _rng(4)
    Hq, Hkv, w, d, N = 4, 2, 6, 8, 40
    q_pos0 = N - w
    q = r.standard_normal((Hq, w, d)).astype(np.float32)
    k = np.tile(r.standard_normal((1, 1, d)).astype(np.float32), (Hkv, N, 1))
    s_max = [Fraction(1, max(c, q_pos0) + 1) for c in range(N)]
    s_mean = [sum(Fraction(1, q_pos0 + m + 1) for m in range(w) if c <= q_pos0 + m) / w
              for c in range(N)]
    for agg_task, expect in ((MAX, s_max), (MEAN, s_mean)):
        for agg_group in (MAX, MEAN):
            S = oracle.score_layer(q, k, 1 / math.sqrt(d), q_pos0, agg_task, agg_group, augment=False)
            for h in range(Hkv):
                np.testing.assert_allclose(S[h], [float(x) for x in expect], rtol=1e-13)
            S = oracle.score_layer(q, k, 1 / math.sqrt(d), q_pos0, agg_task, agg_group, augment=True)
            np.testing.assert_allclose(S[0], [2 * float(x) for x in expect], rtol=1e-13)


def test_exact_rational_softmax_weights(oracle):
    """Logits chosen as ln(integer): attention weights are exact ratios a_c / sum(a)."""
    a = np.array([1, 2, 3, 4, 10, 5], dtype=np.float64)
    N, d = len(a), 2
    q = np.array([[[1.0, 0.0]]], dtype=np.float32)
    k = np.zeros((1, N, d), dtype=np.float32)
    k[0, :, 0] = np.log(a)          # rounded to fp32: ~6e-8 relative in the logit
    k[0, :, 1] = 7.0                # orthogonal to q: must not matter
    S = oracle.score_layer(q, k, 1.0, q_pos0=N, augment=False)
    np.testing.assert_allclose(S[0], a / a.sum(), rtol=1e-6)
    # the scale multiplies the logit: scale 2 squares the weights
    S = oracle.score_layer(q, k, 2.0, q_pos0=N, augment=False)
    np.testing.assert_allclose(S[0], a ** 2 / (a ** 2).sum(), rtol=1e-6)


def test_dominant_key_takes_all_mass(oracle):
    r = _rng(5)
    Hq, Hkv, w, d, N = 2, 2, 3, 8, 30
    q = r.standard_normal((Hq, w, d)).astype(np.float32)
    k = r.standard_normal((Hkv, N, d)).astype(np.float32) * 0.01
    k[0, 7] = 100 * q[0].mean(axis=0) / np.linalg.norm(q[0].mean(axis=0)) + 30 * q[0].sum(axis=0)
    S = oracle.score_layer(q, k, 1.0, q_pos0=N, augment=False)
    assert S[0, 7] > 1 - 1e-9 and np.all(S[0, np.arange(N) != 7] < 1e-9)


# --------------------------------------------------------------------------------------
# Steps 2-4: aggregation (Eqs. 14-16) against a float64 torch composition, and invariants
# --------------------------------------------------------------------------------------

def _torch_scores(q, k, scale, q_pos0, agg_task, agg_group, augment, q_to_kv):
    q = torch.from_numpy(q.astype(np.float64))
    k = torch.from_numpy(k.astype(np.float64))
    Hq, w, d = q.shape
    Hkv, N, _ = k.shape
    kv_of = torch.tensor(q_to_kv if q_to_kv is not None else [j // (Hq // Hkv) for j in range(Hq)])
    logits = torch.einsum("jmd,jcd->jmc", q, k[kv_of]) * scale
    pos = q_pos0 + torch.arange(w)[:, None]
    mask = torch.arange(N)[None, :] > pos
    A = torch.softmax(logits.masked_fill(mask[None], float("-inf")), dim=-1)
    A = torch.nan_to_num(A, nan=0.0)
    S_task = A.amax(dim=1) if agg_task == MAX else A.mean(dim=1)
    S_group = torch.stack([
        (S_task[kv_of == h].amax(dim=0) if agg_group == MAX else S_task[kv_of == h].mean(dim=0))
        for h in range(Hkv)])
    if augment:
        S_group = S_group + S_group.mean(dim=0, keepdim=True)
    return S_group.numpy()


@pytest.mark.parametrize("agg_task,agg_group,augment", list(itertools.product((MAX, MEAN), (MAX, MEAN), (False, True))))
def test_scores_match_torch_composition(oracle, agg_task, agg_group, augment):
    r = _rng(10 + agg_task * 4 + agg_group * 2 + int(augment))
    for (Hq, Hkv, w, d, N, q_pos0, q_to_kv) in [
        (4, 2, 5, 8, 33, 28, None),
        (6, 2, 3, 4, 17, 20, None),          # no mask at all
        (6, 3, 4, 8, 21, 5, None),           # window in the middle: long masked tail
        (4, 2, 4, 8, 19, 15, [1, 0, 0, 1]),  # explicit, non-contiguous group map
        (3, 3, 2, 4, 9, 7, [2, 0, 1]),
    ]:
        q = r.standard_normal((Hq, w, d)).astype(np.float32)
        k = r.standard_normal((Hkv, N, d)).astype(np.float32)
        got = oracle.score_layer(q, k, 0.9, q_pos0, agg_task, agg_group, augment, q_to_kv)
        ref = _torch_scores(q, k, 0.9, q_pos0, agg_task, agg_group, augment, q_to_kv)
        np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-300)


def test_aggregation_invariants(oracle):
    r = _rng(20)
    Hq, Hkv, w, d, N = 6, 2, 4, 8, 25
    G = Hq // Hkv
    q = r.standard_normal((Hq, w, d)).astype(np.float32)
    k = r.standard_normal((Hkv, N, d)).astype(np.float32)
    base = oracle.score_layer(q, k, 0.5, q_pos0=N)
    assert np.all(base >= 0) and np.all(base <= 2)
    # permuting the query heads inside each group changes nothing
    perm = np.concatenate([h * G + r.permutation(G) for h in range(Hkv)])
    np.testing.assert_allclose(oracle.score_layer(q[perm], k, 0.5, q_pos0=N), base, rtol=1e-13)
    # without a mask, permuting the window rows changes nothing
    np.testing.assert_allclose(oracle.score_layer(q[:, r.permutation(w)], k, 0.5, q_pos0=N), base, rtol=1e-13)
    # duplicating every window row leaves max-pooling unchanged
    np.testing.assert_allclose(oracle.score_layer(np.repeat(q, 2, axis=1), k, 0.5, q_pos0=N), base, rtol=1e-13)
    # swapping two KV heads (with their query groups) swaps the rows of S
    swap_q = np.concatenate([q[G:], q[:G]])
    np.testing.assert_allclose(oracle.score_layer(swap_q, k[::-1], 0.5, q_pos0=N), base[::-1], rtol=1e-13)
    # max-pooling dominates average pooling elementwise
    lo = oracle.score_layer(q, k, 0.5, N, MEAN, MEAN, False)
    hi = oracle.score_layer(q, k, 0.5, N, MAX, MAX, False)
    assert np.all(hi >= lo - 1e-15)


# --------------------------------------------------------------------------------------
# Step 5: rank (Eq. 17)
# --------------------------------------------------------------------------------------

def test_rank_is_stable_descending_argsort(oracle):
    r = _rng(30)
    for N in (1, 2, 17, 1000):
        S = r.integers(0, 7, size=N).astype(np.float64) / 7.0   # many ties
        idx, Ss = oracle.rank(S)
        ref = np.argsort(-S, kind="stable")
        assert np.array_equal(idx, ref)
        assert np.array_equal(Ss, S[ref])
        assert sorted(idx.tolist()) == list(range(N))
        assert np.all(np.diff(Ss) <= 0)
        same = Ss[1:] == Ss[:-1]
        assert np.all(idx[1:][same] > idx[:-1][same])
    S = r.standard_normal(257)
    idx, _ = oracle.rank(S)
    assert np.array_equal(idx, np.argsort(-S, kind="stable"))


# --------------------------------------------------------------------------------------
# Step 6: compose (Eq. 19)
# --------------------------------------------------------------------------------------

def test_compose_mean_max_and_single_head(oracle):
    r = _rng(40)
    Hkv, N = 5, 23
    Ss = -np.sort(-r.random((Hkv, N)), axis=1)
    I = oracle.compose(Ss, MEAN)
    for kk in range(N):
        assert abs(I[kk] - float(sum(Fraction(float(x)) for x in Ss[:, kk]) / Hkv)) < 1e-15
    assert np.array_equal(oracle.compose(Ss, MAX), Ss.max(axis=0))
    assert np.all(np.diff(I) <= 0)                       # sorted rows => non-increasing composite
    assert np.array_equal(oracle.compose(Ss[:1], MEAN), Ss[0])   # Hkv = 1: I = S'
    assert np.array_equal(oracle.compose(Ss[:1], MAX), Ss[0])


def test_compose_f32_fixed_order(oracle):
    r = _rng(41)
    Hkv, N = 8, 101
    Ss = r.random((Hkv, N)).astype(np.float32)
    acc = Ss[0].copy()
    for h in range(1, Hkv):
        acc = (acc + Ss[h]).astype(np.float32)
    assert np.array_equal(oracle.compose_f32(Ss, MEAN), (acc / np.float32(Hkv)).astype(np.float32))
    assert np.array_equal(oracle.compose_f32(Ss, MAX), Ss.max(axis=0))
    # and it is the double result rounded, to within one ulp or so
    np.testing.assert_allclose(oracle.compose_f32(Ss, MEAN), oracle.compose(Ss, MEAN), rtol=1e-6)


# --------------------------------------------------------------------------------------
# Step 7: allocation (global pool, B_total, N_l)
# --------------------------------------------------------------------------------------

def test_budget_formula_on_the_papers_grid(oracle):
    """B_total = floor((1 - r) L N) on the paper's compression grid (golden: paper constants)."""
    with open(os.path.join(GOLDEN, "paper_constants.json")) as f:
        g = json.load(f)
    for r_t in g["compression_grid"]["values"]:
        for (L, N) in ((32, 4096), (28, 4096), (40, 4096), (2, 512), (32, 32768), (28, 131072)):
            expect = math.floor((1 - Fraction(str(r_t))) * L * N)
            assert oracle.budget_from_ratio(L, N, r_t) == expect
    # the retention budgets quoted for the benchmark configurations
    assert oracle.budget_from_ratio(2, 512, 0.75) == 256
    assert oracle.budget_from_ratio(32, 8192, 0.80) == 52428
    assert [oracle.budget_from_ratio(32, 32768, r_t) for r_t in (0.95, 0.90, 0.75)] == [52428, 104857, 262144]
    assert oracle.budget_from_ratio(28, 131072, 0.90) == 367001


def test_allocate_brute_force_enumeration(oracle):
    """With per-layer non-increasing composite scores and no ties, the allocation is the unique
    vector (N_1..N_L), sum = B, that maximises the retained composite mass."""
    r = _rng(50)
    for trial in range(30):
        L = int(r.integers(1, 4))
        N = int(r.integers(1, 7))
        vals = r.permutation(L * N * 3)[: L * N].astype(np.float64)   # distinct
        I = -np.sort(-vals.reshape(L, N), axis=1)
        for B in range(L * N + 1):
            n_keep, off = oracle.allocate(I, B)
            best, arg = -1.0, None
            for cand in itertools.product(range(N + 1), repeat=L):
                if sum(cand) != B:
                    continue
                mass = sum(I[l, :cand[l]].sum() for l in range(L))
                if mass > best:
                    best, arg = mass, cand
            assert tuple(n_keep) == arg
            assert off[0] == 0 and np.array_equal(np.diff(off), n_keep) and off[-1] == B


def test_allocate_definition_on_unsorted_pool_and_ties(oracle):
    r = _rng(51)
    L, N = 4, 9
    I = r.integers(0, 5, size=(L, N)).astype(np.float64)   # heavy ties, not sorted
    order = sorted(((-I[l, k], l, k) for l in range(L) for k in range(N)))
    for B in (0, 1, 7, 18, 35, 36):
        n_keep, off = oracle.allocate(I, B)
        expect = np.zeros(L, dtype=np.int64)
        for (_, l, _) in order[:B]:
            expect[l] += 1
        assert np.array_equal(n_keep, expect)
        assert n_keep.sum() == B and np.all(n_keep >= 0) and np.all(n_keep <= N)
    # every score equal: layers fill in order
    n_keep, _ = oracle.allocate(np.ones((3, 4)), 6)
    assert n_keep.tolist() == [4, 2, 0]
    # edge budgets
    assert oracle.allocate(I, 0)[0].tolist() == [0] * L
    assert oracle.allocate(I, L * N)[0].tolist() == [N] * L
    assert oracle.allocate(I[:1], 5)[0].tolist() == [5]
    with pytest.raises(ValueError):
        oracle.allocate(I, L * N + 1)


def test_allocate_threshold_property(oracle):
    r = _rng(52)
    L, N, B = 5, 40, 77
    I = -np.sort(-r.random((L, N)), axis=1)
    n_keep, _ = oracle.allocate(I, B)
    kept = np.concatenate([I[l, :n_keep[l]] for l in range(L)])
    dropped = np.concatenate([I[l, n_keep[l]:] for l in range(L)])
    assert kept.size == B and kept.min() >= dropped.max()


# --------------------------------------------------------------------------------------
# Step 8: gather, and the whole pass
# --------------------------------------------------------------------------------------

def test_gather_is_direct_indexing(oracle):
    r = _rng(60)
    Hkv, N, d = 3, 11, 8
    src = r.integers(0, 2 ** 16, size=(Hkv, N, d)).astype(np.uint16)
    idx = np.stack([r.permutation(N) for _ in range(Hkv)]).astype(np.int32)
    for n_keep in (0, 1, 5, N):
        out = oracle.gather_layer(src, idx, n_keep)
        ref = np.take_along_axis(src, idx[:, :n_keep, None].astype(np.int64), axis=1)
        assert out.shape == (Hkv, n_keep, d) and np.array_equal(out, ref)


def _tiny_problem(seed, L=3, Hq=4, Hkv=2, w=3, d=8, N=24):
    r = _rng(seed)
    q = r.standard_normal((L, Hq, w, d)).astype(np.float32)
    k = r.standard_normal((L, Hkv, N, d)).astype(np.float32)
    v = r.standard_normal((L, Hkv, N, d)).astype(np.float32)
    return q, k, v


def test_compress_is_the_composition_of_its_steps(oracle):
    q, k, v = _tiny_problem(70)
    L, Hkv, N = k.shape[0], k.shape[1], k.shape[2]
    B = 31
    out = oracle.compress(q, k, k, v, 0.35, N - q.shape[2], B)
    I = np.empty((L, N))
    for l in range(L):
        S = oracle.score_layer(q[l], k[l], 0.35, N - q.shape[2])
        assert np.array_equal(out["scores"][l], S)
        Ss = np.empty_like(S)
        for h in range(Hkv):
            idx, Ss[h] = oracle.rank(S[h])
            assert np.array_equal(out["idx"][l, h], idx)
        I[l] = oracle.compose(Ss)
    assert np.array_equal(out["composite"], I)
    n_keep, off = oracle.allocate(I, B)
    assert np.array_equal(out["n_keep"], n_keep) and np.array_equal(out["offsets"], off)
    for l in range(L):
        lo, hi = off[l] * Hkv, off[l + 1] * Hkv
        assert np.array_equal(out["k_out"][lo:hi].reshape(Hkv, n_keep[l], -1),
                              oracle.gather_layer(k[l], out["idx"][l], n_keep[l]))
        assert np.array_equal(out["v_out"][lo:hi].reshape(Hkv, n_keep[l], -1),
                              oracle.gather_layer(v[l], out["idx"][l], n_keep[l]))


def test_compress_invariants(oracle):
    q, k, v = _tiny_problem(71, L=4, N=30)
    L, Hkv, N, d = k.shape
    for B in (0, 17, 59, L * N):
        out = oracle.compress(q, k, k, v, 0.35, N - q.shape[2], B)
        n_keep = out["n_keep"]
        assert n_keep.sum() == B == out["offsets"][-1]                 # budget met exactly
        for l in range(L):
            for h in range(Hkv):
                # every composite token holds exactly one index per KV head: column k of idx
                assert sorted(out["idx"][l, h].tolist()) == list(range(N))
                # each head keeps its own top-N_l tokens by score
                S = out["scores"][l, h]
                kept = out["idx"][l, h, : n_keep[l]]
                rest = out["idx"][l, h, n_keep[l]:]
                if len(kept) and len(rest):
                    assert S[kept].min() >= S[rest].max()
            assert np.all(np.diff(out["composite"][l]) <= 1e-18)
        if B == L * N:
            # nothing evicted: every head's output is a permutation of its input rows
            for l in range(L):
                got = out["k_out"][l * N * Hkv:(l + 1) * N * Hkv].reshape(Hkv, N, d)
                for h in range(Hkv):
                    assert sorted(map(bytes, got[h])) == sorted(map(bytes, k[l, h]))


def test_layer_with_stronger_attention_gets_more_budget(oracle):
    """Layer-adaptive allocation: a layer whose heads concentrate attention on few tokens has
    larger top composite scores than a layer with flat attention, so at a small budget it receives
    (almost) all of it."""
    r = _rng(72)
    L, Hq, Hkv, w, d, N = 2, 2, 2, 2, 8, 50
    q = r.standard_normal((L, Hq, w, d)).astype(np.float32)
    k = np.zeros((L, Hkv, N, d), dtype=np.float32)          # layer 0: flat attention
    k[1] = r.standard_normal((Hkv, N, d)).astype(np.float32) * 4   # layer 1: peaked
    out = oracle.compress(q, k, None, None, 1.0, N, 5)
    assert out["n_keep"].tolist() == [0, 5]


def test_thread_count_does_not_change_results(oracle):
    q, k, v = _tiny_problem(73)
    a = oracle.compress(q, k, k, v, 0.35, 21, 20)
    oracle.set_threads(3)
    try:
        b = oracle.compress(q, k, k, v, 0.35, 21, 20)
    finally:
        oracle.set_threads(1)
    for key in a:
        assert np.array_equal(a[key], b[key])
