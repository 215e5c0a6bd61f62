"""Pins of the oracle's variants: value-norm weighting (App. A.1.3), the unstructured variant
(App. A.2), the per-layer minimum and the position-sorted output order -- against library
routines in float64, brute force on toys, special cases and invariants.  CPU only."""
import itertools

import numpy as np
import pytest
import torch


def _qkv(seed, Hq=4, Hkv=2, w=5, N=23, d=8):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((Hq, w, d), generator=g, dtype=torch.float32)
    k = torch.randn((Hkv, N, d), generator=g, dtype=torch.float32)
    v = torch.randn((Hkv, N, d), generator=g, dtype=torch.float32) * torch.rand((Hkv, N, 1), generator=g) * 4
    return q.numpy(), k.numpy(), v.numpy()


# ---------------------------------------------------------------- v-norm weighting

@pytest.mark.parametrize("agg_task,agg_group,augment", [(0, 1, True), (1, 0, False), (1, 1, True), (0, 0, True)])
def test_vnorm_equals_weighting_the_attention_rows_in_float64(oracle, agg_task, agg_group, augment):
    """A^(w) = A * ||v|| entry by entry, then Eqs. 14-16, rebuilt with torch in float64 from the
    (separately pinned) attention rows and torch's own vector norm."""
    q, k, v = _qkv(1)
    Hq, w, d = q.shape
    Hkv, N, _ = k.shape
    G = Hq // Hkv
    scale, q_pos0 = 0.3, N - w
    got = oracle.score_layer_vnorm(q, k, v, scale, q_pos0, agg_task, agg_group, augment)
    norms = torch.linalg.vector_norm(torch.from_numpy(v).double(), dim=-1)          # [Hkv, N]
    S_task = []
    for j in range(Hq):
        A = torch.from_numpy(oracle.attention_rows(q[j], k[j // G], scale, q_pos0)) * norms[j // G][None, :]
        S_task.append(A.amax(dim=0) if agg_task == 0 else A.mean(dim=0))
    S_task = torch.stack(S_task).reshape(Hkv, G, N)
    S_group = S_task.amax(dim=1) if agg_group == 0 else S_task.mean(dim=1)
    want = S_group + S_group.mean(dim=0, keepdim=True) if augment else S_group
    assert np.allclose(got, want.numpy(), rtol=1e-12, atol=0)


def test_vnorm_special_cases(oracle):
    q, k, v = _qkv(2)
    N, w = k.shape[1], q.shape[1]
    plain = oracle.score_layer(q, k, 0.25, N - w)
    unit = v / np.linalg.norm(v.astype(np.float64), axis=-1, keepdims=True)
    # unit-norm value rows: the weighting changes nothing (up to the rounding of unit rows to fp32)
    assert np.allclose(oracle.score_layer_vnorm(q, k, unit.astype(np.float32), 0.25, N - w), plain, rtol=1e-6)
    # positively homogeneous: 4 x the values (exact in fp32), 4 x the scores
    a = oracle.score_layer_vnorm(q, k, v, 0.25, N - w)
    b = oracle.score_layer_vnorm(q, k, (4 * v).astype(np.float32), 0.25, N - w)
    assert np.allclose(b, 4 * a, rtol=1e-12)
    # a zero value row makes its token worthless for its own head (no head-mean term here)
    v0 = v.copy(); v0[1, 7] = 0
    s = oracle.score_layer_vnorm(q, k, v0, 0.25, N - w, augment=False)
    assert s[1, 7] == 0.0 and s[0, 7] > 0
    # the weight is the norm of the token's value row in the query head's own KV head
    nrm = np.linalg.norm(v.astype(np.float64), axis=-1)
    s_plain = oracle.score_layer(q, k, 0.25, N - w, augment=False)
    assert np.allclose(oracle.score_layer_vnorm(q, k, v, 0.25, N - w, augment=False), s_plain * nrm, rtol=1e-12)


# ---------------------------------------------------------------- unstructured variant

def _scores(seed, L=3, Hkv=2, N=7, ties=False):
    rng = np.random.default_rng(seed)
    S = rng.random((L, Hkv, N))
    if ties:
        S = np.round(S * 4) / 4
    return S


@pytest.mark.parametrize("ties", [False, True])
def test_unstructured_select_is_the_top_b_of_the_pool(oracle, ties):
    S = _scores(3, ties=ties)
    L, Hkv, N = S.shape
    order = sorted(((-S[l, h, c], l, h, c) for l in range(L) for h in range(Hkv) for c in range(N)))
    for B in range(0, L * Hkv * N + 1):
        n, off = oracle.select_unstructured(S, B)
        want = np.zeros((L, Hkv), dtype=np.int64)
        for (_, l, h, c) in order[:B]:
            want[l, h] += 1
        assert np.array_equal(n, want), (B, n, want)
        assert off[0] == 0 and np.array_equal(np.diff(off), want.reshape(-1)) and off[-1] == B
        # what a head keeps is a prefix of its own ranking (Eq. 17)
        for l in range(L):
            for h in range(Hkv):
                idx, _ = oracle.rank(S[l, h])
                kept = {c for (_, ll, hh, c) in order[:B] if (ll, hh) == (l, h)}
                assert kept == set(idx[:n[l, h]].tolist())


def test_unstructured_with_one_head_is_the_structured_allocation(oracle):
    """With a single KV head the composite score is the head's sorted score, so the two coincide."""
    S = _scores(4, L=4, Hkv=1, N=9)
    Ssorted = -np.sort(-S[:, 0, :], axis=-1)
    for B in (0, 5, 17, 36):
        n_u, _ = oracle.select_unstructured(S, B)
        n_s, _ = oracle.allocate(Ssorted, B)
        assert np.array_equal(n_u[:, 0], n_s)


def test_unstructured_keeps_at_least_the_score_mass_of_the_structured_choice(oracle):
    """Dropping the alignment constraint can only raise the sum of the kept scores."""
    S = _scores(5, L=3, Hkv=4, N=12)
    L, Hkv, N = S.shape
    Ss = -np.sort(-S, axis=-1)
    I = Ss.mean(axis=1)
    for B in (3, 10, 20):
        n_s, _ = oracle.allocate(I, B)
        mass_s = sum(Ss[l, :, :n_s[l]].sum() for l in range(L))
        n_u, _ = oracle.select_unstructured(S, B * Hkv)
        mass_u = sum(Ss[l, h, :n_u[l, h]].sum() for l in range(L) for h in range(Hkv))
        assert mass_u >= mass_s - 1e-12


# ---------------------------------------------------------------- per-layer minimum

def test_floor_zero_is_plain_allocation_and_floor_is_respected(oracle):
    rng = np.random.default_rng(6)
    I = -np.sort(-rng.random((4, 10)) * rng.random((4, 1)), axis=-1)
    for B in (0, 7, 23, 40):
        a, ao = oracle.allocate(I, B)
        b, bo = oracle.allocate_floor(I, B, 0)
        assert np.array_equal(a, b) and np.array_equal(ao, bo)
    n, off = oracle.allocate_floor(I, 12, 2)
    assert n.sum() == 12 and n.min() >= 2 and off[-1] == 12
    with pytest.raises(ValueError):
        oracle.allocate_floor(I, 7, 2)          # 4 layers x 2 > 7
    with pytest.raises(ValueError):
        oracle.allocate_floor(I, 12, 11)        # more than a layer holds


def test_floor_by_brute_force_on_toys(oracle):
    """Among all (N_1..N_L) with N_l >= m and sum = B, the result keeps the largest score mass
    (unique without ties)."""
    rng = np.random.default_rng(7)
    for trial in range(20):
        L, N = int(rng.integers(2, 4)), int(rng.integers(3, 7))
        I = -np.sort(-rng.random((L, N)) * rng.random((L, 1)), axis=-1)
        m = int(rng.integers(0, 3))
        for B in range(L * m, L * N + 1):
            n, _ = oracle.allocate_floor(I, B, m)
            best, best_v = None, -1.0
            for cand in itertools.product(range(m, N + 1), repeat=L):
                if sum(cand) != B:
                    continue
                val = sum(I[l, :cand[l]].sum() for l in range(L))
                if val > best_v + 1e-15:
                    best, best_v = cand, val
            assert tuple(n.tolist()) == best, (L, N, m, B, n, best)


# ---------------------------------------------------------------- position-sorted output

def test_sort_kept_is_numpy_sort_of_the_prefix(oracle):
    rng = np.random.default_rng(8)
    Hkv, N = 3, 50
    idx = np.stack([rng.permutation(N) for _ in range(Hkv)]).astype(np.int32)
    nk = np.array([0, 17, 50], dtype=np.int32)
    out = oracle.sort_kept(idx, nk)
    for h in range(Hkv):
        assert np.array_equal(out[h, :nk[h]], np.sort(idx[h, :nk[h]]))
        assert np.array_equal(out[h, nk[h]:], idx[h, nk[h]:])
    same = oracle.sort_kept(idx, 20)        # one count for all heads (the structured case)
    assert all(np.array_equal(same[h, :20], np.sort(idx[h, :20])) for h in range(Hkv))
