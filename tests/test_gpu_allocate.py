"""GPU parity of the budget allocation (Eqs. 20-22) on planted composite scores, through every way the
library has of finding the threshold: the sorted-rows kernel (its narrowing rounds, its exact step for
values with very many copies, its last sort, its bisection) and the histogram passes.  All of them must
agree with the oracle bit for bit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc

import parity as Pz

# (path, max_rounds): the library's choice, the histogram passes, the sorted-rows kernel with its
# default bound, with the bisection at once, and with one and two rounds before the bisection
MODES = [(0, -1), (1, -1), (2, -1), (2, 0), (2, 1), (2, 2)]


def _cuda():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


@pytest.fixture(autouse=True)
def _restore_hooks():
    yield
    kvc.kvc_debug_select_hooks(0, -1)


def _rows(kind, L, Bt, N, rng):
    """Composite scores [L, Bt, N], every row non-increasing, fp32."""
    if kind == "uniform":
        I = rng.random((L, Bt, N), dtype=np.float32)
    elif kind == "near_uniform":              # the benchmark's regime: values of a row differ in their last bits
        I = (1.0 / N) * (1.0 + 1e-4 * rng.random((L, Bt, N), dtype=np.float32))
    elif kind == "all_equal":
        I = np.full((L, Bt, N), 0.25, dtype=np.float32)
    elif kind == "three_values":
        I = rng.integers(1, 4, (L, Bt, N)).astype(np.float32)
    elif kind == "fifty_values":
        I = rng.integers(0, 50, (L, Bt, N)).astype(np.float32) / 64.0
    elif kind == "mostly_one_value":
        I = np.where(rng.random((L, Bt, N)) < 0.7, np.float32(0.5), rng.random((L, Bt, N), dtype=np.float32))
    elif kind == "layers_apart":              # every layer in a range of its own: whole layers kept or dropped
        I = rng.random((L, Bt, N), dtype=np.float32) + np.arange(L, dtype=np.float32)[:, None, None]
    elif kind == "signs_and_zeros":
        I = rng.standard_normal((L, Bt, N)).astype(np.float32)
        I[rng.random((L, Bt, N)) < 0.2] = 0.0
        I[rng.random((L, Bt, N)) < 0.05] = -0.0
    else:
        raise ValueError(kind)
    return np.ascontiguousarray(-np.sort(-I.astype(np.float32), axis=-1))


def _check(I, budget, min_keep=0):
    import oracle
    dev = _cuda()
    L, Bt, N = I.shape
    desc = kvc.kvc_desc_init(L, Bt, 2, 1, 64, N, 8, kvc.BF16)
    desc.min_keep_per_layer = min_keep
    It = torch.from_numpy(I).to(dev)
    ws = torch.empty(kvc.kvc_workspace_size(desc, max(budget, 1)), dtype=torch.uint8, device=dev)
    ref_n = np.empty((Bt, L), dtype=np.int32)
    ref_o = np.empty((Bt, L + 1), dtype=np.int64)
    for b in range(Bt):
        if min_keep:
            ref_n[b], ref_o[b] = oracle.allocate_floor(I[:, b].astype(np.float64), budget, min_keep)
        else:
            ref_n[b], ref_o[b] = oracle.allocate(I[:, b].astype(np.float64), budget)
    for path, rounds in MODES:
        kvc.kvc_debug_select_hooks(path, rounds)
        n_keep = torch.full((Bt, L), -7, dtype=torch.int32, device=dev)
        off = torch.full((Bt, L + 1), -7, dtype=torch.int64, device=dev)
        kvc.kvc_allocate(desc, It, budget, n_keep, off, ws)
        torch.cuda.synchronize()
        got_n, got_o = n_keep.cpu().numpy(), off.cpu().numpy()
        assert np.array_equal(got_n, ref_n), ("n_keep differs (path %d, rounds %d, budget %d): gpu %s oracle %s"
                                              % (path, rounds, budget, got_n.tolist(), ref_n.tolist()))
        assert np.array_equal(got_o, ref_o), (path, rounds, budget)
    kvc.kvc_debug_select_hooks(0, -1)


@pytest.mark.parametrize("kind", ["uniform", "near_uniform", "all_equal", "three_values", "fifty_values",
                                  "mostly_one_value", "layers_apart", "signs_and_zeros"])
@pytest.mark.parametrize("L,Bt,N", [(32, 1, 32768), (28, 2, 5000), (5, 3, 700), (1, 1, 3000), (33, 1, 2100),
                                    (70, 1, 1500), (128, 1, 600), (3, 2, 40)])
def test_every_way_to_the_threshold_matches_the_oracle(kind, L, Bt, N):
    rng = np.random.default_rng(L * 1000 + N)
    I = _rows(kind, L, Bt, N, rng)
    total = L * N
    budgets = sorted({0, 1, 2, total // 10, total // 4, total // 2, total - 1, total,
                      int(rng.integers(0, total + 1))})
    if L * N > 200000:
        budgets = [1, total // 4, total // 2 + 1, total - 1]
    for budget in budgets:
        _check(I, budget)


@pytest.mark.parametrize("kind", ["uniform", "three_values", "all_equal"])
@pytest.mark.parametrize("min_keep", [1, 9, 300])
def test_per_layer_minimum_through_every_way(kind, min_keep):
    rng = np.random.default_rng(min_keep)
    L, Bt, N = 12, 2, 4000
    I = _rows(kind, L, Bt, N, rng)
    for budget in (L * min_keep, L * min_keep + 1, L * N // 3, L * N):
        _check(I, budget, min_keep)


@pytest.mark.parametrize("L,Hkv", [(20, 8), (16, 8), (3, 4)])
def test_per_head_pools_on_both_sides_of_the_sorted_rows_limit(L, Hkv):
    """The per-head selection of App. A.2 pools L * Hkv rows: 160 rows go through the histogram passes
    whatever the hook says, 128 and 12 rows through either way."""
    import oracle
    from paper_2509_05165_b200 import workloads as W
    dev = _cuda()
    N = 300
    cfg = W.WorkloadConfig("per_head_pool", L, Hkv, Hkv, 64, N, 1, dtype="f32", elem_std=1.0)
    desc = kvc.desc_from_config(cfg)
    g = np.random.default_rng(L)
    S = (np.round(g.random((L, 1, Hkv, N)) * 512) / 512).astype(np.float32)            # many exact ties
    scores = torch.from_numpy(S).to(dev)
    ws = torch.empty(kvc.kvc_workspace_size(desc, 0), dtype=torch.uint8, device=dev)
    for B in (1, L * Hkv * N // 3, L * Hkv * N - 1):
        n_ref, off_ref = oracle.select_unstructured(S[:, 0].astype(np.float64), B)
        for path, rounds in MODES:
            kvc.kvc_debug_select_hooks(path, rounds)
            idx = torch.empty((L, 1, Hkv, N), dtype=torch.int32, device=dev)
            n_keep = torch.full((1, L, Hkv), -7, dtype=torch.int32, device=dev)
            off = torch.full((1, L * Hkv + 1), -7, dtype=torch.int64, device=dev)
            kvc.kvc_select_unstructured(desc, scores, B, idx, n_keep, off, ws)
            torch.cuda.synchronize()
            assert np.array_equal(n_ref, n_keep.cpu().numpy()[0]), (path, rounds, B)
            assert np.array_equal(off_ref, off.cpu().numpy()[0]), (path, rounds, B)
    kvc.kvc_debug_select_hooks(0, -1)
    Pz.record("allocate paths L%d Hkv%d" % (L, Hkv), modes=len(MODES))
