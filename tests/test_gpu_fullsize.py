"""GPU parity at the sizes and in the launch configuration the benchmark times (fused
kvc_compress).  The all-double oracle is run end to end on every layer, one layer of inputs on
the host at a time: scores element by element within the stated tolerance; the order, the
composite scores, the allocation and the copied rows exactly against the oracle fed with the
GPU's own previous step; the order and the per-layer allocation also against the oracle's own
(tolerance-aware, with the tie margins reported); and the invariants that hold at any size."""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import workloads as W

import parity as Pz


def _workload(cfg):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    need = 2.6 * 2 * cfg.batch * cfg.n_layers * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim * 2
    if need > free:
        pytest.skip("not enough free device memory for %s" % cfg.name)
    return W.make_workload(cfg, dev), kvc.desc_from_config(cfg)


def _compress(wl, desc, budget, keep=True):
    out = kvc.compress(wl.q, wl.k, wl.v, desc, budget, keep_intermediates=keep)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return out


def _merge(rep, new):
    if rep is None:
        return dict(new)
    for k in ("order_violations", "n_diff"):
        rep[k] += new[k]
    rep["max_gap_at_diff"] = max(rep["max_gap_at_diff"], new["max_gap_at_diff"])
    rep["tie_margin"] = min(rep["tie_margin"], new["tie_margin"])
    return rep


def _check(cfg, retentions=None, score_layers=None, gather_layers=None, strict=False):
    """score_layers: layers compared with the all-double oracle (None = all of them; the end-to-end
    allocation check needs all).  retentions: further budgets checked on the same inputs."""
    import oracle
    oracle.set_threads(len(os.sched_getaffinity(0)))
    wl, desc = _workload(cfg)
    L, Bt, Hkv, N = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.n_ctx
    budgets = [cfg.budget] + [cfg.replace(retention=r).budget for r in (retentions or [])]
    out = _compress(wl, desc, budgets[0])
    S_gpu = out.scores.cpu().numpy(); idx_gpu = out.idx.cpu().numpy(); I_gpu = out.composite.cpu().numpy()
    # ---- invariants of the intermediates at full size
    assert np.all(np.diff(I_gpu, axis=-1) <= 0), "composite scores must be non-increasing"
    layers = list(range(L)) if score_layers is None else list(score_layers)
    I_def = np.empty((Bt, len(layers), N), dtype=np.float64)
    worst, rep = 0.0, None
    for li, l in enumerate(layers):
        for b in range(Bt):
            # P1: scores of the layer against the all-double oracle
            S_def = Pz.oracle_scores(wl, desc, layers=[l], batches=[b])[0, 0]         # [Hkv, N]
            worst = max(worst, Pz.assert_scores_close(S_gpu[l, b], S_def))
            # P2: order and composite scores, exact, from the GPU's own scores
            assert np.array_equal(np.sort(idx_gpu[l, b], axis=-1), np.broadcast_to(np.arange(N), (Hkv, N)))
            Pz.assert_rank_exact(S_gpu[l, b], idx_gpu[l, b])
            Pz.assert_compose_exact(S_gpu[l:l + 1, b:b + 1], idx_gpu[l:l + 1, b:b + 1], I_gpu[l:l + 1, b:b + 1],
                                    desc.agg_head)
            # P3: the order against the oracle's own order, tolerance-aware
            rep = _merge(rep, Pz.end_to_end_report(S_def, idx_gpu[l, b]))
            I_def[b, li] = Pz.oracle_downstream(S_def[None], desc.agg_head)["composite"][0]
    assert rep["order_violations"] == 0 and rep["max_gap_at_diff"] < 2 * Pz.SCORE_RTOL, rep
    rep["max_rel_score_err"] = worst
    rep["layers_scored"] = "%d of %d" % (len(layers), L)
    if strict:
        assert rep["n_diff"] == 0, rep
    # ---- allocation and gather for every budget
    g_layers = [0, L // 2, L - 1] if gather_layers is None else gather_layers
    for i, budget in enumerate(budgets):
        o = out if i == 0 else _compress(wl, desc, budget)
        if i > 0:      # the scores do not depend on the budget
            assert torch.equal(o.composite, out.composite) and torch.equal(o.idx, out.idx)
        n_keep = o.n_keep.cpu().numpy(); off = o.offsets.cpu().numpy()
        assert n_keep.shape == (Bt, L) and np.all(n_keep >= 0) and np.all(n_keep <= N)
        assert np.all(n_keep.sum(axis=1) == budget)
        assert np.all(off[:, 0] == 0) and np.all(np.diff(off, axis=1) == n_keep) and np.all(off[:, -1] == budget)
        Pz.assert_allocate_exact(I_gpu, budget, n_keep, off)                 # staged, exact, in full
        a = dict(sum_abs_dn=0, max_gap_at_diff=0.0, boundary_margin=float("inf"))
        if score_layers is None:
            for b in range(Bt):
                n_def, _ = oracle.allocate(I_def[b], budget)
                r = Pz.assert_allocation_e2e(I_def[b], n_def, n_keep[b], budget, strict=strict)
                a["sum_abs_dn"] += r["sum_abs_dn"]
                a["max_gap_at_diff"] = max(a["max_gap_at_diff"], r["max_gap_at_diff"])
                a["boundary_margin"] = min(a["boundary_margin"], r["boundary_margin"])
        Pz.assert_gather_exact(wl, desc, {l: idx_gpu[l] for l in g_layers}, n_keep, off, o.k_out, o.v_out,
                               layers=g_layers)
        # a pass that keeps no intermediates gives the same compressed cache
        lean = _compress(wl, desc, budget, keep=False)
        assert torch.equal(lean.n_keep, o.n_keep)
        assert torch.equal(lean.k_out.view(torch.uint8), o.k_out.view(torch.uint8))
        assert torch.equal(lean.v_out.view(torch.uint8), o.v_out.view(torch.uint8))
        Pz.record("%s budget %d" % (cfg.name, budget), alloc_sum_abs_dn=a["sum_abs_dn"],
                  alloc_gap_at_diff=a["max_gap_at_diff"], alloc_boundary_margin=a["boundary_margin"],
                  n_keep_min=int(n_keep.min()), n_keep_max=int(n_keep.max()), **rep)
    return rep


def test_llama8b_32k_benchmark_configuration_and_lower_retentions():
    """The configuration bench.py times by default (N = 32768, 25 % retention), every layer, and
    the 10 % and 5 % budgets on the same inputs."""
    _check(W.LLAMA8B_32K, retentions=[0.10, 0.05])


def test_llama8b_8k_configuration():
    _check(W.LLAMA8B_8K)


def test_llama8b_32k_separated_scores():
    """Unit-variance inputs (scores well apart: the GPU order must be the oracle's order wherever
    the oracle's gap exceeds the tolerance), 5 % retention, 8 layers of the shape."""
    _check(W.LLAMA8B_32K.replace(retention=0.05, elem_std=1.0, n_layers=8, name="llama8b_32k_std1_L8"))


def test_gqa4_128k_configuration():
    """The long-context GQA-4 shape (w = 64, 7 query heads per KV head: 448 window rows per KV
    head, scored as four row tiles of whole query heads), all 28 layers."""
    _check(W.GQA4_128K, gather_layers=[0, 27])


@pytest.mark.parametrize("n_ctx,batch,retention", [(131072, 1, 0.25), (16384, 4, 0.10), (4096, 8, 0.50)])
def test_sweep_points(n_ctx, batch, retention):
    """Points of the N x batch x retention sweep on the 8B shape that reach different code paths:
    the longest context, several sequences with medium contexts, many sequences at 50 %."""
    _check(W.sweep_config(n_ctx, batch, retention), gather_layers=[0, 31])


def test_ties_configuration():
    """All keys identical except 1 %: long runs of exactly equal scores at full width."""
    cfg = W.TIES_4K
    wl, desc = _workload(cfg)
    out = _compress(wl, desc, cfg.budget)
    S = out.scores.cpu().numpy(); idx = out.idx.cpu().numpy()
    for l in (0, 31):
        Pz.assert_rank_exact(S[l], idx[l])
    Pz.assert_allocate_exact(out.composite.cpu().numpy(), cfg.budget, out.n_keep.cpu().numpy(),
                             out.offsets.cpu().numpy())
