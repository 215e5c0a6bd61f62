"""GPU parity at the sizes and in the launch configuration the benchmark times (fused
kvc_compress, workspace-held intermediates where possible).  The all-double oracle is run on
sampled layers; everything downstream of the scores is checked exactly against the oracle fed
with the GPU's own previous step, on sampled segments for the per-head steps and in full for
the allocation; invariants that hold at any size are checked on everything."""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import workloads as W

import parity as Pz


def _run(cfg):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    need = 2.6 * 2 * cfg.batch * cfg.n_layers * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim * 2
    if need > free:
        pytest.skip("not enough free device memory for %s" % cfg.name)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    out = kvc.compress(wl.q, wl.k, wl.v, desc, cfg.budget, keep_intermediates=True)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return wl, desc, out


def _check(cfg, layers, segments_per_layer=2):
    import oracle
    oracle.set_threads(len(os.sched_getaffinity(0)))
    wl, desc, out = _run(cfg)
    L, Bt, Hkv, N = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.n_ctx
    budget = cfg.budget
    n_keep = out.n_keep.cpu().numpy(); off = out.offsets.cpu().numpy()
    I = out.composite.cpu().numpy()
    # ---- invariants at full size
    assert n_keep.shape == (Bt, L) and np.all(n_keep >= 0) and np.all(n_keep <= N)
    assert np.all(n_keep.sum(axis=1) == budget)
    assert np.all(off[:, 0] == 0) and np.all(np.diff(off, axis=1) == n_keep) and np.all(off[:, -1] == budget)
    assert np.all(np.diff(I, axis=-1) <= 0), "composite scores must be non-increasing"
    # ---- allocation, exact and in full, from the GPU's own composite scores
    Pz.assert_allocate_exact(I, budget, n_keep, off)
    rng = np.random.default_rng(7)
    worst = 0.0
    for l in layers:
        S_gpu = out.scores[l].cpu().numpy()                      # [Bt, Hkv, N]
        idx_gpu = out.idx[l].cpu().numpy()
        # P1: scores of the whole layer against the all-double oracle
        S_def = Pz.oracle_scores(wl, desc, layers=[l])[0]
        worst = max(worst, Pz.assert_scores_close(S_gpu, S_def))
        # P2: rank on sampled segments, compose on the layer, gather on the layer: exact
        for b in range(Bt):
            for h in rng.choice(Hkv, size=min(segments_per_layer, Hkv), replace=False):
                assert np.array_equal(np.sort(idx_gpu[b, h]), np.arange(N)), "idx must be a permutation"
                Pz.assert_rank_exact(S_gpu[b, h][None], idx_gpu[b, h][None])
        Pz.assert_compose_exact(S_gpu[None], idx_gpu[None], I[l][None], desc.agg_head)
        # P3: tolerance-aware end-to-end order on one sampled segment
        rep = Pz.end_to_end_report(S_def[0, :1], idx_gpu[0, :1])
        assert rep["order_violations"] == 0 and rep["max_gap_at_diff"] < 2 * Pz.SCORE_RTOL, rep
    # gather: every sampled layer, bytes
    Pz.assert_gather_exact(wl, desc, {l: out.idx[l].cpu().numpy() for l in layers}, n_keep, off,
                           out.k_out, out.v_out, layers=layers)
    return worst


def test_llama8b_32k_benchmark_configuration():
    """The configuration bench.py times by default (N = 32768, 25 % retention)."""
    _check(W.LLAMA8B_32K, layers=[0, 13, 31])


def test_llama8b_8k_configuration():
    _check(W.LLAMA8B_8K, layers=[0, 31])


def test_llama8b_32k_low_retention_and_separated_scores():
    """5 % retention, and unit-variance inputs (scores well apart: the GPU order must be the
    oracle's order wherever the oracle's gap exceeds the tolerance)."""
    _check(W.LLAMA8B_32K.replace(retention=0.05, elem_std=1.0, n_layers=8, name="llama8b_32k_r05"), layers=[0, 7])


def test_gqa4_128k_shape_reduced_layers():
    """The long-context GQA-4 shape (w = 64, 7 query heads per KV head: 448 window rows per KV
    head, the CUDA-core scoring path), with 4 of its 28 layers to keep the oracle's share short."""
    _check(W.GQA4_128K.replace(n_layers=4, name="gqa4_128k_L4"), layers=[3], segments_per_layer=1)


def test_ties_configuration():
    """All keys identical except 1 %: long runs of exactly equal scores at full width."""
    cfg = W.TIES_4K
    wl, desc, out = _run(cfg)
    S = out.scores.cpu().numpy(); idx = out.idx.cpu().numpy()
    for l in (0, 31):
        Pz.assert_rank_exact(S[l], idx[l])
    Pz.assert_allocate_exact(out.composite.cpu().numpy(), cfg.budget, out.n_keep.cpu().numpy(),
                             out.offsets.cpu().numpy())
