"""Helpers that compare the CUDA library with the CPU oracle on the same seeded inputs.

Scores are compared with the double-precision oracle within a relative tolerance; every later
step decides integers (orders, counts, copied bytes) from fp32 scores, so it is compared
*staged*: the oracle is fed the GPU's own output of the previous step and the result must then
be identical.  The end-to-end comparison with the all-double oracle is tolerance-aware: where
the two disagree, the oracle's own score gap at that place must be below the tolerance.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle

SCORE_RTOL = 1e-3      # bf16 inputs, fp32 accumulation (the stated bound)
SCORE_ATOL = 1e-30     # masked entries are exact zeros on both sides


def to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def raw_numpy(t: torch.Tensor) -> np.ndarray:
    """The tensor's bytes as a numpy array of a same-width integer/float type."""
    t = t.detach().to("cpu").contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def oracle_scores(wl, desc, layers=None, batches=None) -> np.ndarray:
    """Definition-mode scores [len(layers), len(batches), Hkv, N] (float64)."""
    layers = list(range(desc.n_layers)) if layers is None else list(layers)
    batches = list(range(desc.batch)) if batches is None else list(batches)
    scale = desc.scale if desc.scale > 0 else 1.0 / np.sqrt(desc.head_dim)
    q_to_kv = None
    if desc.q_to_kv:
        q_to_kv = [desc.q_to_kv[j] for j in range(desc.n_q_heads)]
    out = np.empty((len(layers), len(batches), desc.n_kv_heads, desc.n_ctx), dtype=np.float64)
    for li, l in enumerate(layers):
        for bi, b in enumerate(batches):
            out[li, bi] = oracle.score_layer(to_f32_numpy(wl.q[l][b]), to_f32_numpy(wl.k[l][b]), scale,
                                             desc.q_pos0, desc.agg_task, desc.agg_group,
                                             bool(desc.augment_head_mean), q_to_kv)
    return out


def assert_scores_close(S_gpu: np.ndarray, S_def: np.ndarray, rtol=SCORE_RTOL):
    err = np.abs(S_gpu.astype(np.float64) - S_def)
    bound = rtol * np.abs(S_def) + SCORE_ATOL
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err / (np.abs(S_def) + 1e-300)), err.shape)
        raise AssertionError("scores differ: %d entries beyond rtol %.1e; worst at %s gpu=%r oracle=%r"
                             % (bad.sum(), rtol, i, S_gpu[i], S_def[i]))
    rel = err / np.maximum(np.abs(S_def), 1e-300)
    return float(rel[S_def > 0].max()) if (S_def > 0).any() else 0.0


def assert_rank_exact(S_gpu: np.ndarray, idx_gpu: np.ndarray, segments=None):
    """idx_gpu must be the oracle's ranking of the GPU's own scores (Eq. 17), bit for bit."""
    S2 = S_gpu.reshape(-1, S_gpu.shape[-1])
    I2 = idx_gpu.reshape(-1, idx_gpu.shape[-1])
    segs = range(S2.shape[0]) if segments is None else segments
    for s in segs:
        ref, _ = oracle.rank(S2[s].astype(np.float64))
        if not np.array_equal(ref, I2[s]):
            k = int(np.argmax(ref != I2[s]))
            raise AssertionError("segment %d: rank differs first at k=%d: gpu %d (score %r) vs oracle %d (score %r)"
                                 % (s, k, I2[s][k], S2[s][I2[s][k]], ref[k], S2[s][ref[k]]))


def assert_compose_exact(S_gpu: np.ndarray, idx_gpu: np.ndarray, I_gpu: np.ndarray, agg_head: int, units=None):
    """composite == Eq. 19 of the GPU's scores at the GPU's order, evaluated in fp32 in head order."""
    L, Bt, Hkv, N = S_gpu.shape
    units = [(l, b) for l in range(L) for b in range(Bt)] if units is None else units
    for (l, b) in units:
        Ss = np.take_along_axis(S_gpu[l, b], idx_gpu[l, b].astype(np.int64), axis=1)
        ref = oracle.compose_f32(Ss, agg_head)
        if not np.array_equal(ref.view(np.uint32), I_gpu[l, b].view(np.uint32)):
            k = int(np.argmax(ref != I_gpu[l, b]))
            raise AssertionError("composite differs at layer %d seq %d k=%d: gpu %r oracle %r"
                                 % (l, b, k, I_gpu[l, b, k], ref[k]))


def assert_allocate_exact(I_gpu: np.ndarray, budget: int, n_keep_gpu: np.ndarray, offsets_gpu: np.ndarray):
    """n_keep / offsets == Eqs. 20-22 applied to the GPU's composite scores."""
    L, Bt, N = I_gpu.shape
    for b in range(Bt):
        n_ref, off_ref = oracle.allocate(I_gpu[:, b].astype(np.float64), budget)
        assert np.array_equal(n_ref, n_keep_gpu[b]), ("n_keep differs for sequence %d: gpu %s oracle %s"
                                                      % (b, n_keep_gpu[b].tolist(), n_ref.tolist()))
        assert np.array_equal(off_ref, offsets_gpu[b])
        assert int(n_keep_gpu[b].sum()) == budget


def assert_gather_exact(wl, desc, idx_gpu, n_keep, offsets, k_out, v_out, layers=None):
    """K', V' == Eqs. 23-24 with the GPU's idx and n_keep, compared as raw bytes."""
    Hkv, d = desc.n_kv_heads, desc.head_dim
    layers = range(desc.n_layers) if layers is None else layers
    ko, vo = raw_numpy(k_out), raw_numpy(v_out)
    for b in range(desc.batch):
        for l in layers:
            n = int(n_keep[b, l])
            lo = int(offsets[b, l]) * Hkv * d
            for (src, dst, name) in ((wl.k, ko, "K"), (wl.v, vo, "V")):
                ref = oracle.gather_layer(raw_numpy(src[l][b]), idx_gpu[l][b], n)
                got = dst[b, lo:lo + Hkv * n * d].reshape(Hkv, n, d)
                assert np.array_equal(ref, got), "%s' differs at layer %d seq %d" % (name, l, b)


def end_to_end_report(S_def: np.ndarray, idx_gpu: np.ndarray, rtol=SCORE_RTOL):
    """Tolerance-aware comparison of the GPU order with the all-double oracle on [.., N] segments.

    Returns dict(order_violations, n_diff, max_gap_at_diff, tie_margin):
      order_violations: adjacent GPU pairs whose oracle scores are out of order by more than 2*rtol;
      n_diff:           positions where idx differs from the oracle's ranking;
      max_gap_at_diff:  largest relative oracle-score gap among those (must be < 2*rtol);
      tie_margin:       smallest relative gap between adjacent oracle-sorted scores where both agree.
    Gaps are relative to the larger score plus SCORE_ATOL / rtol, i.e. measured against the same
    bound rtol * |S| + SCORE_ATOL that the scores themselves are held to (scores that underflow
    on the GPU are exact zeros there and tiny positive numbers in double).
    """
    floor = SCORE_ATOL / rtol
    S2 = S_def.reshape(-1, S_def.shape[-1])
    I2 = idx_gpu.reshape(-1, idx_gpu.shape[-1])
    viol, ndiff, maxgap, margin = 0, 0, 0.0, np.inf
    for s in range(S2.shape[0]):
        sg = S2[s][I2[s]]
        viol += int(np.sum(sg[:-1] + 2 * SCORE_ATOL < sg[1:] * (1 - 2 * rtol)))
        ref, Ss = oracle.rank(S2[s])
        diff = ref != I2[s]
        ndiff += int(diff.sum())
        if diff.any():
            a, b2 = S2[s][ref[diff]], S2[s][I2[s][diff]]
            gap = np.abs(a - b2) / (np.maximum(a, b2) + floor)
            maxgap = max(maxgap, float(gap.max()))
        agree = ~diff[:-1] & ~diff[1:]
        if agree.any():
            g = (Ss[:-1] - Ss[1:])[agree] / (Ss[:-1][agree] + floor)
            margin = min(margin, float(g.min()))
    return dict(order_violations=viol, n_diff=ndiff, max_gap_at_diff=maxgap, tie_margin=float(margin))


def oracle_downstream(S_def_b: np.ndarray, agg_head: int, budget=None):
    """Eqs. 17-22 of the all-double oracle on its own scores S_def_b [L, Hkv, N] of one sequence."""
    L, Hkv, N = S_def_b.shape
    idx = np.empty(S_def_b.shape, dtype=np.int32)
    Ss = np.empty(S_def_b.shape, dtype=np.float64)
    I = np.empty((L, N), dtype=np.float64)
    for l in range(L):
        for h in range(Hkv):
            idx[l, h], Ss[l, h] = oracle.rank(S_def_b[l, h])
        I[l] = oracle.compose(Ss[l], agg_head)
    out = dict(scores=S_def_b, idx=idx, sorted=Ss, composite=I)
    if budget is not None:
        out["n_keep"], out["offsets"] = oracle.allocate(I, budget)
    return out


def oracle_end_to_end(wl, desc, budget, b=0, layers=None):
    """The all-double oracle for one sequence, step by step in the paper's order (Eqs. 3, 14-22),
    one layer of inputs on the host at a time.  Returns dict(scores [L, Hkv, N], idx, sorted,
    composite [L, N], n_keep [L], offsets [L + 1]); with `layers` only those layers are scored
    and the allocation is left out."""
    L = desc.n_layers
    sel = list(range(L)) if layers is None else list(layers)
    S = np.empty((len(sel), desc.n_kv_heads, desc.n_ctx), dtype=np.float64)
    idx = np.empty(S.shape, dtype=np.int32)
    Ss = np.empty(S.shape, dtype=np.float64)
    I = np.empty((len(sel), desc.n_ctx), dtype=np.float64)
    for li, l in enumerate(sel):
        S[li] = oracle_scores(wl, desc, layers=[l], batches=[b])[0, 0]
        for h in range(desc.n_kv_heads):
            idx[li, h], Ss[li, h] = oracle.rank(S[li, h])
        I[li] = oracle.compose(Ss[li], desc.agg_head)
    out = dict(scores=S, idx=idx, sorted=Ss, composite=I)
    if layers is None:
        out["n_keep"], out["offsets"] = oracle.allocate(I, budget)
    return out


def allocation_report(I_def: np.ndarray, n_def: np.ndarray, n_gpu: np.ndarray, budget: int):
    """Per-layer allocation of the GPU against the all-double oracle's (Eqs. 20-22), one sequence.

    Returns dict(sum_abs_dn, layers_differing, max_gap_at_diff, boundary_margin):
      sum_abs_dn:       sum over the layers of |N_l(gpu) - N_l(oracle)|;
      max_gap_at_diff:  over every composite token one side keeps and the other drops, the largest
                        relative distance of its oracle composite score from the oracle's
                        threshold (the smallest kept pooled value);
      boundary_margin:  relative gap between the smallest kept and the largest dropped pooled
                        value of the oracle (how close the decision at the budget boundary is).
    """
    L, N = I_def.shape
    n_def = np.asarray(n_def, dtype=np.int64)
    n_gpu = np.asarray(n_gpu, dtype=np.int64)
    kept = [I_def[l, n_def[l] - 1] for l in range(L) if n_def[l] > 0]
    dropped = [I_def[l, n_def[l]] for l in range(L) if n_def[l] < N]
    T = min(kept) if kept else None
    margin = float("inf")
    if kept and dropped:
        margin = float((T - max(dropped)) / (T + SCORE_ATOL / SCORE_RTOL))
    gap = 0.0
    differing = []
    for l in range(L):
        if n_gpu[l] != n_def[l]:
            differing.append(l)
            lo, hi = sorted((int(n_gpu[l]), int(n_def[l])))
            ref = T if T is not None else max(dropped)
            gap = max(gap, float(np.max(np.abs(I_def[l, lo:hi] - ref)) / (ref + SCORE_ATOL / SCORE_RTOL)))
    return dict(sum_abs_dn=int(np.abs(n_gpu - n_def).sum()), layers_differing=differing,
                max_gap_at_diff=gap, boundary_margin=margin, budget=int(budget))


def assert_allocation_e2e(I_def, n_def, n_gpu, budget, rtol=SCORE_RTOL, strict=False):
    """The GPU's per-layer allocation equals the all-double oracle's except where the oracle's own
    composite scores lie within the tolerance of its threshold; `strict`: it must be equal."""
    rep = allocation_report(I_def, n_def, n_gpu, budget)
    assert int(np.sum(n_gpu)) == budget, rep
    assert rep["max_gap_at_diff"] < 2 * rtol, rep
    if strict:
        assert rep["sum_abs_dn"] == 0, rep
    return rep


def exact_tie_report(S_def: np.ndarray, idx_gpu: np.ndarray):
    """Positions where the GPU order differs from the oracle's order, and how many of them are
    NOT exact ties of the oracle's double-precision scores (an exact tie is the only difference
    admissible on well-separated inputs)."""
    S2 = S_def.reshape(-1, S_def.shape[-1])
    I2 = idx_gpu.reshape(-1, idx_gpu.shape[-1])
    ndiff = not_tie = 0
    for s in range(S2.shape[0]):
        ref, _ = oracle.rank(S2[s])
        diff = ref != I2[s]
        ndiff += int(diff.sum())
        not_tie += int(np.sum(S2[s][ref[diff]] != S2[s][I2[s][diff]]))
    return dict(n_diff=ndiff, n_diff_not_exact_tie=not_tie)


# Every report a test produces is kept here and printed at the end of the session (conftest).
REPORTS = []


def record(name: str, **fields):
    REPORTS.append((name, fields))
    print("parity[%s]: %s" % (name, fields))
