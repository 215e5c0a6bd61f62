"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded
inputs -- element by element at sizes the oracle finishes in seconds, covering several tiles,
ragged tails, both dtypes, both head sizes, every aggregator, custom GQA maps, strides, batches
and the degenerate budgets."""
import ctypes

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import workloads as W
from paper_2509_05165_b200.binding import alloc_outputs

import parity as Pz


def _cuda():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    return torch.device("cuda:0")


def _host(t):
    return t.detach().cpu().numpy()


def run_staged(wl, desc, budget):
    """The four stage entry points one after another; returns host copies of every output."""
    dev = wl.k[0].device
    out = alloc_outputs(desc, budget, wl.k[0].dtype, dev)
    kvc.kvc_score(desc, wl.q, wl.k, out.scores, out.workspace)
    kvc.kvc_compose(desc, out.scores, out.idx, out.composite, out.workspace)
    kvc.kvc_allocate(desc, out.composite, budget, out.n_keep, out.offsets, out.workspace)
    kvc.kvc_gather(desc, wl.k, wl.v, out.idx, out.n_keep, out.offsets, budget, out.k_out, out.v_out)
    torch.cuda.synchronize()
    return out


def run_fused(wl, desc, budget, keep=True):
    out = kvc.compress(wl.q, wl.k, wl.v, desc, budget, keep_intermediates=keep)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    return out


def check_all(wl, desc, budget, e2e_strict=False, check_e2e=True):
    st = run_staged(wl, desc, budget)
    fu = run_fused(wl, desc, budget)
    # the fused entry runs the same kernels: identical bits
    for name in ("scores", "idx", "composite", "n_keep", "offsets", "k_out", "v_out"):
        a, b = getattr(st, name), getattr(fu, name)
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), "fused != staged for " + name
    S = _host(fu.scores); idx = _host(fu.idx); I = _host(fu.composite)
    n_keep = _host(fu.n_keep); off = _host(fu.offsets)
    # P1: scores against the all-double oracle
    S_def = Pz.oracle_scores(wl, desc)
    worst = Pz.assert_scores_close(S, S_def)
    # P2: staged, exact
    Pz.assert_rank_exact(S, idx)
    Pz.assert_compose_exact(S, idx, I, desc.agg_head)
    Pz.assert_allocate_exact(I, budget, n_keep, off)
    Pz.assert_gather_exact(wl, desc, idx, n_keep, off, fu.k_out, fu.v_out)
    # invariants
    assert np.all(np.sort(idx, axis=-1) == np.arange(desc.n_ctx)[None, None, None, :])
    assert np.all(np.diff(I, axis=-1) <= 0)
    # P3: end to end against the all-double oracle, tolerance-aware: the order of every segment,
    # and the per-layer allocation (equal except where the oracle's composite scores lie within
    # the tolerance of its threshold); tie margins are reported
    rep = None
    if check_e2e:
        rep = Pz.end_to_end_report(S_def, idx)
        assert rep["order_violations"] == 0, rep
        assert rep["max_gap_at_diff"] < 2 * Pz.SCORE_RTOL, rep
        rep["max_rel_score_err"] = worst
        rep["sum_abs_dn"], rep["alloc_gap_at_diff"], rep["boundary_margin"] = 0, 0.0, float("inf")
        for b in range(desc.batch):
            d = Pz.oracle_downstream(S_def[:, b], desc.agg_head, budget)
            a = Pz.assert_allocation_e2e(d["composite"], d["n_keep"], n_keep[b], budget, strict=e2e_strict)
            rep["sum_abs_dn"] += a["sum_abs_dn"]
            rep["alloc_gap_at_diff"] = max(rep["alloc_gap_at_diff"], a["max_gap_at_diff"])
            rep["boundary_margin"] = min(rep["boundary_margin"], a["boundary_margin"])
        if e2e_strict:
            # an exact tie of the oracle's double-precision scores is the only admissible difference
            rep.update(Pz.exact_tie_report(S_def, idx))
            assert rep["n_diff_not_exact_tie"] == 0, rep
        Pz.record(wl.cfg.name, **rep)
    # a fused call that keeps no intermediates gives the same compressed cache
    lean = run_fused(wl, desc, budget, keep=False)
    assert torch.equal(lean.k_out.view(torch.uint8), fu.k_out.view(torch.uint8))
    assert torch.equal(lean.n_keep, fu.n_keep)
    return worst, rep


def test_tiny_config_fp32():
    """The tiny fp32 configuration, whole pass, every element."""
    dev = _cuda()
    cfg = W.TINY
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    assert cfg.budget == 256
    check_all(wl, desc, cfg.budget)


def test_tiny_config_separated_scores_strict_order():
    """Unit-variance inputs give well separated scores: the GPU order must equal the oracle's."""
    dev = _cuda()
    cfg = W.TINY.replace(elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    check_all(wl, desc, cfg.budget, e2e_strict=True)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("f32", 128), ("f32", 64)])
def test_ragged_multi_tile(dtype, d):
    """N spans several tiles with a ragged tail; GQA group 4; window 32; causal window mask."""
    dev = _cuda()
    cfg = W.WorkloadConfig("ragged", 3, 8, 2, d, 1500, 32, dtype=dtype, retention=0.3, elem_std=1.0,
                           hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("agg_task,agg_group,agg_head,augment",
                         [(0, 0, 0, 0), (1, 1, 1, 1), (0, 1, 1, 0), (1, 0, 0, 1), (0, 0, 1, 1)])
def test_aggregator_variants(agg_task, agg_group, agg_head, augment):
    dev = _cuda()
    cfg = W.WorkloadConfig("agg", 2, 6, 2, 64, 700, 8, dtype="bf16", retention=0.5, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg, agg_task=agg_task, agg_group=agg_group, agg_head=agg_head,
                                augment_head_mean=augment)
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("q_pos0_kind", ["none", "middle", "zero"])
def test_mask_positions(q_pos0_kind):
    """No mask (task tokens after the context), a window in the middle, and a window at 0."""
    dev = _cuda()
    cfg = W.WorkloadConfig("mask", 2, 4, 2, 64, 333, 16, dtype="f32", retention=0.4, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    q_pos0 = {"none": cfg.n_ctx + 5, "middle": 100, "zero": 0}[q_pos0_kind]
    desc = kvc.desc_from_config(cfg, q_pos0=q_pos0)
    check_all(wl, desc, cfg.budget)


def test_explicit_group_map_and_scale():
    dev = _cuda()
    cfg = W.WorkloadConfig("map", 2, 6, 3, 64, 400, 8, dtype="bf16", retention=0.25, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    m = (ctypes.c_int32 * 6)(2, 0, 1, 1, 0, 2)
    desc = kvc.desc_from_config(cfg, scale=0.2)
    desc.q_to_kv = ctypes.cast(m, ctypes.POINTER(ctypes.c_int32))
    check_all(wl, desc, cfg.budget)
    # uneven groups: KV head 0 has 4 query heads, head 1 and 2 have one each
    m2 = (ctypes.c_int32 * 6)(0, 0, 1, 0, 2, 0)
    desc.q_to_kv = ctypes.cast(m2, ctypes.POINTER(ctypes.c_int32))
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("Hq,Hkv,w,agg_task,agg_group,q_pos0", [
    (8, 2, 64, 0, 0, None),     # 256 window rows per KV head: two row tiles of two query heads
    (6, 2, 64, 0, 0, None),     # three query heads per KV head: the second row tile is short
    (14, 2, 32, 0, 1, None),    # seven query heads, tiles of four and three, group max
    (4, 1, 128, 1, 0, None),    # one query head per row tile, task mean
    (8, 2, 64, 0, 0, 700),      # the causal window mask cuts through the context
    (7, 1, 64, 1, 1, 1300),
])
def test_more_window_rows_than_one_accumulator_tile(Hq, Hkv, w, agg_task, agg_group, q_pos0):
    """A GQA group whose window rows exceed 128 is scored in row tiles of whole query heads; the
    group aggregate (Eq. 15) is then assembled from the tiles' parts."""
    dev = _cuda()
    cfg = W.WorkloadConfig("rowtiles", 2, Hq, Hkv, 128, 1500, w, dtype="bf16", retention=0.3,
                           elem_std=1.0, hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    for augment in (1, 0):
        kw = dict(agg_task=agg_task, agg_group=agg_group, augment_head_mean=augment)
        if q_pos0 is not None:
            kw["q_pos0"] = q_pos0
        desc = kvc.desc_from_config(cfg, **kw)
        check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("Hq,Hkv,w,d,N,batch,q_pos0", [
    (4, 4, 32, 128, 1000, 1, None),      # no grouping: one query head per KV head
    (8, 2, 8, 64, 2100, 2, None),        # short window, two sequences, head size 64
    (16, 2, 16, 128, 900, 1, None),      # eight query heads of 16 rows fill the accumulator exactly
    (8, 8, 128, 128, 600, 1, None),      # one query head of 128 rows per KV head
    (8, 2, 32, 128, 1300, 1, 5000),      # task-aware: the window lies after the context, nothing is masked
    (8, 2, 32, 128, 4096 + 64, 1, None), # enough runs per unit for several groups of folded records
])
def test_tensor_core_path_shapes(Hq, Hkv, w, d, N, batch, q_pos0):
    """bf16 shapes of the tensor-core scoring path: group sizes, window lengths, head sizes, batch."""
    dev = _cuda()
    cfg = W.WorkloadConfig("shapes", 2, Hq, Hkv, d, N, w, batch=batch, dtype="bf16", retention=0.3,
                           elem_std=1.0, hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    kw = {} if q_pos0 is None else {"q_pos0": q_pos0}
    desc = kvc.desc_from_config(cfg, **kw)
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("Hq,Hkv,w,agg_task,agg_group,q_pos0", [
    (8, 2, 24, 0, 0, None),      # five query heads of 24 rows would fit, four are there: 96 rows
    (8, 2, 100, 0, 0, None),     # one query head of 100 rows per row tile, four row tiles
    (4, 2, 5, 1, 1, None),       # a very short window, task mean, group max
    (4, 2, 1, 0, 0, None),       # a single window row
    (6, 2, 48, 1, 0, 700),       # two heads of 48 rows per tile and a short second tile; mask inside the context
])
def test_window_lengths_other_than_powers_of_two(Hq, Hkv, w, agg_task, agg_group, q_pos0):
    """Any window length up to 128 runs on the tensor-core path, through the variant that reads the
    length at run time."""
    dev = _cuda()
    cfg = W.WorkloadConfig("oddw", 2, Hq, Hkv, 128, 1500, w, dtype="bf16", retention=0.3, elem_std=1.0,
                           hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    kw = dict(agg_task=agg_task, agg_group=agg_group)
    if q_pos0 is not None:
        kw["q_pos0"] = q_pos0
    desc = kvc.desc_from_config(cfg, **kw)
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("Hq,Hkv,w,agg_task,agg_group,q_pos0", [
    (4, 2, 200, 0, 1, 5000),     # task-aware: 200 task tokens after the context, two row tiles per query head
    (4, 2, 300, 1, 0, 5000),     # three row tiles (the last one short), task mean, group max
    (2, 1, 1000, 0, 1, 5000),    # a thousand task tokens: eight row tiles per query head
    (4, 2, 300, 0, 1, None),     # the window is the end of the context: the causal mask runs through 300 rows
    (6, 2, 130, 1, 1, 900),      # barely more than one tile; three query heads per KV head; mask inside
])
def test_windows_longer_than_one_accumulator_tile(Hq, Hkv, w, agg_task, agg_group, q_pos0):
    """Hundreds to thousands of scoring rows per query head (the task-aware setting of Sec. 3.2.1):
    a query head is cut into row tiles of 128 rows, Eq. 14 is completed over a head's tiles."""
    dev = _cuda()
    cfg = W.WorkloadConfig("longwin", 2, Hq, Hkv, 128, 1500, w, dtype="bf16", retention=0.3, elem_std=1.0,
                           hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    kw = dict(agg_task=agg_task, agg_group=agg_group)
    if q_pos0 is not None:
        kw["q_pos0"] = q_pos0
    desc = kvc.desc_from_config(cfg, **kw)
    assert kvc.kvc_score_uses_tensor_cores(desc)
    check_all(wl, desc, cfg.budget)


@pytest.mark.parametrize("scale", [2.0, 0.5])
def test_logits_far_above_the_first_tokens(scale):
    """A large logit scale: for most window rows some token lies tens of nats above token 0, whose
    logit is the reference of the rows' pushed fixed-point sums, so those rows' statistics have to
    come from the folded (reference, sum) records instead; other rows still take the short way."""
    dev = _cuda()
    cfg = W.WorkloadConfig("steep", 2, 8, 2, 128, 1500, 32, dtype="bf16", retention=0.3, elem_std=1.0,
                           hh_frac=0.01)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg, scale=scale)
    check_all(wl, desc, cfg.budget)


def test_batch_and_strided_inputs():
    """Two sequences; K/V/Q are views into larger buffers (non-dense batch/head/token strides)."""
    dev = _cuda()
    cfg = W.WorkloadConfig("strided", 2, 4, 2, 64, 300, 8, batch=2, dtype="bf16", retention=0.35, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    Bt, Hkv, N, d, Hq, w = 2, 2, 300, 64, 4, 8
    k2, v2, q2 = [], [], []
    for l in range(cfg.n_layers):
        kb = torch.zeros((Bt, Hkv + 1, N + 7, 2 * d), dtype=wl.k[l].dtype, device=dev)
        vb = torch.zeros_like(kb)
        qb = torch.zeros((Bt, Hq, w + 3, d + 8), dtype=wl.q[l].dtype, device=dev)
        kb[:, :Hkv, :N, :d] = wl.k[l]; vb[:, :Hkv, :N, :d] = wl.v[l]; qb[:, :, :w, :d] = wl.q[l]
        k2.append(kb[:, :Hkv, :N, :d]); v2.append(vb[:, :Hkv, :N, :d]); q2.append(qb[:, :, :w, :d])
    desc = kvc.desc_from_config(cfg)
    for i in range(3):
        desc.kv_stride[i] = k2[0].stride(i)
        desc.q_stride[i] = q2[0].stride(i)
    dense = run_fused(wl, kvc.desc_from_config(cfg), cfg.budget)
    strided = run_fused(W.Workload(cfg, q2, k2, v2), desc, cfg.budget)
    for name in ("scores", "idx", "composite", "n_keep", "offsets", "k_out", "v_out"):
        assert torch.equal(getattr(dense, name).view(torch.uint8), getattr(strided, name).view(torch.uint8)), name
    check_all(wl, kvc.desc_from_config(cfg), cfg.budget)


@pytest.mark.parametrize("N,w", [(1, 1), (5, 8), (127, 4), (128, 4), (129, 4), (1024, 16), (1025, 16)])
def test_small_and_boundary_lengths(N, w):
    dev = _cuda()
    cfg = W.WorkloadConfig("edge", 2, 2, 1, 64, N, w, dtype="f32", retention=0.5, elem_std=1.0,
                           n_sinks=min(4, N), hh_frac=0.0 if N < 200 else 0.01)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    assert desc.q_pos0 == max(N - w, 0)
    check_all(wl, desc, cfg.budget)


def test_degenerate_budgets():
    dev = _cuda()
    cfg = W.WorkloadConfig("budget", 3, 4, 2, 64, 200, 8, dtype="bf16", elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    total = cfg.n_layers * cfg.n_ctx
    for budget in (0, 1, total - 1, total):
        st = run_fused(wl, desc, budget)
        n_keep = _host(st.n_keep)
        assert n_keep.sum() == budget
        Pz.assert_allocate_exact(_host(st.composite), budget, n_keep, _host(st.offsets))
        Pz.assert_gather_exact(wl, desc, _host(st.idx), n_keep, _host(st.offsets), st.k_out, st.v_out)
    # nothing evicted: every head's compressed K is a permutation of its rows
    st = run_fused(wl, desc, total)
    for l in range(cfg.n_layers):
        got = st.k_out[0].view(cfg.n_layers, 2, cfg.n_ctx, 64)[l]
        for h in range(2):
            a = sorted(map(bytes, Pz.raw_numpy(got[h])))
            b = sorted(map(bytes, Pz.raw_numpy(wl.k[l][0, h])))
            assert a == b


def test_exact_ties_are_broken_by_position_and_layer():
    """All keys identical except a sparse perturbed set: long runs of exactly equal scores.  The
    order must put equal scores in increasing position, and the budget must be handed out in
    layer order among equal composite scores."""
    dev = _cuda()
    cfg = W.WorkloadConfig("ties", 4, 8, 2, 64, 900, 8, dtype="bf16", retention=0.3, hh_mode="ties",
                           hh_frac=0.01, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    fu = run_fused(wl, desc, cfg.budget)
    S = _host(fu.scores); idx = _host(fu.idx)
    n_equal = int((np.diff(np.take_along_axis(S, idx.astype(np.int64), axis=-1), axis=-1) == 0).sum())
    assert n_equal > S.size // 2, "the tie workload should produce long runs of equal scores"
    check_all(wl, desc, cfg.budget)
    # planted composite ties across layers: allocation follows (score desc, layer asc, k asc)
    I = torch.ones((4, 1, 900), device=dev)
    I[2, 0, :10] = 2.0
    n_keep = torch.empty((1, 4), dtype=torch.int32, device=dev)
    off = torch.empty((1, 5), dtype=torch.int64, device=dev)
    ws = torch.empty(kvc.kvc_workspace_size(desc, 1000), dtype=torch.uint8, device=dev)
    kvc.kvc_allocate(desc, I, 1000, n_keep, off, ws)
    assert n_keep.cpu().tolist() == [[900, 90, 10, 0]]
    assert off.cpu().tolist() == [[0, 900, 990, 1000, 1000]]


@pytest.mark.parametrize("N", [1, 2, 31, 33, 255, 257, 400, 1000, 4095, 4097, 8191, 8192, 8193, 12345,
                               32767, 32768, 32769, 40000, 65536, 70000, 131072, 200000])
def test_ranking_alone_across_lengths_and_both_sorts(N):
    """Eqs. 17-19 on scores given by the caller: lengths on both sides of every switch of the
    ranking (places per thread, CTA size, one chunk per segment or several that are merged over one,
    two and three levels, a last chunk of any length), segments that do not start on 16 bytes, and
    values of every kind -- long runs of equal scores, both zeros, negatives, denormals, huge values."""
    dev = _cuda()
    L, Hkv = 2, 3
    cfg = W.WorkloadConfig("rank", L, Hkv, Hkv, 64, N, 1, dtype="f32", elem_std=1.0)
    desc = kvc.desc_from_config(cfg)
    g = np.random.default_rng(1234 + N)
    S = np.empty((L, 1, Hkv, N), dtype=np.float32)
    S[0, 0, 0] = g.random(N, dtype=np.float32) / max(N, 1)                  # probabilities, one exponent range
    S[0, 0, 1] = np.round(g.random(N) * 7).astype(np.float32) / 7           # eight values: long ties
    S[0, 0, 2] = np.exp(g.normal(0, 12, N)).astype(np.float32)              # forty orders of magnitude
    S[1, 0, 0] = g.normal(0, 1, N).astype(np.float32)                       # both signs
    S[1, 0, 1] = 0.25                                                       # all equal: no pass orders anything
    special = np.array([0.0, -0.0, 1e-45, -1e-45, 1.0, -1.0, 3e38, -3e38, 1e-38, 2.0 ** -31], dtype=np.float32)
    S[1, 0, 2] = special[g.integers(0, len(special), N)]
    scores = torch.from_numpy(S).to(dev)
    idx = torch.empty((L, 1, Hkv, N), dtype=torch.int32, device=dev)
    comp = torch.empty((L, 1, N), dtype=torch.float32, device=dev)
    ws = torch.empty(kvc.kvc_workspace_size(desc, 0), dtype=torch.uint8, device=dev)
    kvc.kvc_compose(desc, scores, idx, comp, ws)
    torch.cuda.synchronize()
    Pz.assert_rank_exact(S, _host(idx))
    Pz.assert_compose_exact(S, _host(idx), _host(comp), desc.agg_head)


def test_argument_errors_are_reported_not_launched():
    dev = _cuda()
    cfg = W.WorkloadConfig("err", 1, 2, 1, 64, 64, 4, dtype="f32", elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    out = alloc_outputs(desc, 10, torch.float32, dev)
    small = torch.empty(256, dtype=torch.uint8, device=dev)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_compress(desc, wl.q, wl.k, wl.v, 10, out.k_out, out.v_out, out.n_keep, out.offsets,
                         workspace=small)
    assert e.value.status == -3
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_compress(desc, wl.q, wl.k, wl.v, 65, out.k_out, out.v_out, out.n_keep, out.offsets,
                         workspace=out.workspace)
    assert e.value.status == -1
    torch.cuda.synchronize()
