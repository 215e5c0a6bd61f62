#!/usr/bin/env python
"""Benchmark of the KVCompose compression pass on B200.

One "step" is one whole pass (score -> rank/compose -> allocate -> gather, the fused
kvc_compress entry) over one synthetic prefilled KV cache.  The default workload is the
LLaMA-3.1-8B-shaped cache at N = 32768, window 32, 25 % retention (the configuration the
>= 70 %-of-HBM-roofline target is stated on); --workload picks another one.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--retention R]
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...   (N > 1)
  python bench.py --impl reference ...      # the CPU oracle on the host cores, same metric
  python bench.py --sweep                   # the N x batch x retention sweep on the 8B shape, one JSON line per point
                                            # (points that do not fit the free device memory are recorded as skipped)

Prints ONE JSON line on rank 0.  Multi-GPU: every rank compresses its own sequence (weak
scaling, no data-path collective); the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "context_tokens_per_sec_compressed_end_to_end"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="kvc", choices=["kvc", "reference"])
    ap.add_argument("--workload", default="llama8b_32k")
    ap.add_argument("--retention", type=float, default=None)
    ap.add_argument("--n-ctx", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--layers", type=int, default=None, help="fewer layers of the same shape (profiling captures)")
    ap.add_argument("--elem-std", type=float, default=None)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU work of the oracle leg")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the second, long timed region (0 = leave it out)")
    ap.add_argument("--sweep", action="store_true", help="run the N x batch x retention sweep instead of one workload")
    return ap.parse_args()


def pick_config(args):
    from paper_2509_05165_b200 import workloads as W

    cfg = W.CONFIGS[args.workload]
    kw = {}
    if args.retention is not None:
        kw["retention"] = args.retention
    if args.n_ctx is not None:
        kw["n_ctx"] = args.n_ctx
    if args.batch is not None:
        kw["batch"] = args.batch
    if args.layers is not None:
        kw["n_layers"] = args.layers
        kw["name"] = "%s_L%d" % (cfg.name, args.layers)
    if args.elem_std is not None:
        kw["elem_std"] = args.elem_std
    return cfg.replace(**kw) if kw else cfg


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:  # noqa: BLE001
            pass
    return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(cfg):
    """Bytes the method has to move per pass (all sequences of this rank)."""
    e = 2 if cfg.dtype == "bf16" else 4
    kv = cfg.n_layers * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim * e
    q = cfg.n_layers * cfg.n_q_heads * cfg.window * cfg.head_dim * e
    rho = cfg.budget / float(cfg.n_layers * cfg.n_ctx)
    return dict(score=cfg.batch * (kv + q), gather=cfg.batch * 4 * rho * kv,
                total=cfg.batch * (kv * (1 + 4 * rho) + q))


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "200"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:  # noqa: BLE001
            self.p = None

    def stop(self):
        if self.p is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        time.sleep(0.25)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:  # noqa: BLE001
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def gpu_id(local_rank):
    """nvidia-smi identifier of the torch device (the UUID survives CUDA_VISIBLE_DEVICES remapping)."""
    try:
        return "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:  # noqa: BLE001
        return str(local_rank)


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_sample(cfg, n_layers_sample):
    """Host copies of the first layers of the workload, in the form the oracle takes."""
    from paper_2509_05165_b200 import workloads as W

    dev = "cuda" if torch.cuda.is_available() else "cpu"
    wl = W.make_workload(cfg.replace(batch=1), dev, layers=range(n_layers_sample))
    q = np.stack([t[0].float().cpu().numpy() for t in wl.q])
    k = np.stack([t[0].float().cpu().numpy() for t in wl.k])
    view = torch.int16 if cfg.dtype == "bf16" else torch.float32
    kr = np.stack([t[0].view(view).cpu().numpy() for t in wl.k])
    vr = np.stack([t[0].view(view).cpu().numpy() for t in wl.v])
    return q, k, kr, vr


def time_oracle(cfg, q, k, kr, vr):
    import oracle

    Ls = q.shape[0]
    budget = int(cfg.retention * Ls * cfg.n_ctx)
    t0 = time.perf_counter()
    oracle.compress(q, k, kr, vr, 1.0 / np.sqrt(cfg.head_dim), cfg.n_ctx - cfg.window, budget,
                    want_scores=False)
    return time.perf_counter() - t0


def parity_summary(cfg, gpu_scores, gpu_idx):
    """The GPU's scores and order of layer 0, sequence 0 against the all-double oracle (part of the
    oracle leg, outside every timed region): largest relative score error, positions where the order
    differs with the largest oracle score gap among them, and the smallest gap where both agree."""
    import oracle

    q, k, _, _ = oracle_sample(cfg, 1)
    S_def = oracle.score_layer(q[0], k[0], 1.0 / np.sqrt(cfg.head_dim), cfg.n_ctx - cfg.window)
    S_gpu = gpu_scores.astype(np.float64)
    rel = np.abs(S_gpu - S_def) / np.maximum(np.abs(S_def), 1e-300)
    n_diff, max_gap, margin = 0, 0.0, float("inf")
    for h in range(S_def.shape[0]):
        ref, Ss = oracle.rank(S_def[h])
        diff = ref != gpu_idx[h]
        n_diff += int(diff.sum())
        if diff.any():
            x, y = S_def[h][ref[diff]], S_def[h][gpu_idx[h][diff]]
            max_gap = max(max_gap, float((np.abs(x - y) / np.maximum(x, y)).max()))
        agree = ~diff[:-1] & ~diff[1:]
        if agree.any():
            margin = min(margin, float(((Ss[:-1] - Ss[1:])[agree] / Ss[:-1][agree]).min()))
    return dict(layer=0, tolerance=1e-3, max_rel_score_err=float(rel[S_def > 0].max()), n_order_diff=n_diff,
                max_gap_at_diff=max_gap, tie_margin=margin,
                ok=bool(rel[S_def > 0].max() <= 1e-3 and max_gap < 2e-3))


def cpu_baseline(cfg, target_seconds):
    """The oracle as it stands, on the host cores, on the first layers of the same workload."""
    import oracle

    cores = host_cores()
    oracle.set_threads(cores)
    q, k, kr, vr = oracle_sample(cfg, 1)
    t1 = time_oracle(cfg, q, k, kr, vr)
    Ls = int(max(1, min(cfg.n_layers, round(target_seconds / max(t1, 1e-3)))))
    if Ls > 1:
        q, k, kr, vr = oracle_sample(cfg, Ls)
        t = time_oracle(cfg, q, k, kr, vr)
    else:
        t = t1
    per_pass = t * cfg.n_layers / Ls          # linear in the number of layers
    return dict(value=cfg.n_ctx / per_pass, unit=UNIT, cores=cores, kind="oracle",
                sample="%d of %d layers of %s, one sequence, whole pass incl. gather: %.2f s measured, "
                       "scaled linearly to all layers" % (Ls, cfg.n_layers, cfg.name, t),
                seconds_measured=t, extrapolated=Ls < cfg.n_layers)


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only).  A step is the oracle's
    whole pass over the first layers of the workload (two of them by default: the full workload would take
    minutes per step); value and ms_per_step are scaled linearly to all layers and marked as extrapolated,
    the measured time of a step is reported beside them."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle

    cfg = pick_config(args)
    cores = host_cores()
    oracle.set_threads(cores)
    Ls = min(cfg.n_layers, 2)
    q, k, kr, vr = oracle_sample(cfg, Ls)
    for _ in range(args.warmup):
        time_oracle(cfg, q, k, kr, vr)
    times = [time_oracle(cfg, q, k, kr, vr) for _ in range(args.steps)]
    t_step = sum(times) / len(times)
    value = cfg.n_ctx / (t_step * cfg.n_layers / Ls)
    sample = "%d of %d layers of %s per step, one sequence, scaled linearly to all layers" % (Ls, cfg.n_layers, cfg.name)
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=t_step * 1e3 * cfg.n_layers / Ls, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(cfg, 1), extrapolated=Ls < cfg.n_layers, layers_timed=Ls,
                ms_per_step_measured=t_step * 1e3,
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample,
                                  extrapolated=Ls < cfg.n_layers),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def rank_workload(cfg, rank):
    """Sequences are sharded over the ranks: rank r compresses its own sequence(s), drawn from seed r."""
    return cfg.replace(seed=rank)


def aggregate_tokens_per_s(cfg, world, ms_per_step):
    """Whole-job throughput: every rank holds cfg.batch sequences of cfg.n_ctx context tokens."""
    return cfg.batch * cfg.n_ctx * world / (ms_per_step * 1e-3)


SCORE_SOURCE = os.path.join(ROOT, "paper_2509_05165_b200", "csrc", "score_sm100.cu")
SCORE_PROFILE = os.path.join(ROOT, "profiles", "score_sm100_llama8b_32k_L4.txt")


def score_traffic_bytes(cfg):
    """DRAM traffic of one launch of the scoring kernel on this workload, from the ncu capture summarised in
    profiles/ (dram__bytes_read.sum + dram__bytes_write.sum of a 4-layer capture of the same shape, scaled to
    the workload's layers: the traffic is proportional to them).  None for any other shape, and None as soon
    as the kernel's source is no longer the one the capture was taken on (the summary records its hash)."""
    if not cfg.name.startswith("llama8b_32k") or cfg.n_ctx != 32768 or cfg.batch != 1:
        return None
    try:
        text = open(SCORE_PROFILE).read()
        sha = re.search(r"source_sha256:\s*([0-9a-f]{64})", text).group(1)
        rd = int(re.search(r"dram_bytes_read_per_launch:\s*(\d+)", text).group(1))
        wr = int(re.search(r"dram_bytes_write_per_launch:\s*(\d+)", text).group(1))
        layers = int(re.search(r"capture_layers:\s*(\d+)", text).group(1))
        if hashlib.sha256(open(SCORE_SOURCE, "rb").read()).hexdigest() != sha:
            return None
        return (rd + wr) * cfg.n_layers // layers
    except Exception:  # noqa: BLE001
        return None


def workload_config(cfg, world):
    return dict(workload=cfg.name, n_layers=cfg.n_layers, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                head_dim=cfg.head_dim, n_ctx=cfg.n_ctx, window=cfg.window, batch_per_gpu=cfg.batch,
                retention=cfg.retention, budget_per_sequence=cfg.budget, elem_std=cfg.elem_std,
                sequences_total=cfg.batch * world,
                l2="inputs (%.2f GB of K/V per GPU) exceed the 126 MB L2; no flush needed" %
                   (2 * cfg.batch * cfg.n_layers * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim *
                    (2 if cfg.dtype == "bf16" else 4) / 1e9))


def device_bytes_needed(cfg):
    """Device memory one run of the benchmark holds for this workload: inputs, outputs, workspace, and the
    kept intermediates of the per-stage timing."""
    import paper_2509_05165_b200 as kvc

    e = 2 if cfg.dtype == "bf16" else 4
    kv = 2 * cfg.batch * cfg.n_layers * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim * e
    q = cfg.batch * cfg.n_layers * cfg.n_q_heads * cfg.window * cfg.head_dim * e
    outs = 2 * 2 * cfg.batch * cfg.budget * cfg.n_kv_heads * cfg.head_dim * e
    inter = cfg.batch * cfg.n_layers * cfg.n_ctx * (8 * cfg.n_kv_heads + 4)
    ws = kvc.kvc_workspace_size(kvc.desc_from_config(cfg), cfg.budget)
    draw = cfg.batch * cfg.n_kv_heads * cfg.n_ctx * cfg.head_dim * 4 * 4      # fp32 temporaries of the generator
    return kv + q + outs + inter + ws + draw


def run_workload(args, cfg, world, rank, local_rank, dev, dist):
    """Times one workload; returns the JSON line as a dict on rank 0 (None elsewhere)."""
    import paper_2509_05165_b200 as kvc
    from paper_2509_05165_b200 import workloads as W
    from paper_2509_05165_b200.binding import alloc_outputs

    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    budget = cfg.budget
    out = alloc_outputs(desc, budget, wl.k[0].dtype, dev, keep_intermediates=False)
    stream = torch.cuda.current_stream()

    def step():
        kvc.kvc_compress(desc, wl.q, wl.k, wl.v, budget, out.k_out, out.v_out, out.n_keep, out.offsets,
                         None, None, None, out.device_status, out.workspace, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(n):
        """n passes back to back between two events; ms per pass, max over ranks."""
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for _ in range(n):
            step()
        ev1.record(stream)
        barrier()
        return max_over_ranks([ev0.elapsed_time(ev1) / n], dist, dev)[0]

    # ---- device-resident timing: exactly --steps passes (a burst of a few tens of milliseconds) ...
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # (the clocks are sampled every 200 ms from before the first timed pass to after the last one of the
    # long region: the --steps region alone is shorter than one sampling period)
    sampler = ClockSampler(gpu_id(local_rank)) if rank == 0 else None
    if sampler:
        time.sleep(0.3)                      # let the sampler come up before anything is timed
    kvc.kvc_launch_count(reset=True)
    ms_per_step = timed(args.steps)
    launches = kvc.kvc_launch_count()
    assert int(out.device_status.item()) == 0
    # ---- ... and a long region (seconds: the clocks settle under the power cap)
    sustained = None
    if args.sustained_seconds > 0:
        n_long = max(args.steps, int(args.sustained_seconds * 1e3 / ms_per_step))
        sustained = dict(steps=n_long, ms_per_step=timed(n_long))
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["covers"] = "the %d-step region and the sustained region after it" % args.steps

    # ---- per-stage timing (the stage entry points, events between them)
    inter = alloc_outputs(desc, budget, wl.k[0].dtype, dev, keep_intermediates=True, workspace=out.workspace)
    names = ["score", "compose", "allocate", "gather"]
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    barrier()
    for st in range(args.steps):
        e = evs[st]
        e[0].record(stream)
        kvc.kvc_score(desc, wl.q, wl.k, inter.scores, out.workspace, stream); e[1].record(stream)
        kvc.kvc_compose(desc, inter.scores, inter.idx, inter.composite, out.workspace, stream); e[2].record(stream)
        kvc.kvc_allocate(desc, inter.composite, budget, inter.n_keep, inter.offsets, out.workspace, stream); e[3].record(stream)
        kvc.kvc_gather(desc, wl.k, wl.v, inter.idx, inter.n_keep, inter.offsets, budget, inter.k_out, inter.v_out, stream)
        e[4].record(stream)
    barrier()
    stage_ms = {n: sum(e[i].elapsed_time(e[i + 1]) for e in evs) / args.steps for i, n in enumerate(names)}
    gpu_scores0 = inter.scores[0, 0].cpu().numpy() if rank == 0 else None       # layer 0, sequence 0
    gpu_idx0 = inter.idx[0, 0].cpu().numpy() if rank == 0 else None
    del inter

    # ---- end to end: pinned host inputs -> device, pass, results -> pinned host
    e2e = None
    if not args.no_e2e:
        hq = [t.cpu().pin_memory() for t in wl.q]
        hk = [t.cpu().pin_memory() for t in wl.k]
        hv = [t.cpu().pin_memory() for t in wl.v]
        h_kout = torch.empty(out.k_out.shape, dtype=out.k_out.dtype).pin_memory()
        h_vout = torch.empty(out.v_out.shape, dtype=out.v_out.dtype).pin_memory()
        h_nkeep = torch.empty(out.n_keep.shape, dtype=out.n_keep.dtype).pin_memory()
        h_off = torch.empty(out.offsets.shape, dtype=out.offsets.dtype).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in hq + hk + hv)
        d2h = sum(t.numel() * t.element_size() for t in (h_kout, h_vout, h_nkeep, h_off))

        def e2e_step():
            for l in range(cfg.n_layers):
                wl.q[l].copy_(hq[l], non_blocking=True)
                wl.k[l].copy_(hk[l], non_blocking=True)
                wl.v[l].copy_(hv[l], non_blocking=True)
            step()
            h_kout.copy_(out.k_out, non_blocking=True)
            h_vout.copy_(out.v_out, non_blocking=True)
            h_nkeep.copy_(out.n_keep, non_blocking=True)
            h_off.copy_(out.offsets, non_blocking=True)

        e2e_steps = max(3, min(args.steps, 10))
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        f1.record(stream)
        barrier()
        e2e_ms = max(f0.elapsed_time(f1), (time.perf_counter() - t0) * 1e3) / e2e_steps
        assert int(h_nkeep.sum()) == budget * cfg.batch
        e2e = dict(ms=e2e_ms, h2d=h2d, d2h=d2h, steps=e2e_steps)
        del hq, hk, hv, h_kout, h_vout

    # ---- max over ranks
    t = max_over_ranks([e2e["ms"] if e2e else 0.0] + [stage_ms[n] for n in names], dist, dev)
    e2e_ms = t[0]
    stage_ms = {n: t[1 + i] for i, n in enumerate(names)}
    if rank != 0:
        return None

    tokens = cfg.batch * cfg.n_ctx * world
    value = aggregate_tokens_per_s(cfg, world, ms_per_step)
    peak, peak_kind = measured_peaks()
    ab = algorithmic_bytes(cfg)
    dominant = max(("score", "gather"), key=lambda n: stage_ms[n])
    ach = ab[dominant] / (stage_ms[dominant] * 1e-3) / 1e9

    def pass_frac(ms):
        return ab["total"] / (ms * 1e-3) / 1e9 / peak

    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
        ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16" if cfg.dtype == "bf16" else "f32", data="synthetic",
        config=workload_config(cfg, world), clocks=clocks, gpu_launches=int(launches),
        stage_ms=stage_ms,
        pass_roofline=dict(bytes=ab["total"], achieved=ab["total"] / (ms_per_step * 1e-3) / 1e9, peak=peak,
                           unit="GB/s", frac=pass_frac(ms_per_step), peak_kind=peak_kind,
                           frac_of_8tbs=ab["total"] / (ms_per_step * 1e-3) / 8e12,
                           note="burst: %d passes back to back" % args.steps),
        roofline=dict(bound="hbm", kernel=dominant, achieved=ach, peak=peak, unit="GB/s", frac=ach / peak,
                      traffic=score_traffic_bytes(cfg) if dominant == "score" else None,
                      peak_kind=peak_kind, algorithmic_bytes=ab[dominant]),
    )
    if sustained:
        line["sustained"] = dict(steps=sustained["steps"], ms_per_step=sustained["ms_per_step"],
                                 value=aggregate_tokens_per_s(cfg, world, sustained["ms_per_step"]),
                                 pass_roofline_frac=pass_frac(sustained["ms_per_step"]))
    if e2e:
        line["e2e"] = dict(value=tokens / (e2e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=e2e["h2d"],
                           d2h_bytes_per_step=e2e["d2h"], ms_per_step=e2e_ms, steps=e2e["steps"])
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, args.cpu_seconds)
        line["parity"] = parity_summary(cfg, gpu_scores0, gpu_idx0)
    return line


SWEEP_N = (4096, 16384, 65536, 131072)
SWEEP_BATCH = (1, 4, 8)
SWEEP_RETENTION = (0.05, 0.10, 0.25, 0.50)


def run_sweep(args, world, rank, local_rank, dev, dist):
    """The N x batch x retention sweep on the 8B shape: one JSON line per point.  A point whose inputs,
    outputs and workspace do not fit the free device memory is recorded as skipped, not attempted."""
    from paper_2509_05165_b200 import workloads as W

    args.no_e2e = True
    args.no_cpu_baseline = True
    args.sustained_seconds = 0.0
    for n_ctx in SWEEP_N:
        for batch in SWEEP_BATCH:
            for ret in SWEEP_RETENTION:
                cfg = rank_workload(W.sweep_config(n_ctx, batch, ret), rank)
                free, _ = torch.cuda.mem_get_info()
                need = device_bytes_needed(cfg)
                fits = max_over_ranks([1.0 if need > 0.92 * free else 0.0], dist, dev)[0] == 0.0
                if not fits:
                    if rank == 0:
                        print(json.dumps(dict(metric=METRIC, config=workload_config(cfg, world), value=None,
                                              skipped="memory", bytes_needed=need, bytes_free=free)), flush=True)
                    continue
                line = run_workload(args, cfg, world, rank, local_rank, dev, dist)
                if rank == 0:
                    keep = ("metric", "value", "unit", "n_gpus", "steps", "ms_per_step", "config", "stage_ms", "pass_roofline")
                    print(json.dumps({k: line[k] for k in keep}), flush=True)
                torch.cuda.empty_cache()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    if args.sweep:
        run_sweep(args, world, rank, local_rank, dev, dist)
    else:
        cfg = rank_workload(pick_config(args), rank)
        line = run_workload(args, cfg, world, rank, local_rank, dev, dist)
        if rank == 0:
            print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
