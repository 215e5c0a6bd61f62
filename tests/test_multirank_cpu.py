"""The multi-rank logic of the benchmark on CPU: two gloo ranks shard the sequences (each rank
draws and would compress its own), reduce their times with a maximum, and rank 0 reports the
whole-job throughput.  The path has no data-path collective, so this is all there is to it."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2509_05165_b200 import workloads as W

    base = W.WorkloadConfig("mr", 2, 4, 2, 64, 256, 8, dtype="f32", retention=0.25, elem_std=1.0)
    cfg = bench.rank_workload(base, rank)
    wl = W.make_workload(cfg, "cpu")
    fingerprint = float(wl.k[0].double().sum())
    # every rank reports its own (fake) timings; the job's time is the slowest rank's
    mine = [10.0 + rank, 5.0 - rank, 1.0]
    red = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    gathered = [None] * world
    dist.all_gather_object(gathered, fingerprint)
    if rank == 0:
        torch.save(dict(red=red, fingerprints=gathered,
                        value=bench.aggregate_tokens_per_s(cfg, world, red[0])), os.path.join(out_dir, "r0.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_and_take_the_slowest_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = torch.load(os.path.join(str(tmp_path), "r0.pt"))
    assert r["red"] == [11.0, 5.0, 1.0]                       # element-wise max over the two ranks
    assert r["fingerprints"][0] != r["fingerprints"][1]       # different sequences on different ranks
    assert r["value"] == pytest.approx(2 * 256 / 11.0e-3)     # both ranks' tokens over the slowest time


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench

    monkeypatch.setenv("RANK", "1")
    args = type("A", (), dict(workload="tiny", retention=None, n_ctx=None, batch=None, layers=None,
                              elem_std=None, gpus=2, steps=1, warmup=0))()
    bench.run_reference(args)
    assert capsys.readouterr().out == ""                      # other ranks leave without work


# ---- one sequence's KV heads sharded over two ranks (the driver of paper_2509_05165_b200/sharded.py) ----

class _OracleBackend:
    """The rank-local steps on the CPU, from the oracle (test infrastructure), so that the exchange
    logic of run_head_sharded can be run by two gloo ranks without GPUs."""

    def __init__(self, q, k, v_raw, k_raw, scale, q_pos0, budget, heads_total):
        import numpy as np
        self.np, self.q, self.k, self.k_raw, self.v_raw = np, q, k, k_raw, v_raw
        self.logit_scale, self.q_pos0, self.budget, self.heads_total = scale, q_pos0, budget, heads_total

    def local_head_sum(self):
        import oracle
        np = self.np
        L = self.q.shape[0]
        self.S = np.stack([oracle.score_layer(self.q[l], self.k[l], self.logit_scale, self.q_pos0, augment=False) for l in range(L)])
        return torch.from_numpy(self.S.sum(axis=1))[:, None, :].contiguous()          # [L, 1, N]

    def local_composite(self, head_sum_all, n_kv_heads_total):
        import oracle
        np = self.np
        self.S = self.S + head_sum_all.numpy()[:, 0][:, None, :] / n_kv_heads_total  # Eq. 16
        L, H, N = self.S.shape
        self.idx = np.empty((L, H, N), dtype=np.int32)
        Ss = np.empty((L, H, N))
        for l in range(L):
            for h in range(H):
                self.idx[l, h], Ss[l, h] = oracle.rank(self.S[l, h])
        return torch.from_numpy(np.stack([oracle.compose(Ss[l]) for l in range(L)]))[:, None, :].contiguous()

    def scale(self, x, f):
        x.mul_(f)

    def finish(self, composite_all):
        import oracle
        n_keep, off = oracle.allocate(composite_all.numpy()[:, 0], self.budget)
        return dict(S=self.S, idx=self.idx, n_keep=n_keep, offsets=off, composite=composite_all.numpy()[:, 0])


def _sharded_worker(rank, world, port, out_dir):
    import numpy as np
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2509_05165_b200 import sharded, workloads as W

    cfg = W.WorkloadConfig("shard", 3, 8, 4, 64, 300, 8, dtype="f32", retention=0.3, elem_std=1.0)
    wl = W.make_workload(cfg, "cpu")                       # both ranks draw the same sequence
    Hl, G = cfg.n_kv_heads // world, cfg.group
    hs = slice(rank * Hl, (rank + 1) * Hl)
    qs = slice(rank * Hl * G, (rank + 1) * Hl * G)
    q = np.stack([t[0, qs].numpy() for t in wl.q]); k = np.stack([t[0, hs].numpy() for t in wl.k])
    be = _OracleBackend(q, k, None, None, 1.0 / np.sqrt(cfg.head_dim), cfg.n_ctx - cfg.window, cfg.budget, cfg.n_kv_heads)
    res = sharded.run_head_sharded(be, sharded.ShardInfo(world, cfg.n_kv_heads, 1), sharded.torch_all_reduce())
    torch.save(res, os.path.join(out_dir, "shard%d.pt" % rank))
    dist.barrier()
    dist.destroy_process_group()


def test_kv_heads_sharded_over_two_ranks_match_the_unsharded_oracle(tmp_path, oracle):
    """Two all-reduces (Eq. 16's head sum, Eq. 19's mean over heads) are all the exchange there is:
    the ranks' results put side by side are the unsharded oracle's."""
    import numpy as np
    from paper_2509_05165_b200 import workloads as W

    world, port = 2, _free_port()
    mp.spawn(_sharded_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    parts = [torch.load(os.path.join(str(tmp_path), "shard%d.pt" % r), weights_only=False) for r in range(world)]
    cfg = W.WorkloadConfig("shard", 3, 8, 4, 64, 300, 8, dtype="f32", retention=0.3, elem_std=1.0)
    wl = W.make_workload(cfg, "cpu")
    q = np.stack([t[0].numpy() for t in wl.q]); k = np.stack([t[0].numpy() for t in wl.k])
    full = oracle.compress(q, k, None, None, 1.0 / np.sqrt(cfg.head_dim), cfg.n_ctx - cfg.window, cfg.budget)
    S = np.concatenate([p["S"] for p in parts], axis=1)
    idx = np.concatenate([p["idx"] for p in parts], axis=1)
    assert np.allclose(S, full["scores"], rtol=1e-12, atol=0)
    assert np.array_equal(idx, full["idx"])
    for p in parts:                                          # the allocation is replicated
        assert np.allclose(p["composite"], full["composite"], rtol=1e-12)
        assert np.array_equal(p["n_keep"], full["n_keep"]) and np.array_equal(p["offsets"], full["offsets"])
