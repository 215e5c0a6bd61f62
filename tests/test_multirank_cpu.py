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
