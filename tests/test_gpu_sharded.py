"""The head-sharded pass with the CUDA backend, two ranks emulated on one GPU.

Each "rank" is a Python thread that runs the real driver (run_head_sharded) on its half of the KV
heads; the all-reduce is a stand-in that meets at a host-side barrier and adds the two ranks'
tensors with a device-side add.  Nothing on the GPU waits for anything else: the two ranks' kernels
queue on one stream and run one after the other.  Checked: scores against the oracle, everything downstream exactly
against the oracle fed with the sharded pipeline's own previous step, and identical allocations on
both ranks."""
import threading

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import sharded, workloads as W

import parity as Pz


class _FakeAllReduce:
    def __init__(self, world):
        self.world, self.slots = world, [None] * world
        self.b1, self.b2 = threading.Barrier(world), threading.Barrier(world)

    def for_rank(self, rank):
        def fn(t, op):
            torch.cuda.synchronize()
            self.slots[rank] = t
            self.b1.wait()
            total = self.slots[0].clone()
            for other in self.slots[1:]:
                total = total + other if op == "sum" else torch.maximum(total, other)
            torch.cuda.synchronize()
            self.b2.wait()                      # everyone has read everyone's tensor
            t.copy_(total)
            torch.cuda.synchronize()
        return fn


@pytest.mark.parametrize("agg_head", [1, 0])
def test_two_emulated_ranks_share_the_kv_heads(agg_head):
    import oracle
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    world = 2
    cfg = W.WorkloadConfig("shard", 3, 16, 4, 128, 1500, 32, dtype="bf16", retention=0.3, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    Hl, G = cfg.n_kv_heads // world, cfg.group
    local_cfg = cfg.replace(n_q_heads=cfg.n_q_heads // world, n_kv_heads=Hl)
    fake = _FakeAllReduce(world)
    results, errors = [None] * world, []

    def rank_main(rank):
        try:
            torch.cuda.set_device(dev)
            # both ranks launch on the device's default stream: their kernels run one after the other
            # (the scoring kernel is a persistent grid that wants the GPU to itself)
            q = [t[:, rank * Hl * G:(rank + 1) * Hl * G].contiguous() for t in wl.q]
            k = [t[:, rank * Hl:(rank + 1) * Hl].contiguous() for t in wl.k]
            v = [t[:, rank * Hl:(rank + 1) * Hl].contiguous() for t in wl.v]
            desc = kvc.desc_from_config(local_cfg, augment_head_mean=0, agg_head=agg_head)
            be = sharded.KvcBackend(q, k, v, desc, cfg.budget, torch.cuda.default_stream(dev))
            out = sharded.run_head_sharded(be, sharded.ShardInfo(world, cfg.n_kv_heads, agg_head), fake.for_rank(rank))
            torch.cuda.synchronize()
            results[rank] = (out, k, v, desc)
        except Exception as e:  # noqa: BLE001
            errors.append(e)
            fake.b1.abort(); fake.b2.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(world)]
    for t in threads: t.start()
    for t in threads: t.join(timeout=120)
    assert not errors, errors
    outs = [r[0] for r in results]
    # the allocation is replicated
    assert torch.equal(outs[0].n_keep, outs[1].n_keep) and torch.equal(outs[0].offsets, outs[1].offsets)
    assert int(outs[0].n_keep.sum()) == cfg.budget
    # scores of all heads against the all-double oracle
    S = np.concatenate([o.scores.cpu().numpy() for o in outs], axis=2)
    S_def = Pz.oracle_scores(wl, kvc.desc_from_config(cfg))
    Pz.assert_scores_close(S, S_def)
    # staged: ranking of the sharded scores, composite = mean (or max) over ALL heads to fp32 rounding,
    # allocation exact from the reduced composite, gather exact on every rank's heads
    idx = np.concatenate([o.idx.cpu().numpy() for o in outs], axis=2)
    Pz.assert_rank_exact(S, idx)
    I = outs[0].composite.cpu().numpy()
    assert torch.equal(outs[0].composite, outs[1].composite)
    Ss = np.take_along_axis(S, idx.astype(np.int64), axis=-1).astype(np.float64)
    want = Ss.mean(axis=2) if agg_head == 1 else Ss.max(axis=2)
    assert np.allclose(I, want, rtol=1e-5, atol=0)
    n_keep, off = outs[0].n_keep.cpu().numpy(), outs[0].offsets.cpu().numpy()
    Pz.assert_allocate_exact(I, cfg.budget, n_keep, off)
    for rank, (out, k, v, desc) in enumerate(results):
        Pz.assert_gather_exact(W.Workload(local_cfg, None, k, v), desc, out.idx.cpu().numpy(), n_keep, off,
                               out.k_out, out.v_out)
