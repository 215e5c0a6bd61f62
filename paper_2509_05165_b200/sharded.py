"""One sequence's KV heads sharded over several ranks (tensor-parallel serving).

Scoring (Eqs. 3, 14, 15) and ranking (Eq. 17) are per head and stay on the rank that holds the
head.  Two steps need all heads of a layer: the head-mean term of Eq. 16 and the aggregation over
heads of Eq. 19; each is one all-reduce of an [L, batch, N] fp32 tensor.  The budget allocation
(Eqs. 20-22) then runs replicated on identical inputs, and every rank gathers its own heads
(Eqs. 23-24).  The paper has no multi-GPU formulation; this is the same arithmetic with two sums
taken in another order, so results agree with the single-GPU pass to fp32 rounding.

``run_head_sharded`` is the rank-local driver.  It is written against a small backend interface
so that the exchange logic can be exercised without GPUs: ``KvcBackend`` runs the steps in the CUDA
library; the tests supply a CPU backend built on the oracle and run two gloo ranks.
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Optional

import torch


class KvcBackend:
    """The steps of the pass on this rank's heads, in the CUDA library (argument marshalling only)."""

    def __init__(self, q, k, v, desc_local, budget: int, stream=None):
        from . import binding as B

        self.B, self.q, self.k, self.v, self.desc, self.budget, self.stream = B, q, k, v, desc_local, budget, stream
        if desc_local.augment_head_mean:
            raise ValueError("the local descriptor must have augment_head_mean = 0: Eq. 16 is completed across ranks")
        self.out = B.alloc_outputs(desc_local, budget, k[0].dtype, k[0].device)
        L, Bt, N = desc_local.n_layers, desc_local.batch, desc_local.n_ctx
        self.head_sum = torch.empty((L, Bt, N), dtype=torch.float32, device=k[0].device)

    def local_head_sum(self) -> torch.Tensor:
        o = self.out
        self.B.kvc_score(self.desc, self.q, self.k, o.scores, o.workspace, self.stream)       # Eq. 15 (no Eq. 16)
        self.B.kvc_head_sum(self.desc, o.scores, self.head_sum, self.stream)
        return self.head_sum

    def local_composite(self, head_sum_all: torch.Tensor, n_kv_heads_total: int) -> torch.Tensor:
        o = self.out
        self.B.kvc_add_head_mean(self.desc, o.scores, head_sum_all, n_kv_heads_total, self.stream)   # Eq. 16
        self.B.kvc_compose(self.desc, o.scores, o.idx, o.composite, o.workspace, self.stream)          # Eqs. 17-19, local heads
        return o.composite

    def scale(self, x: torch.Tensor, factor: float) -> None:
        self.B.kvc_scale(x, factor, self.stream)

    def finish(self, composite_all: torch.Tensor):
        o = self.out
        self.B.kvc_allocate(self.desc, composite_all, self.budget, o.n_keep, o.offsets, o.workspace, self.stream)
        if self.desc.keep_position_order:
            self.B.kvc_order_kept(self.desc, o.idx, o.n_keep, o.workspace, self.stream)
        self.B.kvc_gather(self.desc, self.k, self.v, o.idx, o.n_keep, o.offsets, self.budget, o.k_out, o.v_out,
                          self.stream)
        return o


@dataclasses.dataclass
class ShardInfo:
    ranks: int                 # ranks the heads are split over (equal shares)
    n_kv_heads_total: int
    agg_head: int              # 0 = max, 1 = mean (Eq. 19)


def run_head_sharded(backend, info: ShardInfo, all_reduce: Callable[[torch.Tensor, str], None]):
    """The pass on this rank's heads.  ``all_reduce(tensor, op)`` reduces in place over the ranks
    that share the sequence, op being "sum" or "max" (torch.distributed.all_reduce in production)."""
    head_sum = backend.local_head_sum()
    all_reduce(head_sum, "sum")                                    # Eq. 16: all KV heads of the layer
    composite = backend.local_composite(head_sum, info.n_kv_heads_total)
    if info.agg_head == 0:
        all_reduce(composite, "max")                               # Eq. 19 with max-pooling
    else:
        all_reduce(composite, "sum")                               # Eq. 19: mean of the ranks' means (equal shares)
        backend.scale(composite, 1.0 / info.ranks)
    return backend.finish(composite)


def torch_all_reduce(group=None) -> Callable[[torch.Tensor, str], None]:
    import torch.distributed as dist

    def fn(t: torch.Tensor, op: str) -> None:
        dist.all_reduce(t, op=dist.ReduceOp.SUM if op == "sum" else dist.ReduceOp.MAX, group=group)

    return fn


def compress_head_sharded(q, k, v, desc_local, budget: int, n_kv_heads_total: int, group=None,
                          stream: Optional[torch.cuda.Stream] = None):
    """Convenience entry: this rank's Q/K/V hold its own heads; returns the binding's CompressOutputs
    for those heads (n_keep / offsets are identical on all ranks)."""
    import torch.distributed as dist

    ranks = dist.get_world_size(group)
    assert n_kv_heads_total == ranks * desc_local.n_kv_heads, "equal shares of the KV heads per rank"
    backend = KvcBackend(q, k, v, desc_local, budget, stream)
    return run_head_sharded(backend, ShardInfo(ranks, n_kv_heads_total, desc_local.agg_head), torch_all_reduce(group))
