"""kvc_allocate_static: the allocation step for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits -- a serving process whose device
memory is planned once at start-up, a plug-in that only ever sees the host application's
tensors -- so they cannot hand kvc_allocate a workspace.  kvc_allocate_static keeps its scratch
in a fixed array inside the library instead.  This file checks, through the C ABI, that it gives
exactly what kvc_allocate gives, on two calls in a row (the array is shared between calls and
keeps the previous call's contents, so the second call would expose a missing clear).

The file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import paper_2509_05165_b200 as kvc


def _composite(L, Bt, N, seed, dev):
    """Non-increasing rows of non-negative scores, with ties inside and across layers."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.rand((L, Bt, N), generator=g)
    x = torch.round(x * 50) / 50 * torch.rand((L, 1, 1), generator=g)      # coarse grid -> many exact ties
    x = torch.sort(x, dim=-1, descending=True).values
    return x.to(dev).contiguous()


@pytest.mark.gpu
def test_static_scratch_allocation_matches_workspace_allocation_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    L, Bt, N = 5, 3, 1000
    desc = kvc.kvc_desc_init(L, Bt, 4, 2, 64, N, 8, kvc.BF16)
    ws = torch.empty(kvc.kvc_workspace_size(desc, 0), dtype=torch.uint8, device=dev)
    for seed, budget in ((1, 1234), (2, 77), (3, L * N), (4, 0)):        # back-to-back calls, same array
        I = _composite(L, Bt, N, seed, dev)
        n_ref = torch.empty((Bt, L), dtype=torch.int32, device=dev)
        off_ref = torch.empty((Bt, L + 1), dtype=torch.int64, device=dev)
        kvc.kvc_allocate(desc, I, budget, n_ref, off_ref, ws)
        n_got = torch.full((Bt, L), -7, dtype=torch.int32, device=dev)
        off_got = torch.full((Bt, L + 1), -7, dtype=torch.int64, device=dev)
        kvc.kvc_allocate_static(desc, I, budget, n_got, off_got)
        torch.cuda.synchronize()
        assert torch.equal(n_got, n_ref), (seed, n_got.tolist(), n_ref.tolist())   # integers: exact
        assert torch.equal(off_got, off_ref)
        assert n_got.sum(dim=1).tolist() == [budget] * Bt


@pytest.mark.gpu
def test_static_scratch_at_its_largest_batch_and_on_a_side_stream():
    """64 sequences use the whole built-in array; a call on another stream than the default one
    gives the same result as long as nothing else that uses the array overlaps it."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    L, Bt, N = 3, 64, 300
    desc = kvc.kvc_desc_init(L, Bt, 4, 2, 64, N, 8, kvc.BF16)
    ws = torch.empty(kvc.kvc_workspace_size(desc, 0), dtype=torch.uint8, device=dev)
    side = torch.cuda.Stream(dev)
    for seed, budget, stream in ((5, 401, None), (6, 77, side), (7, 640, side)):
        I = _composite(L, Bt, N, seed, dev)
        n_ref = torch.empty((Bt, L), dtype=torch.int32, device=dev)
        off_ref = torch.empty((Bt, L + 1), dtype=torch.int64, device=dev)
        kvc.kvc_allocate(desc, I, budget, n_ref, off_ref, ws)
        torch.cuda.synchronize()                     # the side stream must not start before I and the reference are there
        n_got = torch.full((Bt, L), -7, dtype=torch.int32, device=dev)
        off_got = torch.full((Bt, L + 1), -7, dtype=torch.int64, device=dev)
        torch.cuda.synchronize()
        kvc.kvc_allocate_static(desc, I, budget, n_got, off_got, stream)
        torch.cuda.synchronize()
        assert torch.equal(n_got, n_ref) and torch.equal(off_got, off_ref), (seed, budget)
        assert n_got.sum(dim=1).tolist() == [budget] * Bt


def test_static_scratch_allocation_rejects_a_batch_beyond_its_maximum():
    """Host-side check, no launch: the fixed array covers 64 sequences."""
    desc = kvc.kvc_desc_init(2, 65, 4, 2, 64, 128, 8, kvc.BF16)
    t = torch.zeros(1)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_allocate_static(desc, t, 10, t, t)
    assert e.value.status == -2
    assert "KVC_STATIC_MAX_BATCH" in kvc.kvc_last_error()
