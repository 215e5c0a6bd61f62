"""The scoring kernel's bounded waits: a wait that nothing ends gives up, the call returns with
KVC_ERR_TIMEOUT in its status word, and the next call on the same stream and workspace is good.

The failure is made without faulting, trapping or hanging anything: a test hook of the library
withholds the softmax statistics of one work unit (the flag that nothing sets) and shortens the
bound of the waits to 20 ms; every role of the kernel then leaves through its normal exit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import workloads as W
from paper_2509_05165_b200.binding import alloc_outputs

import parity as Pz

TIMEOUT = -5


@pytest.fixture
def hooks():
    yield kvc.kvc_debug_score_hooks
    kvc.kvc_debug_score_hooks(0, -1)          # whatever the test did, the defaults come back


@pytest.mark.parametrize("withhold_unit", [0, 3])
def test_withheld_statistics_end_in_a_timeout_status_and_the_next_call_is_good(hooks, withhold_unit):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    dev = torch.device("cuda:0")
    # two layers x two KV heads = four units of twelve tiles: 12 CTAs, several runs per unit
    cfg = W.WorkloadConfig("timeout", 2, 8, 2, 128, 1500, 32, dtype="bf16", retention=0.3, elem_std=1.0)
    wl = W.make_workload(cfg, dev)
    desc = kvc.desc_from_config(cfg)
    out = alloc_outputs(desc, cfg.budget, wl.k[0].dtype, dev)

    hooks(20_000_000, withhold_unit)
    kvc.kvc_compress(desc, wl.q, wl.k, wl.v, cfg.budget, out.k_out, out.v_out, out.n_keep, out.offsets,
                     out.idx, out.scores, out.composite, out.device_status, out.workspace)
    torch.cuda.synchronize()                   # the call returns: nothing hangs, nothing faults
    assert int(out.device_status.item()) == TIMEOUT
    # the stand-alone scoring call reports the same condition in its workspace word
    kvc.kvc_score(desc, wl.q, wl.k, out.scores, out.workspace)
    torch.cuda.synchronize()
    off = kvc.kvc_score_status_offset(desc)
    assert int(out.workspace[off:off + 4].view(torch.int32).item()) == TIMEOUT

    hooks(0, -1)
    kvc.kvc_compress(desc, wl.q, wl.k, wl.v, cfg.budget, out.k_out, out.v_out, out.n_keep, out.offsets,
                     out.idx, out.scores, out.composite, out.device_status, out.workspace)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    S_def = Pz.oracle_scores(wl, desc)
    Pz.assert_scores_close(out.scores.cpu().numpy(), S_def)
    Pz.assert_rank_exact(out.scores.cpu().numpy(), out.idx.cpu().numpy())
    assert int(out.n_keep.sum().item()) == cfg.budget
    kvc.kvc_score(desc, wl.q, wl.k, out.scores, out.workspace)
    torch.cuda.synchronize()
    assert int(out.workspace[off:off + 4].view(torch.int32).item()) == 0
