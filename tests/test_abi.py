"""The C-ABI boundary without a GPU: the library builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything could launch."""
import ctypes as C
import os
import re

import pytest
import torch

import paper_2509_05165_b200 as kvc
from paper_2509_05165_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvc.h")).read()
    return sorted(set(re.findall(r"KVC_API\s+[\w\s\*]+?\b(kvc_\w+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = C.CDLL(path)
    names = _declared_symbols()
    assert len(names) >= 11 and "kvc_compress" in names and "kvc_score" in names
    for n in names:
        assert hasattr(lib, n), "libkvc.so does not export " + n
    assert kvc.kvc_version() >= 100


def test_sources_are_blackwell_only():
    flags = " ".join(build.NVCC_FLAGS)
    assert "arch=compute_100a,code=sm_100a" in flags


def test_desc_defaults_follow_the_paper():
    d = kvc.kvc_desc_init(32, 1, 32, 8, 128, 32768, 32, kvc.BF16)
    assert (d.agg_task, d.agg_group, d.agg_head) == (kvc.AGG_MAX, kvc.AGG_MEAN, kvc.AGG_MEAN)
    assert d.augment_head_mean == 1 and d.q_pos0 == 32768 - 32 and d.scale <= 0
    assert not d.q_to_kv


def test_budget_from_ratio_matches_the_formula():
    d = kvc.kvc_desc_init(32, 1, 32, 8, 128, 32768, 32, kvc.BF16)
    assert [kvc.kvc_budget_from_ratio(d, r) for r in (0.95, 0.90, 0.75)] == [52428, 104857, 262144]
    d2 = kvc.kvc_desc_init(40, 1, 40, 8, 128, 4096, 32, kvc.BF16)
    assert kvc.kvc_budget_from_ratio(d2, 0.8) == 32768          # 0.2 * 163840 exactly
    assert kvc.kvc_budget_from_ratio(d2, 0.0) == 40 * 4096
    assert kvc.kvc_budget_from_ratio(d2, 1.0) == 0
    assert kvc.kvc_budget_from_ratio(d2, 1.5) == -1


def test_workspace_size_is_positive_and_monotone_in_n():
    a = kvc.kvc_workspace_size(kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.F32), 256)
    b = kvc.kvc_workspace_size(kvc.kvc_desc_init(2, 1, 4, 2, 64, 1024, 16, kvc.F32), 256)
    assert 0 < a < b and a % 256 == 0


@pytest.mark.parametrize("field,value,status", [
    ("n_layers", 0, -1), ("n_layers", 129, -2), ("batch", 0, -1), ("head_dim", 96, -2),
    ("window", 0, -1), ("n_ctx", 0, -1), ("n_ctx", 1 << 31, -2), ("q_pos0", -1, -1),
    ("dtype", 7, -1), ("agg_task", 2, -1), ("n_q_heads", 5, -1), ("n_kv_heads", 0, -1),
    ("value_norm", 2, -1), ("keep_position_order", -1, -1), ("min_keep_per_layer", -1, -1),
    ("min_keep_per_layer", 513, -1), ("reserved_", 1, -1),
])
def test_bad_descriptors_are_rejected(field, value, status):
    d = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.F32)
    setattr(d, field, value)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_workspace_size(d, 0)
    assert e.value.status == status
    assert kvc.kvc_last_error()


def test_bad_strides_budget_and_group_map_are_rejected():
    d = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.BF16)
    with pytest.raises(kvc.KvcError):
        kvc.kvc_workspace_size(d, 2 * 512 + 1)
    with pytest.raises(kvc.KvcError):
        kvc.kvc_workspace_size(d, -1)
    d.kv_stride[0], d.kv_stride[1], d.kv_stride[2] = 2 * 512 * 64, 512 * 64, 68    # rows 136 B apart
    with pytest.raises(kvc.KvcError):
        kvc.kvc_workspace_size(d, 10)
    d = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.BF16)
    m = (C.c_int32 * 4)(0, 0, 0, 0)                                             # KV head 1 has no member
    d.q_to_kv = C.cast(m, C.POINTER(C.c_int32))
    with pytest.raises(kvc.KvcError):
        kvc.kvc_workspace_size(d, 10)
    m = (C.c_int32 * 4)(0, 1, 2, 0)
    d.q_to_kv = C.cast(m, C.POINTER(C.c_int32))
    with pytest.raises(kvc.KvcError):
        kvc.kvc_workspace_size(d, 10)


def test_null_pointers_are_rejected_before_any_launch():
    lib = binding._load()
    d = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.F32)
    assert lib.kvc_score(C.byref(d), None, None, None, None, 0, None) == -1
    assert lib.kvc_compose(C.byref(d), None, None, None, None, 0, None) == -1
    assert lib.kvc_allocate(C.byref(d), None, 0, None, None, None, 0, None) == -1
    assert lib.kvc_gather(C.byref(d), None, None, None, None, None, 0, None, None, None) == -1
    assert lib.kvc_compress(C.byref(d), None, None, None, 0, None, None, None, None, None, None, None,
                            None, None, 0, None) == -1
    fake = (C.c_void_p * 2)(0x1000, 0x1008)          # second pointer is not 16-byte aligned
    assert lib.kvc_score(C.byref(d), fake, fake, C.c_void_p(0x1000), None, 0, None) == -1
    assert b"aligned" in lib.kvc_last_error()


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_cpu_fallback_without_a_gpu():
    """With valid arguments but no device the call fails with a CUDA error: no silent CPU path."""
    d = kvc.kvc_desc_init(1, 1, 2, 1, 64, 64, 4, kvc.F32)
    q = [torch.zeros(1, 2, 4, 64)]
    k = [torch.zeros(1, 1, 64, 64)]
    S = torch.zeros(1, 1, 1, 64)
    ws = torch.zeros(kvc.kvc_workspace_size(d, 0) + 256, dtype=torch.uint8)
    off = (-ws.data_ptr()) % 256
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_score(d, q, k, S, ws[off:])
    assert e.value.status == -4


def test_scoring_path_query_and_option_defaults():
    d = kvc.kvc_desc_init(32, 1, 32, 8, 128, 32768, 32, kvc.BF16)
    assert (d.value_norm, d.min_keep_per_layer, d.keep_position_order, d.reserved_) == (0, 0, 0, 0)
    assert kvc.kvc_score_uses_tensor_cores(d)
    assert kvc.kvc_score_uses_tensor_cores(kvc.kvc_desc_init(32, 1, 32, 8, 128, 32768, 1000, kvc.BF16))
    assert not kvc.kvc_score_uses_tensor_cores(kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.F32))
    m = (C.c_int32 * 4)(1, 0, 1, 0)
    d2 = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.BF16)
    d2.q_to_kv = C.cast(m, C.POINTER(C.c_int32))
    assert not kvc.kvc_score_uses_tensor_cores(d2)
    # the v-norm option enlarges the workspace by the value norms
    d3 = kvc.kvc_desc_init(2, 1, 4, 2, 64, 512, 16, kvc.BF16)
    a = kvc.kvc_workspace_size(d3, 10)
    d3.value_norm = 1
    assert kvc.kvc_workspace_size(d3, 10) >= a


def test_test_hooks_take_and_restore_their_settings_without_a_device():
    """The hooks only store process-wide settings; they launch nothing and need no GPU."""
    kvc.kvc_debug_select_hooks(2, 0)
    kvc.kvc_debug_select_hooks(1, 5)
    kvc.kvc_debug_select_hooks()                 # automatic choice, default bound
    kvc.kvc_debug_score_hooks(1000000, 3)
    kvc.kvc_debug_score_hooks()                  # default wait bound, nothing withheld
