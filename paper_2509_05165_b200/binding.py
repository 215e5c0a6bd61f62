"""ctypes binding of ``include/kvc.h``: same names, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import List, Optional, Sequence

import torch

from . import build as _build

F32, BF16 = 0, 1
AGG_MAX, AGG_MEAN = 0, 1
KVC_MAX_LAYERS = 128

_STATUS = {0: "KVC_OK", -1: "KVC_ERR_INVALID_ARG", -2: "KVC_ERR_UNSUPPORTED", -3: "KVC_ERR_WORKSPACE",
           -4: "KVC_ERR_CUDA", -5: "KVC_ERR_TIMEOUT"}


class KvcError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (_STATUS.get(status, str(status)), message))
        self.status = status


class KvcDesc(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("window", C.c_int32),
        ("n_ctx", C.c_int64), ("q_pos0", C.c_int64), ("dtype", C.c_int32), ("scale", C.c_float),
        ("agg_task", C.c_int32), ("agg_group", C.c_int32), ("agg_head", C.c_int32),
        ("augment_head_mean", C.c_int32), ("q_to_kv", C.POINTER(C.c_int32)),
        ("q_stride", C.c_int64 * 3), ("kv_stride", C.c_int64 * 3),
        ("value_norm", C.c_int32), ("min_keep_per_layer", C.c_int32), ("keep_position_order", C.c_int32),
        ("reserved_", C.c_int32),
    ]


_lib = None


def library_path() -> str:
    return _build.LIB


def _load():
    """Load libkvc.so; build it first when the sources are newer and nvcc is present.
    There is no fallback: without the library every entry point raises."""
    global _lib
    if _lib is not None:
        return _lib
    if _build.is_stale():
        try:
            _build.build()
        except Exception as e:  # noqa: BLE001
            if not os.path.exists(_build.LIB):
                raise RuntimeError("libkvc.so is missing and could not be built (%s); the kvc entry "
                                   "points have no CPU or PyTorch fallback" % e) from e
    lib = C.CDLL(_build.LIB)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    dp = C.POINTER(KvcDesc)
    lib.kvc_desc_init.argtypes = [dp, i32, i32, i32, i32, i32, i64, i32, i32]
    lib.kvc_desc_init.restype = None
    lib.kvc_budget_from_ratio.argtypes = [dp, C.c_double]
    lib.kvc_budget_from_ratio.restype = i64
    lib.kvc_workspace_size.argtypes = [dp, i64, C.POINTER(sz)]
    lib.kvc_workspace_size.restype = C.c_int
    lib.kvc_score.argtypes = [dp, vp, vp, vp, vp, sz, vp]
    lib.kvc_score.restype = C.c_int
    lib.kvc_score_status_offset.argtypes = [dp, C.POINTER(sz)]
    lib.kvc_score_status_offset.restype = C.c_int
    lib.kvc_debug_score_hooks.argtypes = [i64, i32]
    lib.kvc_debug_score_hooks.restype = None
    lib.kvc_debug_select_hooks.argtypes = [i32, i32]
    lib.kvc_debug_select_hooks.restype = None
    lib.kvc_score_uses_tensor_cores.argtypes = [dp]
    lib.kvc_score_uses_tensor_cores.restype = i32
    lib.kvc_score_weighted.argtypes = [dp, vp, vp, vp, vp, vp, sz, vp]
    lib.kvc_score_weighted.restype = C.c_int
    lib.kvc_order_kept.argtypes = [dp, vp, vp, vp, sz, vp]
    lib.kvc_order_kept.restype = C.c_int
    lib.kvc_select_unstructured.argtypes = [dp, vp, i64, vp, vp, vp, vp, sz, vp]
    lib.kvc_select_unstructured.restype = C.c_int
    lib.kvc_gather_unstructured.argtypes = [dp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.kvc_gather_unstructured.restype = C.c_int
    lib.kvc_compress_unstructured.argtypes = [dp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.kvc_compress_unstructured.restype = C.c_int
    lib.kvc_head_sum.argtypes = [dp, vp, vp, vp]
    lib.kvc_head_sum.restype = C.c_int
    lib.kvc_add_head_mean.argtypes = [dp, vp, vp, i32, vp]
    lib.kvc_add_head_mean.restype = C.c_int
    lib.kvc_scale.argtypes = [vp, i64, C.c_float, vp]
    lib.kvc_scale.restype = C.c_int
    lib.kvc_compose.argtypes = [dp, vp, vp, vp, vp, sz, vp]
    lib.kvc_compose.restype = C.c_int
    lib.kvc_allocate.argtypes = [dp, vp, i64, vp, vp, vp, sz, vp]
    lib.kvc_allocate.restype = C.c_int
    lib.kvc_allocate_static.argtypes = [dp, vp, i64, vp, vp, vp]
    lib.kvc_allocate_static.restype = C.c_int
    lib.kvc_gather.argtypes = [dp, vp, vp, vp, vp, vp, i64, vp, vp, vp]
    lib.kvc_gather.restype = C.c_int
    lib.kvc_compress.argtypes = [dp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.kvc_compress.restype = C.c_int
    lib.kvc_last_error.restype = C.c_char_p
    lib.kvc_launch_count.argtypes = [i32]
    lib.kvc_launch_count.restype = i64
    lib.kvc_version.restype = i32
    _lib = lib
    return lib


def _check(status: int) -> None:
    if status != 0:
        raise KvcError(status, _load().kvc_last_error().decode())


def _dptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _ptr_array(ts: Sequence[torch.Tensor]):
    arr = (C.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
    return arr


def _stream(stream) -> C.c_void_p:
    if stream is None:
        if not torch.cuda.is_available():
            return C.c_void_p(None)      # argument errors are still reported; nothing can launch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _ws(ws: Optional[torch.Tensor]):
    if ws is None:
        return None, 0
    return C.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size()


# ---- the C entry points, one to one ------------------------------------------------------------

def kvc_desc_init(n_layers, batch, n_q_heads, n_kv_heads, head_dim, n_ctx, window, dtype) -> KvcDesc:
    d = KvcDesc()
    _load().kvc_desc_init(C.byref(d), n_layers, batch, n_q_heads, n_kv_heads, head_dim, n_ctx, window, dtype)
    return d


def kvc_budget_from_ratio(desc: KvcDesc, r_target: float) -> int:
    return int(_load().kvc_budget_from_ratio(C.byref(desc), float(r_target)))


def kvc_workspace_size(desc: KvcDesc, budget: int) -> int:
    out = C.c_size_t(0)
    _check(_load().kvc_workspace_size(C.byref(desc), int(budget), C.byref(out)))
    return int(out.value)


def kvc_score(desc, q: Sequence[torch.Tensor], k: Sequence[torch.Tensor], scores: torch.Tensor,
              workspace: torch.Tensor, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_score(C.byref(desc), _ptr_array(q), _ptr_array(k), _dptr(scores), wp, wb,
                             _stream(stream)))


def kvc_score_weighted(desc, q, k, v, scores: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    """``kvc_score`` with the attention weights multiplied by the tokens' value norms (v-norm variant)."""
    wp, wb = _ws(workspace)
    _check(_load().kvc_score_weighted(C.byref(desc), _ptr_array(q), _ptr_array(k), _ptr_array(v), _dptr(scores),
                                      wp, wb, _stream(stream)))


def kvc_score_uses_tensor_cores(desc: KvcDesc) -> bool:
    """Whether scoring this problem runs on the tensor-core kernel (else on the CUDA-core kernels)."""
    r = int(_load().kvc_score_uses_tensor_cores(C.byref(desc)))
    if r < 0:
        _check(r)
    return r == 1


def kvc_score_status_offset(desc: KvcDesc) -> int:
    """Byte offset, in the workspace given to ``kvc_score``, of that call's int32 device status."""
    out = C.c_size_t(0)
    _check(_load().kvc_score_status_offset(C.byref(desc), C.byref(out)))
    return int(out.value)


def kvc_debug_score_hooks(wait_limit_ns: int = 0, withhold_unit: int = -1) -> None:
    """Test hook: bound of the scoring kernel's device-side waits, and a unit whose statistics
    are withheld so that those waits expire.  The defaults restore normal operation."""
    _load().kvc_debug_score_hooks(int(wait_limit_ns), int(withhold_unit))


def kvc_debug_select_hooks(path: int = 0, max_rounds: int = -1) -> None:
    """Test hook: which way the allocation finds its threshold (0 automatic, 1 histogram passes,
    2 sorted-rows kernel) and the sorted-rows kernel's bound on rounds.  The defaults restore normal operation."""
    _load().kvc_debug_select_hooks(int(path), int(max_rounds))


def kvc_head_sum(desc, scores, head_sum, stream=None) -> None:
    _check(_load().kvc_head_sum(C.byref(desc), _dptr(scores), _dptr(head_sum), _stream(stream)))


def kvc_add_head_mean(desc, scores, head_sum, n_kv_heads_total: int, stream=None) -> None:
    _check(_load().kvc_add_head_mean(C.byref(desc), _dptr(scores), _dptr(head_sum), int(n_kv_heads_total),
                                     _stream(stream)))


def kvc_scale(x: torch.Tensor, factor: float, stream=None) -> None:
    _check(_load().kvc_scale(_dptr(x), x.numel(), float(factor), _stream(stream)))


def kvc_compose(desc, scores, idx, composite, workspace, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_compose(C.byref(desc), _dptr(scores), _dptr(idx), _dptr(composite), wp, wb,
                               _stream(stream)))


def kvc_allocate(desc, composite, budget, n_keep, offsets, workspace, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_allocate(C.byref(desc), _dptr(composite), int(budget), _dptr(n_keep),
                                _dptr(offsets), wp, wb, _stream(stream)))


def kvc_allocate_static(desc, composite, budget, n_keep, offsets, stream=None) -> None:
    """``kvc_allocate`` for callers that cannot allocate a workspace: the scratch is a fixed array
    inside the library (batch <= 64).  Calls that overlap on the GPU share that array and race."""
    _check(_load().kvc_allocate_static(C.byref(desc), _dptr(composite), int(budget), _dptr(n_keep),
                                       _dptr(offsets), _stream(stream)))


def kvc_order_kept(desc, idx, n_keep, workspace, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_order_kept(C.byref(desc), _dptr(idx), _dptr(n_keep), wp, wb, _stream(stream)))


def kvc_select_unstructured(desc, scores, budget_entries, idx, n_keep, offsets, workspace, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_select_unstructured(C.byref(desc), _dptr(scores), int(budget_entries), _dptr(idx),
                                           _dptr(n_keep), _dptr(offsets), wp, wb, _stream(stream)))


def kvc_gather_unstructured(desc, k, v, idx, n_keep, offsets, budget_entries, k_out, v_out, stream=None) -> None:
    _check(_load().kvc_gather_unstructured(C.byref(desc), _ptr_array(k), _ptr_array(v), _dptr(idx), _dptr(n_keep),
                                           _dptr(offsets), int(budget_entries), _dptr(k_out), _dptr(v_out),
                                           _stream(stream)))


def kvc_compress_unstructured(desc, q, k, v, budget_entries, k_out, v_out, n_keep, offsets, idx_out=None,
                              scores_out=None, device_status=None, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_compress_unstructured(C.byref(desc), _ptr_array(q), _ptr_array(k), _ptr_array(v),
                                             int(budget_entries), _dptr(k_out), _dptr(v_out), _dptr(n_keep),
                                             _dptr(offsets), _dptr(idx_out), _dptr(scores_out),
                                             _dptr(device_status), wp, wb, _stream(stream)))


def kvc_gather(desc, k, v, idx, n_keep, offsets, budget, k_out, v_out, stream=None) -> None:
    _check(_load().kvc_gather(C.byref(desc), _ptr_array(k), _ptr_array(v), _dptr(idx), _dptr(n_keep),
                              _dptr(offsets), int(budget), _dptr(k_out), _dptr(v_out), _stream(stream)))


def kvc_compress(desc, q, k, v, budget, k_out, v_out, n_keep, offsets, idx_out=None, scores_out=None,
                 composite_out=None, device_status=None, workspace=None, stream=None) -> None:
    wp, wb = _ws(workspace)
    _check(_load().kvc_compress(C.byref(desc), _ptr_array(q), _ptr_array(k), _ptr_array(v), int(budget),
                                _dptr(k_out), _dptr(v_out), _dptr(n_keep), _dptr(offsets),
                                _dptr(idx_out), _dptr(scores_out), _dptr(composite_out),
                                _dptr(device_status), wp, wb, _stream(stream)))


def kvc_last_error() -> str:
    return _load().kvc_last_error().decode()


def kvc_launch_count(reset: bool = False) -> int:
    return int(_load().kvc_launch_count(1 if reset else 0))


def kvc_version() -> int:
    return int(_load().kvc_version())


# ---- conveniences: descriptor from a workload config, output allocation -------------------------

def desc_from_config(cfg, **overrides) -> KvcDesc:
    """Descriptor with the paper's defaults for a ``workloads.WorkloadConfig``."""
    d = kvc_desc_init(cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_ctx,
                      cfg.window, BF16 if cfg.dtype == "bf16" else F32)
    for key, val in overrides.items():
        setattr(d, key, val)
    return d


@dataclasses.dataclass
class CompressOutputs:
    k_out: torch.Tensor        # [Bt, budget * Hkv * d]
    v_out: torch.Tensor
    n_keep: torch.Tensor       # [Bt, L] int32
    offsets: torch.Tensor      # [Bt, L + 1] int64
    idx: Optional[torch.Tensor]        # [L, Bt, Hkv, N] int32
    scores: Optional[torch.Tensor]     # [L, Bt, Hkv, N] fp32
    composite: Optional[torch.Tensor]  # [L, Bt, N] fp32
    device_status: torch.Tensor
    workspace: torch.Tensor

    def layer(self, b: int, l: int, n_keep_host, offsets_host, Hkv: int, d: int):
        """Views of layer l of sequence b: (K', V') each [Hkv, N_l, d]."""
        lo = int(offsets_host[b][l]) * Hkv * d
        n = int(n_keep_host[b][l])
        return (self.k_out[b, lo:lo + Hkv * n * d].view(Hkv, n, d),
                self.v_out[b, lo:lo + Hkv * n * d].view(Hkv, n, d))


def alloc_outputs(desc: KvcDesc, budget: int, dtype: torch.dtype, device, keep_intermediates=True,
                  workspace: Optional[torch.Tensor] = None) -> CompressOutputs:
    L, Bt, Hkv, N, d = desc.n_layers, desc.batch, desc.n_kv_heads, desc.n_ctx, desc.head_dim
    kw = dict(device=device)
    ws = workspace if workspace is not None else torch.empty(kvc_workspace_size(desc, budget),
                                                             dtype=torch.uint8, **kw)
    return CompressOutputs(
        k_out=torch.empty((Bt, budget * Hkv * d), dtype=dtype, **kw),
        v_out=torch.empty((Bt, budget * Hkv * d), dtype=dtype, **kw),
        n_keep=torch.empty((Bt, L), dtype=torch.int32, **kw),
        offsets=torch.empty((Bt, L + 1), dtype=torch.int64, **kw),
        idx=torch.empty((L, Bt, Hkv, N), dtype=torch.int32, **kw) if keep_intermediates else None,
        scores=torch.empty((L, Bt, Hkv, N), dtype=torch.float32, **kw) if keep_intermediates else None,
        composite=torch.empty((L, Bt, N), dtype=torch.float32, **kw) if keep_intermediates else None,
        device_status=torch.zeros(1, dtype=torch.int32, **kw),
        workspace=ws,
    )


def compress(q: List[torch.Tensor], k: List[torch.Tensor], v: List[torch.Tensor], desc: KvcDesc,
             budget: int, keep_intermediates: bool = True, out: Optional[CompressOutputs] = None,
             stream=None) -> CompressOutputs:
    """Allocate outputs (unless given) and run ``kvc_compress`` on the current stream."""
    if out is None:
        out = alloc_outputs(desc, budget, k[0].dtype, k[0].device, keep_intermediates)
    kvc_compress(desc, q, k, v, budget, out.k_out, out.v_out, out.n_keep, out.offsets, out.idx,
                 out.scores, out.composite, out.device_status, out.workspace, stream)
    return out
