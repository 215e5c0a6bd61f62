"""numpy-facing wrappers around ``kvc_oracle.c`` (TEST INFRASTRUCTURE ONLY).

The C file is compiled with gcc on first use (``build()``); the wrappers only
marshal numpy arrays -- every number is produced by the C code.  Only the
test-suite, the smoke check and the benchmark's cpu-baseline leg may use this.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

AGG_MAX = 0
AGG_MEAN = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvc_oracle.c")
_LIB = os.path.join(_HERE, "libkvc_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP for the timed leg). Returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp",
                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True, capture_output=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = C.CDLL(_LIB)
    i32, i64, f64 = C.c_int32, C.c_int64, C.c_double
    p = C.c_void_p
    lib.oracle_set_threads.argtypes = [C.c_int]
    lib.oracle_get_threads.restype = C.c_int
    lib.oracle_has_openmp.restype = C.c_int
    lib.oracle_attention_rows.argtypes = [p, p, i64, i32, i32, f64, i64, p]
    lib.oracle_attention_rows.restype = None
    lib.oracle_score_layer.argtypes = [p, p, i32, i32, i64, i32, i32, f64, i64, i32, i32, i32, p, p]
    lib.oracle_score_layer.restype = C.c_int
    lib.oracle_score_layer_vnorm.argtypes = [p, p, p, i32, i32, i64, i32, i32, f64, i64, i32, i32, i32, p, p]
    lib.oracle_score_layer_vnorm.restype = C.c_int
    lib.oracle_allocate_floor.argtypes = [p, i32, i64, i64, i64, p, p]
    lib.oracle_allocate_floor.restype = C.c_int
    lib.oracle_select_unstructured.argtypes = [p, i32, i32, i64, i64, p, p]
    lib.oracle_select_unstructured.restype = C.c_int
    lib.oracle_sort_kept.argtypes = [p, i32, i64, p, p]
    lib.oracle_sort_kept.restype = None
    lib.oracle_rank.argtypes = [p, i64, p, p]
    lib.oracle_rank.restype = C.c_int
    lib.oracle_compose.argtypes = [p, i32, i64, i32, p]
    lib.oracle_compose.restype = None
    lib.oracle_compose_f32.argtypes = [p, i32, i64, i32, p]
    lib.oracle_compose_f32.restype = None
    lib.oracle_budget_from_ratio.argtypes = [i32, i64, f64]
    lib.oracle_budget_from_ratio.restype = i64
    lib.oracle_allocate.argtypes = [p, i32, i64, i64, p, p]
    lib.oracle_allocate.restype = C.c_int
    lib.oracle_gather_layer.argtypes = [p, p, i32, i64, i64, i32, p]
    lib.oracle_gather_layer.restype = None
    lib.oracle_compress.argtypes = [p, p, p, p, i32, i32, i32, i64, i32, i32, i64, f64, i64,
                                    i32, i32, i32, i32, p, i64, p, p, p, p, p, p, p]
    lib.oracle_compress.restype = C.c_int
    _lib = lib
    return lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _map(q_to_kv, Hq):
    if q_to_kv is None:
        return None
    m = np.ascontiguousarray(q_to_kv, dtype=np.int32)
    assert m.shape == (Hq,)
    return m


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_load().oracle_get_threads())


def has_openmp() -> bool:
    return bool(_load().oracle_has_openmp())


def attention_rows(q, k, scale, q_pos0):
    """q [w, d], k [N, d] -> A [w, N] float64 (Eq. 3 with the causal window mask)."""
    q, k = _f32(q), _f32(k)
    w, d = q.shape
    N = k.shape[0]
    assert k.shape[1] == d
    A = np.empty((w, N), dtype=np.float64)
    _load().oracle_attention_rows(_ptr(q), _ptr(k), N, d, w, float(scale), int(q_pos0), _ptr(A))
    return A


def score_layer(q, k, scale, q_pos0, agg_task=AGG_MAX, agg_group=AGG_MEAN, augment=True,
                q_to_kv=None):
    """q [Hq, w, d], k [Hkv, N, d] -> S [Hkv, N] float64 (Eqs. 14-16)."""
    q, k = _f32(q), _f32(k)
    Hq, w, d = q.shape
    Hkv, N, d2 = k.shape
    assert d == d2
    m = _map(q_to_kv, Hq)
    S = np.empty((Hkv, N), dtype=np.float64)
    rc = _load().oracle_score_layer(_ptr(q), _ptr(k), Hq, Hkv, N, d, w, float(scale), int(q_pos0),
                                    int(agg_task), int(agg_group), int(bool(augment)), _ptr(m),
                                    _ptr(S))
    if rc:
        raise RuntimeError("oracle_score_layer failed (%d)" % rc)
    return S


def score_layer_vnorm(q, k, v, scale, q_pos0, agg_task=AGG_MAX, agg_group=AGG_MEAN, augment=True,
                      q_to_kv=None):
    """The v-norm variant (App. A.1.3): q [Hq, w, d], k, v [Hkv, N, d] -> S [Hkv, N] float64."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    Hq, w, d = q.shape
    Hkv, N, d2 = k.shape
    assert d == d2 and v.shape == k.shape
    m = _map(q_to_kv, Hq)
    S = np.empty((Hkv, N), dtype=np.float64)
    rc = _load().oracle_score_layer_vnorm(_ptr(q), _ptr(k), _ptr(v), Hq, Hkv, N, d, w, float(scale),
                                          int(q_pos0), int(agg_task), int(agg_group),
                                          int(bool(augment)), _ptr(m), _ptr(S))
    if rc:
        raise RuntimeError("oracle_score_layer_vnorm failed (%d)" % rc)
    return S


def rank(S):
    """S [N] -> (idx [N] int32, S_sorted [N] float64): Eqs. 17-18, ties to the smaller position."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    (N,) = S.shape
    idx = np.empty(N, dtype=np.int32)
    Ss = np.empty(N, dtype=np.float64)
    if _load().oracle_rank(_ptr(S), N, _ptr(idx), _ptr(Ss)):
        raise RuntimeError("oracle_rank failed")
    return idx, Ss


def compose(S_sorted, agg_head=AGG_MEAN):
    """S_sorted [Hkv, N] -> I [N] float64 (Eq. 19)."""
    S_sorted = np.ascontiguousarray(S_sorted, dtype=np.float64)
    Hkv, N = S_sorted.shape
    I = np.empty(N, dtype=np.float64)
    _load().oracle_compose(_ptr(S_sorted), Hkv, N, int(agg_head), _ptr(I))
    return I


def compose_f32(S_sorted, agg_head=AGG_MEAN):
    """Eq. 19 in single precision, heads added left to right, one division at the end."""
    S_sorted = np.ascontiguousarray(S_sorted, dtype=np.float32)
    Hkv, N = S_sorted.shape
    I = np.empty(N, dtype=np.float32)
    _load().oracle_compose_f32(_ptr(S_sorted), Hkv, N, int(agg_head), _ptr(I))
    return I


def budget_from_ratio(L, N, r_target):
    return int(_load().oracle_budget_from_ratio(int(L), int(N), float(r_target)))


def allocate(I, B):
    """I [L, N] -> (n_keep [L] int32, offsets [L+1] int64): global top-B of the pooled scores."""
    I = np.ascontiguousarray(I, dtype=np.float64)
    L, N = I.shape
    n_keep = np.empty(L, dtype=np.int32)
    offsets = np.empty(L + 1, dtype=np.int64)
    rc = _load().oracle_allocate(_ptr(I), L, N, int(B), _ptr(n_keep), _ptr(offsets))
    if rc:
        raise ValueError("oracle_allocate failed (%d)" % rc)
    return n_keep, offsets


def allocate_floor(I, B, min_keep):
    """Eqs. 20-22 with a per-layer minimum: I [L, N] -> (n_keep [L], offsets [L+1])."""
    I = np.ascontiguousarray(I, dtype=np.float64)
    L, N = I.shape
    n_keep = np.empty(L, dtype=np.int32)
    offsets = np.empty(L + 1, dtype=np.int64)
    rc = _load().oracle_allocate_floor(_ptr(I), L, N, int(B), int(min_keep), _ptr(n_keep), _ptr(offsets))
    if rc:
        raise ValueError("oracle_allocate_floor failed (%d)" % rc)
    return n_keep, offsets


def select_unstructured(S, B):
    """App. A.2: S [L, Hkv, N] -> (n_keep [L, Hkv] int32, offsets [L*Hkv+1] int64): the B best
    entries of the pool over (layer, head, position)."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    L, Hkv, N = S.shape
    n_keep = np.empty(L * Hkv, dtype=np.int32)
    offsets = np.empty(L * Hkv + 1, dtype=np.int64)
    rc = _load().oracle_select_unstructured(_ptr(S), L, Hkv, N, int(B), _ptr(n_keep), _ptr(offsets))
    if rc:
        raise ValueError("oracle_select_unstructured failed (%d)" % rc)
    return n_keep.reshape(L, Hkv), offsets


def sort_kept(idx, n_keep):
    """idx [Hkv, N], n_keep [Hkv] -> idx with every head's first n_keep[h] positions ascending."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    Hkv, N = idx.shape
    nk = np.ascontiguousarray(np.broadcast_to(np.asarray(n_keep, dtype=np.int32), (Hkv,)))
    out = np.empty_like(idx)
    _load().oracle_sort_kept(_ptr(idx), Hkv, N, _ptr(nk), _ptr(out))
    return out


def gather_layer(src, idx, n_keep):
    """src [Hkv, N, ...] any dtype, idx [Hkv, N] -> dst [Hkv, n_keep, ...] (bytes copied)."""
    src = np.ascontiguousarray(src)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    Hkv, N = idx.shape
    assert src.shape[0] == Hkv and src.shape[1] == N
    row_bytes = src[0, 0].nbytes if src.ndim > 2 else src.itemsize
    dst = np.empty((Hkv, int(n_keep)) + src.shape[2:], dtype=src.dtype)
    _load().oracle_gather_layer(_ptr(src), _ptr(idx), Hkv, N, row_bytes, int(n_keep), _ptr(dst))
    return dst


def compress(q, k, k_raw, v_raw, scale, q_pos0, B, agg_task=AGG_MAX, agg_group=AGG_MEAN,
             agg_head=AGG_MEAN, augment=True, q_to_kv=None, want_scores=True):
    """Whole pass for one sequence.

    q [L, Hq, w, d], k [L, Hkv, N, d] as float32 (exact widenings of the cache dtype);
    k_raw / v_raw [L, Hkv, N, row] in the cache's own dtype viewed as uint8/uint16/float32
    (or None to skip the gather).  Returns a dict.
    """
    q, k = _f32(q), _f32(k)
    L, Hq, w, d = q.shape
    _, Hkv, N, _ = k.shape
    m = _map(q_to_kv, Hq)
    S = np.empty((L, Hkv, N), dtype=np.float64) if want_scores else None
    I = np.empty((L, N), dtype=np.float64)
    idx = np.empty((L, Hkv, N), dtype=np.int32)
    n_keep = np.empty(L, dtype=np.int32)
    offsets = np.empty(L + 1, dtype=np.int64)
    k_out = v_out = None
    row_bytes = 0
    if k_raw is not None:
        k_raw = np.ascontiguousarray(k_raw)
        v_raw = np.ascontiguousarray(v_raw)
        row_bytes = k_raw[0, 0, 0].nbytes
        k_out = np.empty((int(B) * Hkv,) + k_raw.shape[3:], dtype=k_raw.dtype)
        v_out = np.empty_like(k_out)
    rc = _load().oracle_compress(_ptr(q), _ptr(k), _ptr(k_raw), _ptr(v_raw), L, Hq, Hkv, N, d, w,
                                 row_bytes, float(scale), int(q_pos0), int(agg_task),
                                 int(agg_group), int(agg_head), int(bool(augment)), _ptr(m),
                                 int(B), _ptr(S), _ptr(idx), _ptr(I), _ptr(n_keep),
                                 _ptr(offsets), _ptr(k_out), _ptr(v_out))
    if rc:
        raise RuntimeError("oracle_compress failed (%d)" % rc)
    return dict(scores=S, idx=idx, composite=I, n_keep=n_keep, offsets=offsets, k_out=k_out,
                v_out=v_out)
