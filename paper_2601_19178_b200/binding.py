"""Thin ctypes binding of libckv.so: same names as the C ABI, argument marshalling only.

Every step of the decode path runs inside the CUDA library; there is no fallback.  If the
shared library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# CKV_LIBRARY names another build of the same library (the range-checked libckv_bounds.so of build.py --bounds)
LIB_PATH = os.environ.get("CKV_LIBRARY") or os.path.join(_HERE, "libckv.so")

CKV_F32, CKV_BF16 = 0, 1
CKV_SOFTMAX, CKV_SILU_OVER_L = 0, 1
(CKV_OK, CKV_ERR_INVALID_ARG, CKV_ERR_SHAPE, CKV_ERR_STATE, CKV_ERR_INDEX_RANGE,
 CKV_ERR_UNKNOWN_USER, CKV_ERR_OOM, CKV_ERR_CUDA, CKV_ERR_UNSUPPORTED, CKV_ERR_TOO_LARGE) = range(10)

# every symbol include/ckv.h declares
EXPORTS = (
    "ckv_create", "ckv_destroy", "ckv_pool_load", "ckv_cache_put", "ckv_cache_put_batch",
    "ckv_cache_evict", "ckv_cache_clear", "ckv_attend", "ckv_attend_static", "ckv_materialize",
    "ckv_user_length", "ckv_cache_append", "ckv_cache_blob_bytes", "ckv_cache_export", "ckv_cache_import",
    "ckv_cache_bytes", "ckv_set_option", "ckv_get_option", "ckv_last_stat", "ckv_strerror",
    "ckv_last_cuda_error", "ckv_version", "ckv_route", "ckv_project", "ckv_pool_load_sides", "ckv_attend_visible",
)


class ckv_config(ctypes.Structure):
    _fields_ = [("n_groups", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("mode", ctypes.c_int32), ("scale", ctypes.c_float), ("device", ctypes.c_int32)]


class CkvError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        msg = f"{where}: {lib.ckv_strerror(status).decode()} (status {status})"
        super().__init__(msg + (f" [{detail}]" if detail else ""))


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python paper_2601_19178_b200/build.py` "
            "(there is no fallback implementation)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    p64, cs = ctypes.POINTER(ctypes.c_int64), ctypes.c_char_p
    sig = {
        "ckv_create": (i32, [ctypes.POINTER(ckv_config), ctypes.POINTER(vp)]),
        "ckv_destroy": (i32, [vp]),
        "ckv_pool_load": (i32, [vp, vp, vp, i32, i32, vp]),
        "ckv_pool_load_sides": (i32, [vp, vp, vp, i32, i32, i32, vp]),
        "ckv_attend_visible": (i32, [vp, i32, vp, vp, vp, vp, vp, vp]),
        "ckv_cache_put": (i32, [vp, i64, i32, vp, vp, vp, vp, i32, vp]),
        "ckv_cache_put_batch": (i32, [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp]),
        "ckv_cache_append": (i32, [vp, i64, i32, vp, vp, vp, vp, i32, vp]),
        "ckv_cache_evict": (i32, [vp, i64]),
        "ckv_cache_clear": (i32, [vp]),
        "ckv_attend": (i32, [vp, i32, vp, vp, vp, vp, vp]),
        "ckv_attend_static": (i32, [vp, i32, vp, vp, vp, vp, vp]),
        "ckv_materialize": (i32, [vp, i64, vp, vp, vp]),
        "ckv_user_length": (i32, [vp, i64, p64]),
        "ckv_cache_blob_bytes": (i32, [vp, i32, vp, p64]),
        "ckv_cache_export": (i32, [vp, i32, vp, vp, i64, vp]),
        "ckv_cache_import": (i32, [vp, i32, vp, vp, vp, i64, vp]),
        "ckv_cache_bytes": (i32, [vp, p64, p64]),
        "ckv_set_option": (i32, [vp, cs, i64]),
        "ckv_get_option": (i32, [vp, cs, p64]),
        "ckv_last_stat": (i32, [vp, cs, p64]),
        "ckv_strerror": (cs, [i32]),
        "ckv_last_cuda_error": (cs, [vp]),
        "ckv_version": (i32, []),
        "ckv_route": (i32, [i32, i32, i32, i32, i32, vp, vp, vp, vp, i32, vp]),
        "ckv_project": (i32, [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        f = getattr(L, name)
        f.restype, f.argtypes = res, args
    return L


lib = _load()


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / raw int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("numpy argument must be C-contiguous")
        return x.ctypes.data
    if hasattr(x, "data_ptr"):
        if not x.is_contiguous():
            raise ValueError("tensor argument must be contiguous")
        return x.data_ptr()
    raise TypeError(f"cannot take the address of {type(x)}")


def _host_i64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int64)


def _host_i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _check(ctx, status: int, where: str):
    if status != CKV_OK:
        detail = lib.ckv_last_cuda_error(ctx).decode() if status in (CKV_ERR_CUDA, CKV_ERR_OOM) and ctx else ""
        raise CkvError(status, where, detail)


# ---- functions named like the C ABI -------------------------------------------------
def ckv_create(n_groups: int, head_dim: int, dtype: int, mode: int, scale: float = 0.0,
               out_dtype: Optional[int] = None, device: int = 0) -> int:
    cfg = ckv_config(n_groups, head_dim, dtype, dtype if out_dtype is None else out_dtype, mode,
                     float(scale), device)
    h = ctypes.c_void_p()
    _check(None, lib.ckv_create(ctypes.byref(cfg), ctypes.byref(h)), "ckv_create")
    return h.value


def ckv_destroy(ctx) -> None:
    lib.ckv_destroy(ctx)


def ckv_pool_load(ctx, pool_K, pool_V, n_entries: int, d_shared: int, stream=None) -> None:
    _check(ctx, lib.ckv_pool_load(ctx, _ptr(pool_K), _ptr(pool_V), n_entries, d_shared, _stream(stream)),
           "ckv_pool_load")


def ckv_pool_load_sides(ctx, pool_K, pool_V, n_entries: int, d_shared_k: int, d_shared_v: int, stream=None) -> None:
    """ckv_pool_load with a shared width per side; 0 = that side is not shared (its pool may be None)."""
    _check(ctx, lib.ckv_pool_load_sides(ctx, _ptr(pool_K), _ptr(pool_V), n_entries, d_shared_k, d_shared_v,
                                        _stream(stream)), "ckv_pool_load_sides")


def ckv_cache_put(ctx, user: int, L: int, idx_K, idx_V, user_K, user_V, d_user: int, stream=None) -> None:
    _check(ctx, lib.ckv_cache_put(ctx, int(user), int(L), _ptr(idx_K), _ptr(idx_V), _ptr(user_K),
                                  _ptr(user_V), d_user, _stream(stream)), "ckv_cache_put")


def ckv_cache_put_batch(ctx, users, hist_off, idx_K, idx_V, user_K, user_V, d_user: int, stream=None) -> None:
    users, hist_off = _host_i64(users), _host_i64(hist_off)
    if hist_off.shape[0] != users.shape[0] + 1:
        raise ValueError("hist_off must have len(users) + 1 entries")
    _check(ctx, lib.ckv_cache_put_batch(ctx, users.shape[0], users.ctypes.data, hist_off.ctypes.data,
                                        _ptr(idx_K), _ptr(idx_V), _ptr(user_K), _ptr(user_V), d_user,
                                        _stream(stream)), "ckv_cache_put_batch")


def ckv_cache_append(ctx, user: int, L_new: int, idx_K, idx_V, user_K, user_V, d_user: int, stream=None) -> None:
    _check(ctx, lib.ckv_cache_append(ctx, int(user), int(L_new), _ptr(idx_K), _ptr(idx_V), _ptr(user_K),
                                     _ptr(user_V), d_user, _stream(stream)), "ckv_cache_append")


def ckv_cache_evict(ctx, user: int) -> None:
    _check(ctx, lib.ckv_cache_evict(ctx, int(user)), "ckv_cache_evict")


def ckv_cache_clear(ctx) -> None:
    _check(ctx, lib.ckv_cache_clear(ctx), "ckv_cache_clear")


def ckv_attend(ctx, users, q_off, queries, out, stream=None) -> None:
    """users: host int64 [n]; q_off: host int32 [n+1]; queries/out: device (or host) buffers."""
    users, q_off = _host_i64(users), _host_i32(q_off)
    if q_off.shape[0] != users.shape[0] + 1:
        raise ValueError("q_off must have len(users) + 1 entries")
    _check(ctx, lib.ckv_attend(ctx, users.shape[0], users.ctypes.data, q_off.ctypes.data, _ptr(queries),
                               _ptr(out), _stream(stream)), "ckv_attend")


def ckv_attend_visible(ctx, users, q_off, vis, queries, out, stream=None) -> None:
    """ckv_attend with a visible length per query row: vis int32 [q_off[n]] (host array or device tensor)."""
    users, q_off = _host_i64(users), _host_i32(q_off)
    if q_off.shape[0] != users.shape[0] + 1:
        raise ValueError("q_off must have len(users) + 1 entries")
    if isinstance(vis, np.ndarray):
        vis = _host_i32(vis)
    _check(ctx, lib.ckv_attend_visible(ctx, users.shape[0], users.ctypes.data, q_off.ctypes.data, _ptr(vis),
                                       _ptr(queries), _ptr(out), _stream(stream)), "ckv_attend_visible")


def ckv_attend_static(ctx, users, q_off, queries, out, stream=None) -> None:
    """ckv_attend for callers that must not allocate device memory (a latency-critical
    serving section, a process whose memory belongs to another allocator): same result, but
    the work tables and split-reduction partials live in a fixed 8 MiB array inside the
    library.  queries/out must be device buffers; raises CkvError(CKV_ERR_TOO_LARGE) beyond
    256 users per call or when the partial results do not fit.  Calls that may overlap on the
    GPU race on that array."""
    users, q_off = _host_i64(users), _host_i32(q_off)
    if q_off.shape[0] != users.shape[0] + 1:
        raise ValueError("q_off must have len(users) + 1 entries")
    _check(ctx, lib.ckv_attend_static(ctx, users.shape[0], users.ctypes.data, q_off.ctypes.data,
                                      _ptr(queries), _ptr(out), _stream(stream)), "ckv_attend_static")


def ckv_materialize(ctx, user: int, K_out, V_out, stream=None) -> None:
    _check(ctx, lib.ckv_materialize(ctx, int(user), _ptr(K_out), _ptr(V_out), _stream(stream)),
           "ckv_materialize")


def ckv_user_length(ctx, user: int) -> int:
    v = ctypes.c_int64()
    _check(ctx, lib.ckv_user_length(ctx, int(user), ctypes.byref(v)), "ckv_user_length")
    return v.value


def ckv_cache_blob_bytes(ctx, L) -> int:
    L = _host_i32(L)
    v = ctypes.c_int64()
    _check(ctx, lib.ckv_cache_blob_bytes(ctx, L.shape[0], L.ctypes.data, ctypes.byref(v)), "ckv_cache_blob_bytes")
    return v.value


def ckv_cache_export(ctx, users, blob, nbytes: int, stream=None) -> None:
    """Writes the packed caches of `users` (host int64 [n]) to `blob` (host or device buffer of nbytes)."""
    users = _host_i64(users)
    _check(ctx, lib.ckv_cache_export(ctx, users.shape[0], users.ctypes.data, _ptr(blob), int(nbytes),
                                     _stream(stream)), "ckv_cache_export")


def ckv_cache_import(ctx, users, L, blob, nbytes: int, stream=None) -> None:
    """Stores `users` (host int64 [n]) with history lengths L (host int32 [n]) from a packed blob."""
    users, L = _host_i64(users), _host_i32(L)
    if L.shape[0] != users.shape[0]:
        raise ValueError("L must have len(users) entries")
    _check(ctx, lib.ckv_cache_import(ctx, users.shape[0], users.ctypes.data, L.ctypes.data, _ptr(blob), int(nbytes),
                                     _stream(stream)), "ckv_cache_import")


def ckv_cache_bytes(ctx):
    a, b = ctypes.c_int64(), ctypes.c_int64()
    _check(ctx, lib.ckv_cache_bytes(ctx, ctypes.byref(a), ctypes.byref(b)), "ckv_cache_bytes")
    return a.value, b.value


def ckv_set_option(ctx, name: str, value: int) -> None:
    _check(ctx, lib.ckv_set_option(ctx, name.encode(), int(value)), "ckv_set_option")


def ckv_get_option(ctx, name: str) -> int:
    v = ctypes.c_int64()
    _check(ctx, lib.ckv_get_option(ctx, name.encode(), ctypes.byref(v)), "ckv_get_option")
    return v.value


def ckv_last_stat(ctx, name: str) -> int:
    v = ctypes.c_int64()
    _check(ctx, lib.ckv_last_stat(ctx, name.encode(), ctypes.byref(v)), "ckv_last_stat")
    return v.value


def ckv_version() -> int:
    return int(lib.ckv_version())


def ckv_route(device: int, n: int, n_groups: int, d_in: int, n_entries: int, x, W, bias, idx_out, variant: int = 0,
              stream=None) -> None:
    """Router indices of n positions: x [n][d_in], W [G][n_entries][d_in] (bf16, device), bias [G][n_entries] fp32
    or None, idx_out [n][G] int32 (device); variant 0 / 2 = tcgen05 kernel, 1 = warp-level tensor-core kernel."""
    _check(None, lib.ckv_route(device, n, n_groups, d_in, n_entries, _ptr(x), _ptr(W), _ptr(bias), _ptr(idx_out),
                               int(variant), _stream(stream)), "ckv_route")


def ckv_project(device: int, n: int, n_groups: int, d_in: int, d_out: int, x, W, bias, out, stream=None) -> None:
    """User-specific low-dimensional projection: x [n][d_in], W [G][d_out][d_in] (bf16, device), bias [G][d_out]
    fp32 or None, out [n][G][d_out] bf16 (device)."""
    _check(None, lib.ckv_project(device, n, n_groups, d_in, d_out, _ptr(x), _ptr(W), _ptr(bias), _ptr(out),
                                 _stream(stream)), "ckv_project")
