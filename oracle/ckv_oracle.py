"""ctypes front end of the C oracle (oracle/ckv_oracle.c).

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the bench's
CPU-baseline leg may import this module; the CUDA library never does.

`build()` compiles the C file with gcc (-O2, OpenMP over users) into
oracle/_ckv_oracle.so; `attend`, `materialize` and `compression_rate` call it.
Array conventions are those of `synth.workloads`.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ckv_oracle.c")
_LIB = os.path.join(_HERE, "_ckv_oracle.so")
_lib = None

_DTYPE = {"f32": 0, "bf16": 1}
_MODE = {"softmax": 0, "silu_over_l": 1}


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                        "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, i64, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double
        lib.ckv_oracle_attend.restype = i32
        lib.ckv_oracle_attend.argtypes = [i32, i32, f64, i32, i32, i32, i32, vp, vp, i64, vp,
                                          vp, vp, vp, vp, vp, vp, i64, vp, vp, i32]
        lib.ckv_oracle_materialize.restype = i32
        lib.ckv_oracle_materialize.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp,
                                               i64, i64, vp, vp]
        lib.ckv_oracle_attend_variants.restype = i32
        lib.ckv_oracle_attend_variants.argtypes = [i32, i32, f64, i32, i32, i32, i32, i32, vp, vp, i64, vp,
                                                   vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, i32]
        lib.ckv_oracle_materialize_side.restype = i32
        lib.ckv_oracle_materialize_side.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, i64, i64, vp]
        lib.ckv_oracle_compression_rate.restype = f64
        lib.ckv_oracle_compression_rate.argtypes = [i32, i32]
        lib.ckv_oracle_max_threads.restype = i32
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(a: np.ndarray, dtype: str, name: str) -> np.ndarray:
    want = np.float32 if dtype == "f32" else np.uint16
    if a.dtype != want:
        raise TypeError(f"{name}: expected {want.__name__} for dtype {dtype}, got {a.dtype}")
    return np.ascontiguousarray(a)


def max_threads() -> int:
    return int(_load().ckv_oracle_max_threads())


def compression_rate(d_a: int, d_u: int) -> float:
    return float(_load().ckv_oracle_compression_rate(int(d_a), int(d_u)))


def attend(dtype: str, mode: str, scale: float, pool_K, pool_V, hist_off, idx_K, idx_V,
           user_K, user_V, q_off, queries, sel: Optional[Sequence[int]] = None,
           n_threads: int = 0) -> np.ndarray:
    """Outputs, float64 [sum of selected users' M, G, d] (all users when sel is None)."""
    lib = _load()
    pool_K, pool_V = _check(pool_K, dtype, "pool_K"), _check(pool_V, dtype, "pool_V")
    user_K, user_V = _check(user_K, dtype, "user_K"), _check(user_V, dtype, "user_V")
    queries = _check(queries, dtype, "queries")
    G, m, d_g = pool_K.shape
    d_u = user_K.shape[-1]
    d = d_g + d_u
    assert pool_V.shape == pool_K.shape and queries.shape[1:] == (G, d)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    q_off64 = np.ascontiguousarray(q_off, dtype=np.int64)
    idx_K = np.ascontiguousarray(idx_K, dtype=np.int32)
    idx_V = np.ascontiguousarray(idx_V, dtype=np.int32)
    U = hist_off.shape[0] - 1
    assert idx_K.shape == (hist_off[-1], G) and user_K.shape == (hist_off[-1], G, d_u)
    if sel is None:
        sel_arr, n_sel, rows = None, U, int(q_off64[-1])
    else:
        sel_arr = np.ascontiguousarray(sel, dtype=np.int64)
        n_sel = sel_arr.shape[0]
        rows = int((q_off64[sel_arr + 1] - q_off64[sel_arr]).sum())
    out = np.empty((rows, G, d), dtype=np.float64)
    rc = lib.ckv_oracle_attend(_DTYPE[dtype], _MODE[mode], float(scale), G, m, d_g, d_u,
                               _p(pool_K), _p(pool_V), U, _p(hist_off), _p(idx_K), _p(idx_V),
                               _p(user_K), _p(user_V), _p(q_off64), _p(queries),
                               n_sel, _p(sel_arr), _p(out), int(n_threads))
    if rc == 1:
        raise IndexError("pool index out of range")
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return out


def materialize(dtype: str, pool_K, pool_V, idx_K, idx_V, user_K, user_V, pos0: int, L: int):
    """Full-width (K, V) of one user in the input dtype: [L, G, d] each."""
    lib = _load()
    pool_K, pool_V = _check(pool_K, dtype, "pool_K"), _check(pool_V, dtype, "pool_V")
    user_K, user_V = _check(user_K, dtype, "user_K"), _check(user_V, dtype, "user_V")
    idx_K = np.ascontiguousarray(idx_K, dtype=np.int32)
    idx_V = np.ascontiguousarray(idx_V, dtype=np.int32)
    G, m, d_g = pool_K.shape
    d_u = user_K.shape[-1]
    K = np.empty((L, G, d_g + d_u), dtype=pool_K.dtype)
    V = np.empty_like(K)
    rc = lib.ckv_oracle_materialize(_DTYPE[dtype], G, m, d_g, d_u, _p(pool_K), _p(pool_V),
                                    _p(idx_K), _p(idx_V), _p(user_K), _p(user_V),
                                    int(pos0), int(L), _p(K), _p(V))
    if rc != 0:
        raise IndexError("pool index out of range")
    return K, V


def attend_variants(dtype: str, mode: str, scale: float, d_a: int, pool_K, pool_V, hist_off, idx_K, idx_V,
                    user_K, user_V, q_off, queries, vis=None, sel: Optional[Sequence[int]] = None,
                    n_threads: int = 0) -> np.ndarray:
    """The decode path with a shared width per side and a visible length per query.

    pool_K / pool_V: [G, m, d_g] or None for a side that is not shared (its cached part user_K / user_V is then
    the full [P, G, d_a] row and its indices are ignored).  vis: int32 [Q] (query row r attends positions
    0 .. vis[r]-1 of its user) or None (all positions).  Returns float64 [rows of the selected users, G, d_a]."""
    lib = _load()
    user_K, user_V = _check(user_K, dtype, "user_K"), _check(user_V, dtype, "user_V")
    queries = _check(queries, dtype, "queries")
    G = queries.shape[1]
    assert queries.shape[2] == d_a
    dims, pools, m = [], [], None
    for pool, user, name in ((pool_K, user_K, "K"), (pool_V, user_V, "V")):
        if pool is None:
            dims.append(0)
            pools.append(None)
            assert user.shape[-1] == d_a, f"{name} is not shared: its cached part must be d_a wide"
        else:
            pool = _check(pool, dtype, "pool_" + name)
            assert pool.shape[0] == G and pool.shape[2] + user.shape[-1] == d_a
            assert m is None or m == pool.shape[1]
            m = pool.shape[1]
            dims.append(pool.shape[2])
            pools.append(pool)
    hist_off = np.ascontiguousarray(hist_off, dtype=np.int64)
    q_off64 = np.ascontiguousarray(q_off, dtype=np.int64)
    idx_K = None if pools[0] is None else np.ascontiguousarray(idx_K, dtype=np.int32)
    idx_V = None if pools[1] is None else np.ascontiguousarray(idx_V, dtype=np.int32)
    vis_arr = None if vis is None else np.ascontiguousarray(vis, dtype=np.int32)
    assert vis_arr is None or vis_arr.shape == (int(q_off64[-1]),)
    U = hist_off.shape[0] - 1
    if sel is None:
        sel_arr, n_sel, rows = None, U, int(q_off64[-1])
    else:
        sel_arr = np.ascontiguousarray(sel, dtype=np.int64)
        n_sel = sel_arr.shape[0]
        rows = int((q_off64[sel_arr + 1] - q_off64[sel_arr]).sum())
    out = np.empty((rows, G, d_a), dtype=np.float64)
    rc = lib.ckv_oracle_attend_variants(_DTYPE[dtype], _MODE[mode], float(scale), G, int(m or 1), int(d_a),
                                        dims[0], dims[1], _p(pools[0]), _p(pools[1]), U, _p(hist_off),
                                        _p(idx_K), _p(idx_V), _p(user_K), _p(user_V), _p(q_off64), _p(queries),
                                        _p(vis_arr), n_sel, _p(sel_arr), _p(out), int(n_threads))
    if rc == 1:
        raise IndexError("pool index out of range")
    if rc == 3:
        raise ValueError("a visible length is outside [0, L_u]")
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return out


def materialize_side(dtype: str, d_a: int, pool, idx, cached, pos0: int, L: int) -> np.ndarray:
    """Full-width rows [L, G, d_a] of one side (K or V) of one user in the input dtype; pool None = the side is
    not shared and `cached` already holds the full rows."""
    lib = _load()
    cached = _check(cached, dtype, "cached")
    G = cached.shape[1]
    if pool is None:
        d_g, m, idx_arr = 0, 1, None
    else:
        pool = _check(pool, dtype, "pool")
        d_g, m = pool.shape[2], pool.shape[1]
        idx_arr = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.empty((L, G, d_a), dtype=cached.dtype)
    rc = lib.ckv_oracle_materialize_side(_DTYPE[dtype], G, m, int(d_a), d_g, _p(pool), _p(idx_arr), _p(cached),
                                         int(pos0), int(L), _p(out))
    if rc != 0:
        raise IndexError("pool index out of range")
    return out
