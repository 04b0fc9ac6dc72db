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
