"""Second, independent formulation of the oracle in numpy (float64).

TEST INFRASTRUCTURE ONLY.  Where oracle/ckv_oracle.c rebuilds rows and attends
in one pass, this file first materialises the user's full-width K and V with
array indexing (Eq. (Kc), Eq. (K): user part first), then applies the textbook
attention definition with matrix products.  The two are compared on small
inputs by the CPU tests; this one is too slow and memory-hungry for big ones.
"""
from __future__ import annotations

import numpy as np


def _f64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:  # bfloat16 bit patterns, widened exactly
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def materialize_f64(pool, idx, user, p0: int, L: int) -> np.ndarray:
    """[L, G, d_u + d_g] float64: concat(user[i, g], pool[g][idx[i, g]])."""
    G = pool.shape[0]
    rows = idx[p0:p0 + L]                                    # [L, G]
    coll = _f64(pool)[np.arange(G)[None, :], rows]           # [L, G, d_g]  Eq. (Kc)
    return np.concatenate([_f64(user[p0:p0 + L]), coll], axis=-1)  # Eq. (K)


def attend(mode: str, scale: float, pool_K, pool_V, hist_off, idx_K, idx_V, user_K, user_V,
           q_off, queries) -> np.ndarray:
    G = pool_K.shape[0]
    d = pool_K.shape[2] + user_K.shape[2]
    U = len(hist_off) - 1
    out = np.zeros((int(q_off[-1]), G, d), dtype=np.float64)
    qf = _f64(queries)
    for u in range(U):
        p0, L = int(hist_off[u]), int(hist_off[u + 1] - hist_off[u])
        q0, q1 = int(q_off[u]), int(q_off[u + 1])
        if L == 0 or q1 == q0:
            continue
        K = materialize_f64(pool_K, idx_K, user_K, p0, L)
        V = materialize_f64(pool_V, idx_V, user_V, p0, L)
        for g in range(G):
            S = scale * (qf[q0:q1, g] @ K[:, g].T)           # [M, L]
            if mode == "softmax":
                E = np.exp(S - S.max(axis=1, keepdims=True))
                W = E / E.sum(axis=1, keepdims=True)
            else:
                W = S / (1.0 + np.exp(-S)) / L
            out[q0:q1, g] = W @ V[:, g]
    return out


def attend_variants(mode: str, scale: float, d_a: int, pool_K, pool_V, hist_off, idx_K, idx_V, user_K, user_V,
                    q_off, queries, vis=None) -> np.ndarray:
    """The same second formulation for the variants: a side whose pool is None is taken as cached full-width
    rows (sharing only keys or only values, Sec. 5.5), and `vis` gives every query row the number of leading
    positions it may see (self-attention over the cached sequence, Sec. 2.1), applied as a boolean mask on the
    full score matrix."""
    G = queries.shape[1]
    U = len(hist_off) - 1
    out = np.zeros((int(q_off[-1]), G, d_a), dtype=np.float64)
    qf = _f64(queries)
    for u in range(U):
        p0, L = int(hist_off[u]), int(hist_off[u + 1] - hist_off[u])
        q0, q1 = int(q_off[u]), int(q_off[u + 1])
        if L == 0 or q1 == q0:
            continue
        K = _f64(user_K[p0:p0 + L]) if pool_K is None else materialize_f64(pool_K, idx_K, user_K, p0, L)
        V = _f64(user_V[p0:p0 + L]) if pool_V is None else materialize_f64(pool_V, idx_V, user_V, p0, L)
        n_vis = np.full(q1 - q0, L) if vis is None else np.asarray(vis[q0:q1])
        seen = np.arange(L)[None, :] < n_vis[:, None]        # [M, L]
        for g in range(G):
            S = scale * (qf[q0:q1, g] @ K[:, g].T)           # [M, L]
            if mode == "softmax":
                Sm = np.where(seen, S, -np.inf)
                mx = Sm.max(axis=1, keepdims=True)
                E = np.exp(Sm - np.where(np.isfinite(mx), mx, 0.0))   # exp(-inf) = 0 for what is not seen
                Z = E.sum(axis=1, keepdims=True)
                W = np.divide(E, Z, out=np.zeros_like(E), where=Z > 0)
            else:
                W = np.where(seen, S / (1.0 + np.exp(-S)), 0.0) / L
            out[q0:q1, g] = W @ V[:, g]
    return out
