"""Oracle of the prefill router (Sec. 4.3), numpy float64.

TEST INFRASTRUCTURE ONLY.  The router scores every history position against every global-pool
entry, M = X W_g^T + b_g per group g, and the position takes the entry with the largest score:
I[i][g] = argmax_j M[i][j].  Written out as that definition: one matrix product per group, one
arg-max per row (numpy's arg-max returns the first, i.e. lowest, index among equal maxima).
Inputs may be bfloat16 bit patterns (uint16), widened exactly.
"""
from __future__ import annotations

import numpy as np


def _f64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:  # bfloat16 bit patterns, widened exactly
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def scores(x, W, bias=None) -> np.ndarray:
    """M [G][n][m] float64 for x [n][d_in], W [G][m][d_in], bias [G][m] or None."""
    X, Wf = _f64(x), _f64(W)
    M = np.stack([X @ Wf[g].T for g in range(Wf.shape[0])])
    if bias is not None:
        M = M + np.asarray(bias, dtype=np.float64)[:, None, :]
    return M


def route(x, W, bias=None) -> np.ndarray:
    """I [n][G] int32: lowest index of the row maximum of M."""
    return np.argmax(scores(x, W, bias), axis=2).T.astype(np.int32)


def project(x, W, bias=None) -> np.ndarray:
    """User-specific low-dimensional part (Sec. 4.2): y [n][G][d_out] float64 = x . W[g][c] + bias[g][c]
    for x [n][d_in], W [G][d_out][d_in], bias [G][d_out] or None -- the linear layer written out."""
    X, Wf = _f64(x), _f64(W)
    y = np.einsum("nk,gck->ngc", X, Wf)
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None]
    return y
