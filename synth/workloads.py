"""Workload shapes and the seeded generator of synthetic decode-stage inputs.

The five named workloads are the benchmark configurations of this library
(SASRec-style target attention, an HSTU-style pointwise config, long ragged
histories and a high-concurrency serving batch).  They stand in for the
paper's MicroVideo / KuaiVideo / EBNeRD workloads (Sec. 5.1), which are not
available offline: only shapes, value distributions, index skew and length
mix are modelled, no record of any dataset is reproduced.

Array conventions (all C-contiguous numpy arrays):

  pool_K, pool_V : [G, m, d_g]     global K/V pool, one per group (layer x head)
  idx_K,  idx_V  : [P, G] int32    per-position pool indices, P = sum of L_u
  user_K, user_V : [P, G, d_u]     low-dimensional user-specific part
  hist_off       : [U+1] int64     ragged history offsets into the P axis
  queries        : [Q, G, d]       candidate/target queries, Q = sum of M_u
  q_off          : [U+1] int32     ragged query offsets
  users          : [U] int64       user ids (arbitrary, distinct)

Floating tensors are float32 for dtype "f32"; for dtype "bf16" they are uint16
arrays of bfloat16 bit patterns (values drawn in fp32 and rounded once,
round-to-nearest-even).
"""
from __future__ import annotations

import concurrent.futures
import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

SOFTMAX = "softmax"
SILU_OVER_L = "silu_over_l"


@dataclass(frozen=True)
class Workload:
    name: str
    n_groups: int            # layers * heads; each group has its own pool and indices
    d_shared: int            # d_g
    d_user: int              # d_u
    n_entries: int           # m, pool rows per group
    n_users: int
    hist_len: Tuple[int, int]  # (L_min, L_max) inclusive; equal => fixed length
    n_queries: int           # candidates per user (M)
    mode: str                # SOFTMAX | SILU_OVER_L
    dtype: str               # "f32" | "bf16"
    zipf_s: Optional[float]  # None => uniform indices
    pool_var: float          # variance of pool entries
    user_var: float          # variance of user-specific K/V entries
    seed: int
    describe: str = ""

    @property
    def head_dim(self) -> int:
        return self.d_shared + self.d_user

    @property
    def default_scale(self) -> float:
        # softmax: 1/sqrt(d_a); pointwise SiLU config is written without a scale
        return 1.0 / float(np.sqrt(self.head_dim)) if self.mode == SOFTMAX else 1.0


_BASE_SEED = 0xC0117EC7

WORKLOADS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", 2, 28, 4, 1024, 64, (200, 200), 1, SOFTMAX, "f32", None,
                     1.0 / 32, 1.0 / 32, _BASE_SEED + 1,
                     "SASRec-style 1 layer x 2 heads, d=28+4, pool 1024, 64 users, L=200, 1 query, fp32"),
    "cfg2": Workload("cfg2", 8, 30, 2, 4096, 1024, (1024, 1024), 100, SOFTMAX, "bf16", 1.1,
                     1.0 / 32, 1.0 / 32, _BASE_SEED + 2,
                     "SASRec-style 2 layers x 4 heads, d=30+2, pool 4096, 1024 users, L=1024, 100 candidates, bf16"),
    "cfg3": Workload("cfg3", 8, 30, 2, 8192, 2048, (4096, 4096), 128, SILU_OVER_L, "bf16", 1.2,
                     1.0 / 32, 0.05, _BASE_SEED + 3,
                     "HSTU-style SiLU(QK^T)/L, 8 heads, d=30+2, pool 8192, 2048 users, L=4096, 128 candidates, bf16"),
    "cfg4": Workload("cfg4", 4, 60, 4, 16384, 512, (1000, 16384), 1, SOFTMAX, "bf16", None,
                     1.0 / 64, 1.0 / 64, _BASE_SEED + 4,
                     "long ragged histories, 4 heads, d=60+4, pool 16384, 512 users, L~U[1000,16384], 1 query, bf16"),
    "cfg5": Workload("cfg5", 4, 31, 1, 2048, 65536, (512, 512), 16, SOFTMAX, "bf16", 1.05,
                     1.0 / 32, 1.0 / 32, _BASE_SEED + 5,
                     "serving batch, 65536 users, L=512, 4 heads, d=31+1, pool 2048, 16 candidates, bf16"),
}


def scaled(w: Workload, **changes) -> Workload:
    """A copy of `w` with some fields replaced (smaller user counts, lengths...)."""
    return dataclasses.replace(w, **changes)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(rng: np.random.Generator, shape, var: float, dtype: str) -> np.ndarray:
    x = rng.standard_normal(shape, dtype=np.float32)
    x *= np.float32(np.sqrt(var))
    return f32_to_bf16_bits(x) if dtype == "bf16" else x


def _indices(rng: np.random.Generator, P: int, G: int, m: int, zipf_s: Optional[float]) -> np.ndarray:
    """[P, G] int32 pool rows.  Zipf: P(rank r) ~ r^-s, rank -> row through a
    seeded permutation per group, so the hot rows are scattered over the pool."""
    if zipf_s is None:
        return rng.integers(0, m, size=(P, G), dtype=np.int32)
    w = np.arange(1, m + 1, dtype=np.float64) ** (-float(zipf_s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    out = np.empty((P, G), dtype=np.int32)

    def fill(g, perm, u):
        ranks = np.searchsorted(cdf, u, side="left")
        np.minimum(ranks, m - 1, out=ranks)
        out[:, g] = perm[ranks]

    # the draws stay in the stream's order (group by group); only the table look-ups run side by side
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(G, 4)) as ex:
        pending = []
        for g in range(G):
            perm = rng.permutation(m).astype(np.int32)
            pending.append(ex.submit(fill, g, perm, rng.random(P)))
        for f in pending:
            f.result()
    return out


def generate(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Draw every input tensor of workload `w`.  Deterministic in (w, seed)."""
    ss = np.random.SeedSequence(w.seed if seed is None else seed)
    (s_len, s_pk, s_pv, s_ik, s_iv, s_uk, s_uv, s_q, s_id) = [
        np.random.Generator(np.random.Philox(c)) for c in ss.spawn(9)]
    G, m, dg, du, d = w.n_groups, w.n_entries, w.d_shared, w.d_user, w.head_dim
    U, M = w.n_users, w.n_queries
    lo, hi = w.hist_len
    lens = np.full(U, lo, dtype=np.int64) if lo == hi else s_len.integers(lo, hi + 1, size=U, dtype=np.int64)
    hist_off = np.zeros(U + 1, dtype=np.int64)
    np.cumsum(lens, out=hist_off[1:])
    P = int(hist_off[-1])
    q_off = (np.arange(U + 1, dtype=np.int64) * M).astype(np.int32)
    Q = int(q_off[-1])
    # every tensor has a random stream of its own, so the draws can run side by side (numpy releases the
    # interpreter lock inside them) without changing a single value
    jobs = {
        "pool_K": lambda: _normal(s_pk, (G, m, dg), w.pool_var, w.dtype),
        "pool_V": lambda: _normal(s_pv, (G, m, dg), w.pool_var, w.dtype),
        "idx_K": lambda: _indices(s_ik, P, G, m, w.zipf_s),
        "idx_V": lambda: _indices(s_iv, P, G, m, w.zipf_s),
        "user_K": lambda: _normal(s_uk, (P, G, du), w.user_var, w.dtype),
        "user_V": lambda: _normal(s_uv, (P, G, du), w.user_var, w.dtype),
        "queries": lambda: _normal(s_q, (Q, G, d), 1.0, w.dtype),
    }
    if P * G >= 1 << 20:
        with concurrent.futures.ThreadPoolExecutor(max_workers=len(jobs)) as ex:
            futures = {k: ex.submit(f) for k, f in jobs.items()}
            data = {k: f.result() for k, f in futures.items()}
    else:
        data = {k: f() for k, f in jobs.items()}
    data["hist_off"] = hist_off
    data["q_off"] = q_off
    # distinct, non-contiguous ids so that a lookup bug cannot hide behind id == slot
    data["users"] = s_id.permutation(U).astype(np.int64) * 7919 + 1000003
    return data
