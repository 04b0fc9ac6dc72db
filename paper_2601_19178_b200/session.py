"""A small convenience wrapper over the C-ABI calls for torch users: owns the context
handle and converts between torch dtypes and the library's enums.  No arithmetic here."""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from . import binding as B

_DT = {torch.float32: B.CKV_F32, torch.bfloat16: B.CKV_BF16}
_MODE = {"softmax": B.CKV_SOFTMAX, "silu_over_l": B.CKV_SILU_OVER_L}


def as_device_tensor(a: np.ndarray, dtype: str, device="cuda") -> torch.Tensor:
    """numpy array (float32, or uint16 bf16 bit patterns, or integers) -> device tensor."""
    if dtype == "bf16" and a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


class CollectiveKV:
    def __init__(self, n_groups: int, head_dim: int, dtype: torch.dtype, mode: str = "softmax",
                 scale: float = 0.0, out_dtype: Optional[torch.dtype] = None, device: int = 0):
        self.n_groups, self.head_dim, self.dtype = n_groups, head_dim, dtype
        self.out_dtype = out_dtype or dtype
        self.device = torch.device("cuda", device)
        self.d_user = None
        self.ctx = B.ckv_create(n_groups, head_dim, _DT[dtype], _MODE[mode], scale, _DT[self.out_dtype], device)

    def close(self):
        if self.ctx:
            B.ckv_destroy(self.ctx)
            self.ctx = None

    __del__ = close

    def pool_load(self, pool_K: torch.Tensor, pool_V: torch.Tensor):
        G, m, dg = pool_K.shape
        assert G == self.n_groups and pool_V.shape == pool_K.shape and pool_K.dtype == self.dtype
        B.ckv_pool_load(self.ctx, pool_K, pool_V, m, dg)
        self.d_user = self.head_dim - dg

    def pool_load_sides(self, pool_K: Optional[torch.Tensor], pool_V: Optional[torch.Tensor]):
        """Sharing only keys or only values: None for the side that is not shared (its rows are then cached full
        width and handed to the cache calls as that side's user part)."""
        shared = [p for p in (pool_K, pool_V) if p is not None]
        m = shared[0].shape[1] if shared else 1
        dk = 0 if pool_K is None else pool_K.shape[2]
        dv = 0 if pool_V is None else pool_V.shape[2]
        B.ckv_pool_load_sides(self.ctx, pool_K, pool_V, m, dk, dv)
        self.d_user = self.head_dim - max(dk, dv)

    def cache_put(self, user: int, idx_K, idx_V, user_K, user_V):
        B.ckv_cache_put(self.ctx, user, idx_K.shape[0], idx_K, idx_V, user_K, user_V, self.d_user)

    def cache_append(self, user: int, idx_K, idx_V, user_K, user_V):
        """New interactions behind a cached user's history (arguments describe the new positions only)."""
        B.ckv_cache_append(self.ctx, user, idx_K.shape[0], idx_K, idx_V, user_K, user_V, self.d_user)

    def cache_put_batch(self, users, hist_off, idx_K, idx_V, user_K, user_V):
        B.ckv_cache_put_batch(self.ctx, users, hist_off, idx_K, idx_V, user_K, user_V, self.d_user)

    def attend(self, users, q_off, queries: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty(queries.shape, dtype=self.out_dtype, device=queries.device)
        B.ckv_attend(self.ctx, users, q_off, queries, out)
        return out

    def attend_visible(self, users, q_off, vis, queries: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """attend with a visible length per query row (self-attention over the cached sequence)."""
        if out is None:
            out = torch.empty(queries.shape, dtype=self.out_dtype, device=queries.device)
        B.ckv_attend_visible(self.ctx, users, q_off, vis, queries, out)
        return out

    def export_blob(self, users) -> torch.Tensor:
        """Packed caches of `users` as one pinned host buffer (the form a serving system keeps in
        host memory and loads per request batch)."""
        L = [B.ckv_user_length(self.ctx, int(u)) for u in users]
        nbytes = B.ckv_cache_blob_bytes(self.ctx, L)
        blob = torch.empty(max(nbytes, 1), dtype=torch.uint8).pin_memory()
        B.ckv_cache_export(self.ctx, users, blob, nbytes)
        torch.cuda.current_stream().synchronize()
        return blob[:nbytes]

    def import_blob(self, users, lengths, blob: torch.Tensor):
        """Loads `users` (history lengths `lengths`) from a packed blob (host or device tensor)."""
        B.ckv_cache_import(self.ctx, users, lengths, blob, blob.numel() * blob.element_size())

    def materialize(self, user: int):
        L = B.ckv_user_length(self.ctx, user)
        K = torch.empty((L, self.n_groups, self.head_dim), dtype=self.dtype, device=self.device)
        V = torch.empty_like(K)
        B.ckv_materialize(self.ctx, user, K, V)
        return K, V

    def set_option(self, name: str, value: int):
        B.ckv_set_option(self.ctx, name, value)

    def stat(self, name: str) -> int:
        return B.ckv_last_stat(self.ctx, name)
