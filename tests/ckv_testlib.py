"""Helpers shared by the GPU tests: drive the CUDA library through its C ABI on synthetic
inputs and compare with the CPU oracle.  (The oracle is imported here, in test code only.)"""
import numpy as np
import torch

import synth
from oracle import ckv_oracle as O

TOL = {"bf16": (2e-3, 1e-2), "f32": (1e-5, 1e-5)}      # (atol, rtol): |g - o| <= atol + rtol |o|
ROW_TOL = {"bf16": 1e-2, "f32": 2e-5}                   # row-wise max|g - o| / max|o|

_TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}


def to_dev(a, dtype):
    from paper_2601_19178_b200.session import as_device_tensor
    return as_device_tensor(a, dtype)


def make_session(w, data, scale=0.0, out_dtype=None, **options):
    import paper_2601_19178_b200 as ckv
    s = ckv.CollectiveKV(w.n_groups, w.head_dim, _TORCH_DT[w.dtype], w.mode, scale,
                         _TORCH_DT[out_dtype] if out_dtype else None)
    s.pool_load(to_dev(data["pool_K"], w.dtype), to_dev(data["pool_V"], w.dtype))
    s.cache_put_batch(data["users"], data["hist_off"], to_dev(data["idx_K"], "i"),
                      to_dev(data["idx_V"], "i"), to_dev(data["user_K"], w.dtype),
                      to_dev(data["user_V"], w.dtype))
    for k, v in options.items():
        s.set_option(k, v)
    return s


def gpu_attend(w, data, scale=0.0, out_dtype=None, session=None, **options):
    s = session or make_session(w, data, scale, out_dtype, **options)
    out = s.attend(data["users"], data["q_off"], to_dev(data["queries"], w.dtype))
    torch.cuda.synchronize()
    res = out.float().cpu().numpy().astype(np.float64)
    if session is None:
        s.close()
    return res


def oracle_attend(w, data, scale=None, sel=None):
    return O.attend(w.dtype, w.mode, w.default_scale if scale is None else scale, data["pool_K"],
                    data["pool_V"], data["hist_off"], data["idx_K"], data["idx_V"], data["user_K"],
                    data["user_V"], data["q_off"], data["queries"], sel=sel)


def assert_close(got, want, dtype, what=""):
    atol, rtol = TOL[dtype]
    err = np.abs(got - want)
    bound = atol + rtol * np.abs(want)
    worst = float((err - bound).max()) if err.size else -1.0
    assert worst <= 0, f"{what}: element tolerance exceeded by {worst:.3e} (max err {err.max():.3e})"
    if err.size:
        denom = np.abs(want).max(axis=-1, keepdims=True)
        rows = denom[..., 0] > 0
        if rows.any():
            rel = (err.max(axis=-1)[rows] / denom[..., 0][rows]).max()
            assert rel <= ROW_TOL[dtype], f"{what}: row-normalised error {rel:.3e} > {ROW_TOL[dtype]}"
