"""The C ABI: the library loads, exports what include/ckv.h declares (CPU), and returns the
documented error codes (GPU)."""
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "ckv.h")).read()
    return sorted(set(re.findall(r"CKV_API[^;(]*?\b(ckv_[a-z0-9_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    import __graft_entry__ as entry
    entry.build()
    import paper_2601_19178_b200 as ckv
    names = _declared()
    assert len(names) >= 15
    assert sorted(ckv.EXPORTS) == names
    for n in names:
        assert getattr(ckv.lib, n) is not None
    assert ckv.ckv_version() >= 100
    assert ckv.lib.ckv_strerror(ckv.CKV_ERR_UNKNOWN_USER) == b"unknown user"


def test_header_is_plain_c(tmp_path):
    import subprocess
    src = tmp_path / "t.c"
    src.write_text('#include "ckv.h"\nint main(void){ckv_config c; (void)c; return (int)CKV_OK;}\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-c", str(src),
                    "-o", str(tmp_path / "t.o")], check=True)


def test_create_rejects_bad_configs_without_a_gpu():
    import paper_2601_19178_b200 as ckv
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_create(0, 32, ckv.CKV_BF16, ckv.CKV_SOFTMAX)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_create(2, 48, ckv.CKV_BF16, ckv.CKV_SOFTMAX)
    assert e.value.status == ckv.CKV_ERR_UNSUPPORTED
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_create(2, 32, 7, ckv.CKV_SOFTMAX)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG


@pytest.mark.gpu
def test_error_codes():
    import torch
    import paper_2601_19178_b200 as ckv
    import synth
    from ckv_testlib import to_dev
    w = synth.Workload("abi", 2, 30, 2, 50, 2, (10, 10), 1, "softmax", "bf16", None, 1 / 32, 1 / 32, 9)
    d = synth.generate(w)
    ctx = ckv.ckv_create(2, 32, ckv.CKV_BF16, ckv.CKV_SOFTMAX)
    ik, iv = to_dev(d["idx_K"], "i"), to_dev(d["idx_V"], "i")
    uk, uv = to_dev(d["user_K"], "bf16"), to_dev(d["user_V"], "bf16")
    q = to_dev(d["queries"], "bf16")
    out = torch.empty_like(q)

    def status(fn, *a):
        with pytest.raises(ckv.CkvError) as e:
            fn(*a)
        return e.value.status

    assert status(ckv.ckv_cache_put_batch, ctx, d["users"], d["hist_off"], ik, iv, uk, uv, 2) == ckv.CKV_ERR_STATE
    assert status(ckv.ckv_attend, ctx, d["users"], d["q_off"], q, out) == ckv.CKV_ERR_STATE
    pk, pv = to_dev(d["pool_K"], "bf16"), to_dev(d["pool_V"], "bf16")
    assert status(ckv.ckv_pool_load, ctx, pk, pv, 50, 33) == ckv.CKV_ERR_SHAPE
    assert status(ckv.ckv_pool_load, ctx, pk, None, 50, 30) == ckv.CKV_ERR_INVALID_ARG
    ckv.ckv_pool_load(ctx, pk, pv, 50, 30)
    assert status(ckv.ckv_cache_put_batch, ctx, d["users"], d["hist_off"], ik, iv, uk, uv, 3) == ckv.CKV_ERR_SHAPE
    assert status(ckv.ckv_attend, ctx, d["users"], d["q_off"], q, out) == ckv.CKV_ERR_UNKNOWN_USER
    bad = ik.clone()
    bad[7, 1] = 50
    assert status(ckv.ckv_cache_put_batch, ctx, d["users"], d["hist_off"], bad, iv, uk, uv, 2) == ckv.CKV_ERR_INDEX_RANGE
    bad[7, 1] = -1
    assert status(ckv.ckv_cache_put_batch, ctx, d["users"], d["hist_off"], ik, bad, uk, uv, 2) == ckv.CKV_ERR_INDEX_RANGE
    assert status(ckv.ckv_user_length, ctx, int(d["users"][0])) == ckv.CKV_ERR_UNKNOWN_USER   # nothing stored
    ckv.ckv_cache_put_batch(ctx, d["users"], d["hist_off"], ik, iv, uk, uv, 2)
    assert ckv.ckv_user_length(ctx, int(d["users"][1])) == 10
    assert status(ckv.ckv_pool_load, ctx, pk, pv, 49, 30) == ckv.CKV_ERR_SHAPE       # users are cached
    assert status(ckv.ckv_attend, ctx, d["users"], np.array([0, 2, 1], np.int32), q, out) == ckv.CKV_ERR_INVALID_ARG
    assert status(ckv.ckv_attend, ctx, np.array([1, 2], np.int64), d["q_off"], q, out) == ckv.CKV_ERR_UNKNOWN_USER
    assert status(ckv.ckv_set_option, ctx, "no_such_option", 1) == ckv.CKV_ERR_INVALID_ARG
    ckv.ckv_attend(ctx, d["users"], d["q_off"], q, out)            # still usable after all of that
    torch.cuda.synchronize()
    assert ckv.ckv_last_stat(ctx, "launches") >= 1
    assert torch.isfinite(out.float()).all()
    ckv.ckv_cache_clear(ctx)
    assert ckv.ckv_cache_bytes(ctx) == (0, 0)
    ckv.ckv_destroy(ctx)
