"""ckv_attend_static: the decode call for callers that cannot allocate device memory
(latency-critical serving sections, processes whose GPU memory belongs to another allocator).

It must return what ckv_attend returns, call after call, although its work tables and
split-reduction partials live in one fixed array shared by all calls.  This file is collected
last on purpose (its name sorts after the other test files)."""
import numpy as np
import pytest
import torch

import synth
from ckv_testlib import assert_close, make_session, oracle_attend, to_dev

pytestmark = pytest.mark.gpu


def _run(fn, s, users, q_off, q):
    out = torch.full(q.shape, float("nan"), dtype=s.out_dtype, device=q.device)
    fn(s.ctx, users, q_off, q, out)
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("name,kw,family", [
    ("cfg4", dict(n_users=5, hist_len=(1, 5000), n_queries=2), 2),   # warp-level tensor-core kernel, 64-wide heads
    ("cfg5", dict(n_users=40, hist_len=(1, 900)), 2),                # warp-level tensor-core kernel, 32-wide heads
    ("cfg1", dict(n_users=90, hist_len=(1, 1500), n_queries=3), 1),  # fp32: CUDA-core kernel; two table launches
])
def test_static_entry_point_matches_ckv_attend_twice_in_a_row(name, kw, family):
    import paper_2601_19178_b200 as ckv
    w = synth.scaled(synth.WORKLOADS[name], **kw)
    d = synth.generate(w)
    s = make_session(w, d, split_len=256)
    q = to_dev(d["queries"], w.dtype)
    want = _run(ckv.ckv_attend, s, d["users"], d["q_off"], q)
    assert s.stat("split_items") > 0, "the case must exercise the scratch memory"
    assert s.stat("kernel") == family
    # the first call on a device does the set-up (the driver may only now load the part of the library's device
    # image that holds the array); from then on the device's free memory must not move (the output tensor of
    # _run comes out of torch's cache, which the earlier runs of the same shape have filled)
    first = _run(ckv.ckv_attend_static, s, d["users"], d["q_off"], q)
    free_before = torch.cuda.mem_get_info()[0]
    # a different request in between leaves other contents in the shared array
    half = w.n_users // 2
    _run(ckv.ckv_attend_static, s, d["users"][:half], d["q_off"][:half + 1], q[: int(d["q_off"][half])])
    second = _run(ckv.ckv_attend_static, s, d["users"], d["q_off"], q)
    assert torch.cuda.mem_get_info()[0] == free_before, "ckv_attend_static changed the device's free memory"
    assert_close(first, want, w.dtype, "first call")
    assert_close(second, want, w.dtype, "second call")
    assert np.array_equal(first, second)
    assert_close(first, oracle_attend(w, d), w.dtype, "vs oracle")
    s.close()


def test_static_entry_point_rejects_what_does_not_fit():
    import paper_2601_19178_b200 as ckv
    w = synth.scaled(synth.WORKLOADS["cfg5"], n_users=300, hist_len=(64, 64))
    d = synth.generate(w)
    s = make_session(w, d)
    q = to_dev(d["queries"], w.dtype)
    out = torch.empty_like(q)
    with pytest.raises(ckv.CkvError) as e:                       # more than 256 users in one call
        ckv.ckv_attend_static(s.ctx, d["users"], d["q_off"], q, out)
    assert e.value.status == ckv.CKV_ERR_TOO_LARGE
    with pytest.raises(ckv.CkvError) as e:                       # host buffers would need staging memory
        ckv.ckv_attend_static(s.ctx, d["users"][:4], d["q_off"][:5], q.cpu(), out)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
    s.close()
    # partial results beyond the fixed array: many chunks x many queries
    w2 = synth.scaled(synth.WORKLOADS["cfg2"], n_users=64, hist_len=(4096, 4096), n_queries=128)
    d2 = synth.generate(w2)
    s2 = make_session(w2, d2, split_len=64)
    q2 = to_dev(d2["queries"], w2.dtype)
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_attend_static(s2.ctx, d2["users"], d2["q_off"], q2, torch.empty_like(q2))
    assert e.value.status == ckv.CKV_ERR_TOO_LARGE
    s2.close()
