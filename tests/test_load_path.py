"""Decode-stage load path (Sec. 4.4): packed caches exported to host memory, imported per request
batch, attended.  The blob layout documented in include/ckv.h is rebuilt here in numpy from the raw
inputs, so the test pins the format and not just a round trip."""
import numpy as np
import pytest
import torch

import synth
from ckv_testlib import assert_close, gpu_attend, make_session, oracle_attend, to_dev

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS
CASES = {
    "cfg1": synth.scaled(W["cfg1"], n_users=5, hist_len=(0, 90)),                      # fp32, 16-bit indices
    "cfg4": synth.scaled(W["cfg4"], n_users=6, hist_len=(1, 300)),                     # bf16, d_user 4
    "cfg5": synth.scaled(W["cfg5"], n_users=9, hist_len=(33, 33)),                     # bf16, d_user 1
    "wide_idx": synth.Workload("wide", 2, 32, 0, 70000, 4, (7, 120), 3, "softmax", "bf16", None, 1 / 32, 1 / 32, 5),
}


def expected_blob(w, d, order):
    """The documented layout: [K idx | V idx | user K | user V], per user [G][Lpad] entries, padding
    entries zero, sections at multiples of 256 bytes."""
    G, du = w.n_groups, w.d_user
    idt = np.uint16 if w.n_entries <= 65536 else np.int32
    edt = np.uint32 if w.dtype == "f32" else np.uint16
    secs = [[], [], [], []]
    for u in order:
        a, b = int(d["hist_off"][u]), int(d["hist_off"][u + 1])
        L = b - a
        Lpad = (L + 31) // 32 * 32
        for si, key in enumerate(("idx_K", "idx_V")):
            t = np.zeros((G, Lpad), dtype=idt)
            t[:, :L] = d[key][a:b].T.astype(idt)
            secs[si].append(t.reshape(-1))
        for si, key in enumerate(("user_K", "user_V")):
            t = np.zeros((G, Lpad, du), dtype=edt)
            if du > 0:
                src = d[key][a:b]
                t[:, :L, :] = np.transpose(src.view(edt) if src.dtype != edt else src, (1, 0, 2))
            secs[2 + si].append(t.reshape(-1))
    out = bytearray()
    for sec in secs:
        raw = np.concatenate(sec).tobytes() if sec else b""
        out += raw
        out += b"\0" * ((-len(out)) % 256)
    return bytes(out)


@pytest.mark.parametrize("name", sorted(CASES))
def test_export_matches_documented_layout_and_import_reproduces_attention(name):
    import paper_2601_19178_b200 as ckv
    w = CASES[name]
    d = synth.generate(w)
    s = make_session(w, d)
    ref = gpu_attend(w, d, session=s)
    order = list(range(w.n_users))[::-1]                       # any order of users
    users = d["users"][order]
    blob = s.export_blob(users)
    L = np.diff(d["hist_off"])[order].astype(np.int32)
    assert blob.numel() == ckv.ckv_cache_blob_bytes(s.ctx, L)
    assert blob.numpy().tobytes() == expected_blob(w, d, order)
    s.close()

    # a fresh context that only knows the pool: load the batch, attend
    dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    s2 = ckv.CollectiveKV(w.n_groups, w.head_dim, dt, w.mode)
    s2.pool_load(to_dev(d["pool_K"], w.dtype), to_dev(d["pool_V"], w.dtype))
    s2.import_blob(users, L, blob)
    got = gpu_attend(w, d, session=s2)
    assert np.array_equal(got, ref), "imported caches must give bit-identical outputs"
    assert_close(got, oracle_attend(w, d), w.dtype, name)
    # the same blob from device memory, under new ids, next to the first copy
    s2.import_blob(users + 1000, L, blob.cuda())
    d2 = dict(d)
    d2["users"] = d["users"] + 1000
    assert np.array_equal(gpu_attend(w, d2, session=s2), ref)
    comp, _ = ckv.ckv_cache_bytes(s2.ctx)
    s2.close()
    per_unit = 2 * (2 if w.n_entries <= 65536 else 4) + 2 * w.d_user * (4 if w.dtype == "f32" else 2)
    assert comp == 2 * int(d["hist_off"][-1]) * w.n_groups * per_unit


def test_import_rejects_bad_blobs_and_leaves_the_cache_unchanged():
    import paper_2601_19178_b200 as ckv
    w = CASES["cfg5"]
    d = synth.generate(w)
    s = make_session(w, d)
    users = d["users"]
    L = np.diff(d["hist_off"]).astype(np.int32)
    blob = s.export_blob(users)
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_cache_export(s.ctx, np.array([987654], dtype=np.int64), blob, blob.numel())
    assert e.value.status == ckv.CKV_ERR_UNKNOWN_USER
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_cache_import(s.ctx, users + 50, L, blob, blob.numel() - 256)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_cache_import(s.ctx, users + 50, -L, blob, blob.numel())
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
    bad = blob.clone()
    bad.view(torch.int16)[5] = w.n_entries                     # one K index out of range (pool has 2048 rows)
    with pytest.raises(ckv.CkvError) as e:
        s.import_blob(users + 50, L, bad)
    assert e.value.status == ckv.CKV_ERR_INDEX_RANGE
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_user_length(s.ctx, int(users[0]) + 50)
    assert e.value.status == ckv.CKV_ERR_UNKNOWN_USER
    # the original users are untouched
    assert_close(gpu_attend(w, d, session=s), oracle_attend(w, d), w.dtype, "after rejected import")
    s.close()


@pytest.mark.parametrize("name", ["cfg1", "cfg4", "cfg5"])
def test_append_equals_put_of_the_whole_history(name):
    """New interactions appended in two steps: the packed cache and the attention output must be the bits that
    a single put of the whole history gives."""
    import paper_2601_19178_b200 as ckv
    w = synth.scaled(CASES[name], hist_len=(40, 200))
    d = synth.generate(w)
    ref = make_session(w, d)
    want_out = gpu_attend(w, d, session=ref)
    want_blob = ref.export_blob(d["users"]).numpy().tobytes()
    ref.close()

    dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    s = ckv.CollectiveKV(w.n_groups, w.head_dim, dt, w.mode)
    s.pool_load(to_dev(d["pool_K"], w.dtype), to_dev(d["pool_V"], w.dtype))
    ho = d["hist_off"]
    cuts = [(3, 30), (0, 17), (39, 1)]                           # (first put, first append) positions; rest in the second append
    for u in range(w.n_users):
        a, b = int(ho[u]), int(ho[u + 1])
        n0, n1 = cuts[u % len(cuts)]
        c0, c1 = a + n0, a + n0 + n1
        sl = lambda lo, hi: (to_dev(d["idx_K"][lo:hi], "i"), to_dev(d["idx_V"][lo:hi], "i"),
                             to_dev(d["user_K"][lo:hi], w.dtype), to_dev(d["user_V"][lo:hi], w.dtype))
        s.cache_put(int(d["users"][u]), *sl(a, c0))
        s.cache_append(int(d["users"][u]), *sl(c0, c1))
        # host inputs for the second append
        ckv.ckv_cache_append(s.ctx, int(d["users"][u]), b - c1, np.ascontiguousarray(d["idx_K"][c1:b]),
                             np.ascontiguousarray(d["idx_V"][c1:b]), np.ascontiguousarray(d["user_K"][c1:b]),
                             np.ascontiguousarray(d["user_V"][c1:b]), w.d_user)
        assert ckv.ckv_user_length(s.ctx, int(d["users"][u])) == b - a
    assert s.export_blob(d["users"]).numpy().tobytes() == want_blob
    assert np.array_equal(gpu_attend(w, d, session=s), want_out)
    comp, _ = ckv.ckv_cache_bytes(s.ctx)
    assert comp == int(ho[-1]) * w.n_groups * (2 * 2 + 2 * w.d_user * (4 if w.dtype == "f32" else 2))
    # error paths: unknown user, index out of range (the user keeps the old history)
    u0 = int(d["users"][0])
    one = (np.zeros((1, w.n_groups), np.int32), np.zeros((1, w.n_groups), np.int32),
           np.zeros((1, w.n_groups, w.d_user), d["user_K"].dtype), np.zeros((1, w.n_groups, w.d_user), d["user_K"].dtype))
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_cache_append(s.ctx, 424242, 1, *one, w.d_user)
    assert e.value.status == ckv.CKV_ERR_UNKNOWN_USER
    bad = (np.full((1, w.n_groups), w.n_entries, np.int32),) + one[1:]
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_cache_append(s.ctx, u0, 1, *bad, w.d_user)
    assert e.value.status == ckv.CKV_ERR_INDEX_RANGE
    assert ckv.ckv_user_length(s.ctx, u0) == int(ho[1] - ho[0])
    assert np.array_equal(gpu_attend(w, d, session=s), want_out)
    s.close()


def test_storage_of_replaced_and_evicted_users_is_reused():
    """A cache that is updated continuously must not grow: replacing one user a thousand times, cycling
    import / evict over a batch and appending to a user all hand their old storage back."""
    import paper_2601_19178_b200 as B
    w = synth.scaled(synth.WORKLOADS["cfg5"], n_users=24, hist_len=(40, 700))
    d = synth.generate(w)
    s = make_session(w, d)
    cap0 = s.stat("arena_capacity_units")
    G = w.n_groups
    ho = d["hist_off"]
    ik, iv = to_dev(d["idx_K"], "i"), to_dev(d["idx_V"], "i")
    uk, uv = to_dev(d["user_K"], w.dtype), to_dev(d["user_V"], w.dtype)
    want = gpu_attend(w, d, session=s)
    # one user replaced 1000 times by histories of the other users' lengths
    target = int(d["users"][3])
    for r in range(1000):
        u = r % w.n_users
        sl = slice(int(ho[u]), int(ho[u + 1]))
        s.cache_put(target, ik[sl], iv[sl], uk[sl], uv[sl])
    sl = slice(int(ho[3]), int(ho[4]))
    s.cache_put(target, ik[sl], iv[sl], uk[sl], uv[sl])
    assert s.stat("arena_capacity_units") <= 2 * cap0
    assert np.array_equal(gpu_attend(w, d, session=s), want)
    # import / evict cycles of half the users
    half = d["users"][: w.n_users // 2]
    lens = np.diff(ho)[: w.n_users // 2].astype(np.int32)
    blob = s.export_blob(half)
    used = []
    for _ in range(50):
        for u in half:
            B.ckv_cache_evict(s.ctx, int(u))
        s.import_blob(half, lens, blob)
        used.append(s.stat("arena_used_units"))
    assert s.stat("arena_capacity_units") <= 2 * cap0 and max(used) <= 2 * cap0
    assert np.array_equal(gpu_attend(w, d, session=s), want)
    # everything evicted: nothing stays in use
    for u in d["users"]:
        B.ckv_cache_evict(s.ctx, int(u))
    assert s.stat("arena_used_units") == 0 and s.stat("arena_free_runs") == 0
    s.close()
