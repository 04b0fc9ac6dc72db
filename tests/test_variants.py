"""The two variants of the decode path through the C ABI against the oracle: sharing only keys or only values
(Sec. 5.5, ablation on sharing keys or values) and a visible length per query (self-attention over the cached
sequence, Sec. 2.1)."""
import numpy as np
import pytest
import torch

import synth
from ckv_testlib import _TORCH_DT, assert_close, to_dev
from oracle import ckv_oracle as O

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS


def full_rows(d, side):
    """Full-width rows of one side for all positions (numpy indexing; user part first)."""
    pool, idx, user = d["pool_" + side], d["idx_" + side], d["user_" + side]
    G = pool.shape[0]
    return np.ascontiguousarray(np.concatenate([user, pool[np.arange(G)[None, :], idx]], axis=-1))


def side_session(w, d, share_k, share_v, **options):
    import paper_2601_19178_b200 as ckv
    s = ckv.CollectiveKV(w.n_groups, w.head_dim, _TORCH_DT[w.dtype], w.mode)
    s.pool_load_sides(to_dev(d["pool_K"], w.dtype) if share_k else None, to_dev(d["pool_V"], w.dtype) if share_v else None)
    uk = d["user_K"] if share_k else full_rows(d, "K")
    uv = d["user_V"] if share_v else full_rows(d, "V")
    s.cache_put_batch(d["users"], d["hist_off"], to_dev(d["idx_K"], "i") if share_k else None,
                      to_dev(d["idx_V"], "i") if share_v else None, to_dev(uk, w.dtype), to_dev(uv, w.dtype))
    for k, v in options.items():
        s.set_option(k, v)
    return s, uk, uv


def oracle_sides(w, d, share_k, share_v, uk, uv, vis=None):
    return O.attend_variants(w.dtype, w.mode, w.default_scale, w.head_dim, d["pool_K"] if share_k else None,
                             d["pool_V"] if share_v else None, d["hist_off"], d["idx_K"], d["idx_V"], uk, uv,
                             d["q_off"], d["queries"], vis=vis)


SIDE_CASES = {
    "cfg1": synth.scaled(W["cfg1"], n_users=7, hist_len=(1, 700), n_queries=3),       # fp32: CUDA-core kernel
    "cfg4": synth.scaled(W["cfg4"], n_users=6, hist_len=(1, 3000), n_queries=2),      # 64-wide heads, split histories
    "cfg5": synth.scaled(W["cfg5"], n_users=30, hist_len=(1, 600)),                   # 32-wide heads, 16 queries
    "cfg3": synth.scaled(W["cfg3"], n_users=3, hist_len=(100, 900), n_queries=40),    # SiLU, 40 queries (three 16-row tiles)
}


@pytest.mark.parametrize("name", sorted(SIDE_CASES))
@pytest.mark.parametrize("share", [(True, False), (False, True), (False, False)], ids=["K_only", "V_only", "none"])
@pytest.mark.parametrize("kernel,loader", [(0, 0), (1, 0), (2, 1)])
def test_one_sided_sharing_matches_oracle(name, share, kernel, loader):
    w = SIDE_CASES[name]
    if kernel == 2 and w.dtype == "f32":
        pytest.skip("the warp-level tensor-core kernel takes bf16 only")
    d = synth.generate(w)
    s, uk, uv = side_session(w, d, *share, kernel=kernel, split_len=256, mma_loader=loader)
    out = s.attend(d["users"], d["q_off"], to_dev(d["queries"], w.dtype))
    torch.cuda.synchronize()
    assert s.stat("kernel") == (1 if kernel == 1 or w.dtype == "f32" else 2)
    assert_close(out.float().cpu().numpy().astype(np.float64), oracle_sides(w, d, *share, uk, uv), w.dtype,
                 f"{name} share={share}")
    # the rebuilt rows are a pure copy of input bits
    u = w.n_users // 2
    p0, p1 = int(d["hist_off"][u]), int(d["hist_off"][u + 1])
    K, V = s.materialize(int(d["users"][u]))
    for got, side in ((K, "K"), (V, "V")):
        want = full_rows(d, side)[p0:p1]
        g = got.view(torch.int16).cpu().numpy().view(np.uint16) if w.dtype == "bf16" else got.cpu().numpy()
        assert np.array_equal(g, want)
    # storage accounting: a side that is not shared costs the full row and no index
    import paper_2601_19178_b200 as ckv
    comp, full = ckv.ckv_cache_bytes(s.ctx)
    e = 4 if w.dtype == "f32" else 2
    per_unit = sum((2 + w.d_user * e) if sh else w.head_dim * e for sh in share)
    assert comp == int(d["hist_off"][-1]) * w.n_groups * per_unit
    s.close()


@pytest.mark.parametrize("name,kw", [("cfg2", dict(n_users=5, hist_len=(1, 900))),
                                     ("cfg3", dict(n_users=3, hist_len=(100, 1400)))])
@pytest.mark.parametrize("share", [(True, False), (False, True), (False, False)], ids=["K_only", "V_only", "none"])
def test_one_sided_sharing_on_the_tcgen05_kernel(name, kw, share):
    """Many queries per user: the library's choice for these shapes is the tcgen05 kernel, whose producers copy a
    side that is not shared from the user's full-width rows."""
    w = synth.scaled(W[name], **kw)
    d = synth.generate(w)
    s, uk, uv = side_session(w, d, *share, split_len=512)
    out = s.attend(d["users"], d["q_off"], to_dev(d["queries"], w.dtype))
    torch.cuda.synchronize()
    assert s.stat("kernel") == 3 and s.stat("device_errors") == 0
    assert_close(out.float().cpu().numpy().astype(np.float64), oracle_sides(w, d, *share, uk, uv), w.dtype,
                 f"{name} share={share}")
    s.close()


def test_one_sided_sharing_survives_export_import_and_append():
    w = synth.scaled(W["cfg5"], n_users=8, hist_len=(5, 300))
    d = synth.generate(w)
    s, uk, uv = side_session(w, d, True, False)
    q = to_dev(d["queries"], w.dtype)
    want = s.attend(d["users"], d["q_off"], q).clone()
    lens = np.diff(d["hist_off"]).astype(np.int32)
    blob = s.export_blob(d["users"])
    import paper_2601_19178_b200 as ckv
    t = ckv.CollectiveKV(w.n_groups, w.head_dim, torch.bfloat16, w.mode)
    t.pool_load_sides(to_dev(d["pool_K"], w.dtype), None)
    t.import_blob(d["users"], lens, blob)
    assert torch.equal(t.attend(d["users"], d["q_off"], q), want)
    # append: user 0 put with half of its history, the rest appended
    a, b = int(d["hist_off"][0]), int(d["hist_off"][1])
    h = a + (b - a) // 2
    u0 = int(d["users"][0])
    t.cache_put(u0, to_dev(d["idx_K"][a:h], "i"), None, to_dev(uk[a:h], w.dtype), to_dev(uv[a:h], w.dtype))
    t.cache_append(u0, to_dev(d["idx_K"][h:b], "i"), None, to_dev(uk[h:b], w.dtype), to_dev(uv[h:b], w.dtype))
    assert torch.equal(t.attend(d["users"], d["q_off"], q), want)
    s.close()
    t.close()


def test_pool_load_sides_rejects_what_it_cannot_store():
    import paper_2601_19178_b200 as ckv
    w = synth.scaled(W["cfg5"], n_users=2, hist_len=(8, 8))
    d = synth.generate(w)
    s = ckv.CollectiveKV(w.n_groups, w.head_dim, torch.bfloat16, w.mode)
    pk = to_dev(d["pool_K"], w.dtype)
    with pytest.raises(ckv.CkvError) as e:                       # two shared sides of different widths
        ckv.ckv_pool_load_sides(s.ctx, pk, pk[:, :, :16].contiguous(), w.n_entries, w.d_shared, 16)
    assert e.value.status == ckv.CKV_ERR_SHAPE
    with pytest.raises(ckv.CkvError) as e:                       # a shared side needs its pool
        ckv.ckv_pool_load_sides(s.ctx, None, pk, w.n_entries, w.d_shared, w.d_shared)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
    s.close()


# ---------------------------------------------------------------- visible lengths
def _vis_for(w, d, kind, rng):
    lens = np.diff(d["hist_off"])
    out = []
    for L in lens:
        M = w.n_queries
        if kind == "causal_tail":          # the last M positions as queries of a causal self-attention
            out.append(np.clip(np.arange(L - M + 1, L + 1), 0, L))
        elif kind == "causal_spread":      # M queries spread over the history, each seeing what lies before it
            out.append(np.clip(np.linspace(0, L, M).astype(np.int64), 0, L))
        elif kind == "random":
            out.append(rng.integers(0, L + 1, size=M))
        else:                              # everything visible: must equal ckv_attend
            out.append(np.full(M, L))
    return np.concatenate(out).astype(np.int32)


VIS_CASES = {
    "cfg1": synth.scaled(W["cfg1"], n_users=6, hist_len=(1, 900), n_queries=5),
    "cfg4": synth.scaled(W["cfg4"], n_users=5, hist_len=(1, 2500), n_queries=3),
    "cfg5": synth.scaled(W["cfg5"], n_users=20, hist_len=(1, 700)),
    "cfg2": synth.scaled(W["cfg2"], n_users=3, hist_len=(200, 900), n_queries=44),
    "cfg3": synth.scaled(W["cfg3"], n_users=3, hist_len=(100, 800), n_queries=24),
}


@pytest.mark.parametrize("name", sorted(VIS_CASES))
@pytest.mark.parametrize("kind", ["causal_tail", "random"])
@pytest.mark.parametrize("kernel,loader", [(0, 0), (1, 0), (2, 1)])
def test_visible_lengths_match_oracle(name, kind, kernel, loader):
    from ckv_testlib import make_session
    w = VIS_CASES[name]
    if kernel == 2 and w.dtype == "f32":
        pytest.skip("the warp-level tensor-core kernel takes bf16 only")
    d = synth.generate(w)
    vis = _vis_for(w, d, kind, np.random.default_rng(3))
    s = make_session(w, d, kernel=kernel, split_len=256, mma_loader=loader)
    q = to_dev(d["queries"], w.dtype)
    out = s.attend_visible(d["users"], d["q_off"], vis, q)                                  # host array
    out_dev = s.attend_visible(d["users"], d["q_off"], torch.from_numpy(vis).cuda(), q)     # device tensor
    torch.cuda.synchronize()
    assert torch.equal(out, out_dev)
    want = O.attend_variants(w.dtype, w.mode, w.default_scale, w.head_dim, d["pool_K"], d["pool_V"], d["hist_off"],
                             d["idx_K"], d["idx_V"], d["user_K"], d["user_V"], d["q_off"], d["queries"], vis=vis)
    assert_close(out.float().cpu().numpy().astype(np.float64), want, w.dtype, f"{name} {kind}")
    s.close()


@pytest.mark.parametrize("name,kw", [
    ("cfg2", dict(n_users=4, hist_len=(1, 1500), n_queries=100)),      # softmax, one block of queries, tails
    ("cfg2", dict(n_users=3, hist_len=(300, 2500), n_queries=300)),    # three blocks of queries per user
    ("cfg3", dict(n_users=3, hist_len=(100, 1700), n_queries=128)),    # SiLU
])
@pytest.mark.parametrize("kind", ["causal_tail", "causal_spread", "random", "all"])
@pytest.mark.parametrize("split_len", [0, 512])
def test_visible_lengths_on_the_tcgen05_kernel(name, kw, kind, split_len):
    """Many queries per user (self-attention over the cached sequence is the case with as many queries as
    positions): the tcgen05 kernel masks per query row and skips the tiles behind the largest limit of a block of
    128 queries; with split histories a chunk that no row of the block sees yields an empty partial result."""
    from ckv_testlib import make_session
    w = synth.scaled(W[name], **kw)
    d = synth.generate(w)
    vis = _vis_for(w, d, kind, np.random.default_rng(5))
    s = make_session(w, d, split_len=split_len)
    q = to_dev(d["queries"], w.dtype)
    out = s.attend_visible(d["users"], d["q_off"], vis, q)
    torch.cuda.synchronize()
    assert s.stat("kernel") == 3 and s.stat("device_errors") == 0
    if split_len:
        assert s.stat("split_items") > 0
    want = O.attend_variants(w.dtype, w.mode, w.default_scale, w.head_dim, d["pool_K"], d["pool_V"], d["hist_off"],
                             d["idx_K"], d["idx_V"], d["user_K"], d["user_V"], d["q_off"], d["queries"], vis=vis)
    assert_close(out.float().cpu().numpy().astype(np.float64), want, w.dtype, f"{name} {kind}")
    if kind == "all":
        assert torch.equal(out, s.attend(d["users"], d["q_off"], q))
    s.close()


@pytest.mark.parametrize("name", ["cfg4", "cfg5"])
def test_everything_visible_equals_plain_attend(name):
    from ckv_testlib import make_session
    w = VIS_CASES[name]
    d = synth.generate(w)
    s = make_session(w, d, kernel=2, split_len=256)
    q = to_dev(d["queries"], w.dtype)
    a = s.attend(d["users"], d["q_off"], q).clone()
    b = s.attend_visible(d["users"], d["q_off"], _vis_for(w, d, "all", None), q)
    assert torch.equal(a, b)
    s.close()


def test_visible_lengths_with_one_sided_sharing():
    w = synth.scaled(W["cfg5"], n_users=10, hist_len=(1, 400))
    d = synth.generate(w)
    vis = _vis_for(w, d, "random", np.random.default_rng(8))
    s, uk, uv = side_session(w, d, False, True)
    out = s.attend_visible(d["users"], d["q_off"], vis, to_dev(d["queries"], w.dtype))
    torch.cuda.synchronize()
    assert_close(out.float().cpu().numpy().astype(np.float64), oracle_sides(w, d, False, True, uk, uv, vis=vis), w.dtype)
    s.close()
