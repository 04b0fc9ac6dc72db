"""Pins of the oracle's variants (a shared width per side, a visible length per query) against things
other than itself: hand-worked values, the base oracle on the common domain, a library attention routine
with a boolean mask, closed forms, brute-force loops.  Each test names the mistake it would catch.  No GPU."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import ckv_oracle as O
from oracle import ckv_oracle_np as N
from test_oracle_pins import _as_f64, _fixture_inputs, _read_fixture, _tiny


def _variants(dtype, mode, scale, d, d_a, share_k=True, share_v=True, vis=None, full_K=None, full_V=None, **kw):
    return O.attend_variants(dtype, mode, scale, d_a,
                             d["pool_K"] if share_k else None, d["pool_V"] if share_v else None,
                             d["hist_off"], d["idx_K"], d["idx_V"],
                             d["user_K"] if share_k else full_K, d["user_V"] if share_v else full_V,
                             d["q_off"], d["queries"], vis=vis, **kw)


def _full_rows(d, side):
    """Full-width rows of one side for all positions, by Python loops (user part first, then the pool row)."""
    pool, idx, user = d["pool_" + side], d["idx_" + side], d["user_" + side]
    P, G, du = user.shape
    dg = pool.shape[2]
    out = np.zeros((P, G, du + dg), dtype=pool.dtype)
    for i in range(P):
        for g in range(G):
            out[i, g, :du] = user[i, g]
            out[i, g, du:] = pool[g, idx[i, g]]
    return out


# ---------------------------------------------------------------- hand-worked values
def test_hand_worked_visible_lengths(golden_dir):
    """A mask off by one, a divisor that follows the visible count, or a mask applied to the wrong row."""
    f, d = _fixture_inputs(golden_dir)
    v = _read_fixture(os.path.join(golden_dir, "hand_worked_variants.txt"))
    d = {**d, "queries": np.concatenate([d["queries"], d["queries"]]), "q_off": np.array([0, 2], dtype=np.int32)}
    vis = v["vis"].astype(np.int32)
    out = _variants("f32", "softmax", float(f["softmax_scale"][0]), d, 3, vis=vis)
    np.testing.assert_allclose(out.reshape(6), v["softmax_out_vis"], atol=1e-12)
    out = _variants("f32", "silu_over_l", float(f["silu_scale"][0]), d, 3, vis=vis)
    np.testing.assert_allclose(out.reshape(6), v["silu_out_vis"], atol=2e-12)


@pytest.mark.parametrize("mode,key", [("softmax", "softmax"), ("silu_over_l", "silu")])
def test_hand_worked_one_sided_sharing(golden_dir, mode, key):
    """Full-width rows read with the wrong width, pool part added to an unshared side, sides swapped."""
    f, d = _fixture_inputs(golden_dir)
    v = _read_fixture(os.path.join(golden_dir, "hand_worked_variants.txt"))
    fk = v["full_K"].reshape(2, 1, 3).astype(np.float32)
    fv = v["full_V"].reshape(2, 1, 3).astype(np.float32)
    scale = float(f[key + "_scale"][0])
    want = f[key + "_out"]
    np.testing.assert_allclose(_variants("f32", mode, scale, d, 3, share_v=False, full_V=fv).reshape(3), want, atol=2e-12)
    np.testing.assert_allclose(_variants("f32", mode, scale, d, 3, share_k=False, full_K=fk).reshape(3), want, atol=2e-12)
    np.testing.assert_allclose(
        _variants("f32", mode, scale, d, 3, share_k=False, share_v=False, full_K=fk, full_V=fv).reshape(3), want, atol=2e-12)
    # the fixture notices full-width K and V handed in the wrong way round
    wrong = _variants("f32", mode, scale, d, 3, share_k=False, share_v=False, full_K=fv, full_V=fk).reshape(3)
    assert np.abs(wrong - want).max() > 1e-3


# ---------------------------------------------------------------- the base oracle on the common domain
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
def test_variants_reduce_to_the_base_oracle(dtype, mode):
    """Both sides shared with one width and no visible lengths is the base path: same bits."""
    w, d = _tiny(dtype, mode)
    base = O.attend(dtype, mode, 0.7, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"], d["idx_V"],
                    d["user_K"], d["user_V"], d["q_off"], d["queries"])
    assert np.array_equal(_variants(dtype, mode, 0.7, d, w.head_dim), base)
    lens = np.diff(d["hist_off"])
    vis_all = np.repeat(lens, np.diff(d["q_off"])).astype(np.int32)
    assert np.array_equal(_variants(dtype, mode, 0.7, d, w.head_dim, vis=vis_all), base)
    sel = [2, 0]
    assert np.array_equal(_variants(dtype, mode, 0.7, d, w.head_dim, sel=sel),
                          O.attend(dtype, mode, 0.7, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"], d["idx_V"],
                                   d["user_K"], d["user_V"], d["q_off"], d["queries"], sel=sel))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("share", [(True, False), (False, True), (False, False)])
def test_one_sided_sharing_equals_base_oracle_on_rebuilt_rows(dtype, mode, share):
    """A side that is not shared, fed with the rows the shared form would rebuild (loop-built), gives the bits
    of the shared form: catches a wrong row stride or a pool term left in."""
    w, d = _tiny(dtype, mode)
    base = O.attend(dtype, mode, 1.1, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"], d["idx_V"],
                    d["user_K"], d["user_V"], d["q_off"], d["queries"])
    got = _variants(dtype, mode, 1.1, d, w.head_dim, share_k=share[0], share_v=share[1],
                    full_K=_full_rows(d, "K"), full_V=_full_rows(d, "V"))
    assert np.array_equal(got, base)


def test_sides_may_have_different_shared_widths():
    """K shared with d_g = 5 (d_u = 3), V shared with d_g = 2 (d_u = 6): against the numpy formulation."""
    w, d = _tiny("f32", "softmax")
    rng = np.random.default_rng(3)
    G, m = w.n_groups, w.n_entries
    P = int(d["hist_off"][-1])
    d2 = {**d, "pool_V": rng.standard_normal((G, m, 2)).astype(np.float32),
          "user_V": rng.standard_normal((P, G, 6)).astype(np.float32)}
    a = _variants("f32", "softmax", 0.8, d2, 8)
    b = N.attend_variants("softmax", 0.8, 8, d2["pool_K"], d2["pool_V"], d2["hist_off"], d2["idx_K"], d2["idx_V"],
                          d2["user_K"], d2["user_V"], d2["q_off"], d2["queries"])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- a library routine with a mask
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_visible_lengths_equal_masked_library_attention(dtype):
    """Softmax branch with visible lengths == torch SDPA (fp64) with a boolean mask on loop-built K, V."""
    w, d = _tiny(dtype, "softmax", n_queries=5, hist_len=(3, 17))
    rng = np.random.default_rng(5)
    lens = np.diff(d["hist_off"])
    vis = np.concatenate([rng.integers(1, L + 1, size=w.n_queries) for L in lens]).astype(np.int32)
    got = _variants(dtype, "softmax", 0.6, d, w.head_dim, vis=vis)
    K, V = _as_f64(_full_rows(d, "K")), _as_f64(_full_rows(d, "V"))
    q = _as_f64(d["queries"])
    for u in range(w.n_users):
        p0, p1 = int(d["hist_off"][u]), int(d["hist_off"][u + 1])
        q0, q1 = int(d["q_off"][u]), int(d["q_off"][u + 1])
        mask = torch.from_numpy(np.arange(p1 - p0)[None, :] < vis[q0:q1, None])
        for g in range(w.n_groups):
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(q[q0:q1, g])[None], torch.from_numpy(K[p0:p1, g])[None],
                torch.from_numpy(V[p0:p1, g])[None], attn_mask=mask[None], scale=0.6)[0].numpy()
            np.testing.assert_allclose(got[q0:q1, g], ref, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("share", [(True, True), (True, False), (False, True)])
def test_two_formulations_agree_on_variants(mode, share):
    w, d = _tiny("bf16", mode, n_queries=4)
    rng = np.random.default_rng(9)
    lens = np.diff(d["hist_off"])
    vis = np.concatenate([rng.integers(0, L + 1, size=w.n_queries) for L in lens]).astype(np.int32)
    fk, fv = _full_rows(d, "K"), _full_rows(d, "V")
    a = _variants("bf16", mode, 0.9, d, w.head_dim, share_k=share[0], share_v=share[1], vis=vis, full_K=fk, full_V=fv)
    b = N.attend_variants(mode, 0.9, w.head_dim, d["pool_K"] if share[0] else None, d["pool_V"] if share[1] else None,
                          d["hist_off"], d["idx_K"], d["idx_V"], d["user_K"] if share[0] else fk,
                          d["user_V"] if share[1] else fv, d["q_off"], d["queries"], vis=vis)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- closed forms and invariants
def test_visible_length_closed_forms():
    """vis = 0: zero row.  vis = 1, softmax: the first value row.  Causal self-attention: the last query sees
    everything and equals the unmasked result; what lies behind a query's horizon cannot change its output."""
    w, d = _tiny("f32", "softmax", n_users=1, hist_len=(9, 9), n_queries=9)
    L = 9
    V = _as_f64(_full_rows(d, "V"))
    vis = np.arange(1, L + 1, dtype=np.int32)                     # causal: query i sees positions 0..i
    out = _variants("f32", "softmax", 1.3, d, w.head_dim, vis=vis)
    np.testing.assert_allclose(out[0], V[0], atol=1e-12)
    full = _variants("f32", "softmax", 1.3, d, w.head_dim)
    np.testing.assert_allclose(out[L - 1], full[L - 1], atol=1e-14)
    zero = _variants("f32", "softmax", 1.3, d, w.head_dim, vis=np.zeros(L, dtype=np.int32))
    assert not zero.any()
    # change everything behind position 4: queries 0..4 keep their outputs, query 5 on moves
    d2 = {**d, "idx_K": d["idx_K"].copy(), "user_V": d["user_V"].copy()}
    d2["idx_K"][5:] = (d2["idx_K"][5:] + 1) % w.n_entries
    d2["user_V"][5:] += 1.0
    out2 = _variants("f32", "softmax", 1.3, d2, w.head_dim, vis=vis)
    assert np.array_equal(out2[:5], out[:5]) and np.abs(out2[5:] - out[5:]).max() > 1e-3


def test_pointwise_divisor_is_the_history_length():
    """SiLU mode with a visible length: the sum stops at the horizon, the divisor stays L_u."""
    w, d = _tiny("f32", "silu_over_l", n_users=1, hist_len=(6, 6), n_queries=1)
    K, V = _as_f64(_full_rows(d, "K")), _as_f64(_full_rows(d, "V"))
    q = _as_f64(d["queries"])
    got = _variants("f32", "silu_over_l", 0.5, d, w.head_dim, vis=np.array([4], dtype=np.int32))
    for g in range(w.n_groups):
        o = np.zeros(w.head_dim)
        for i in range(4):
            s = 0.5 * float(q[0, g] @ K[i, g])
            o += s / (1.0 + np.exp(-s)) * V[i, g]
        np.testing.assert_allclose(got[0, g], o / 6.0, rtol=1e-12, atol=1e-14)


def test_bad_visible_length_and_index_are_reported():
    w, d = _tiny("f32", "softmax", n_users=1, hist_len=(4, 4), n_queries=1)
    with pytest.raises(ValueError):
        _variants("f32", "softmax", 1.0, d, w.head_dim, vis=np.array([5], dtype=np.int32))
    bad = {**d, "idx_V": d["idx_V"].copy()}
    bad["idx_V"][0, 0] = w.n_entries
    with pytest.raises(IndexError):
        _variants("f32", "softmax", 1.0, bad, w.head_dim)
    # ... but the indices of a side that is not shared are never read
    _variants("f32", "softmax", 1.0, bad, w.head_dim, share_v=False, full_V=_full_rows(d, "V"))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_materialize_side_is_bit_exact(dtype):
    w, d = _tiny(dtype)
    for side in ("K", "V"):
        rows = _full_rows(d, side)
        for u in range(w.n_users):
            p0, L = int(d["hist_off"][u]), int(d["hist_off"][u + 1] - d["hist_off"][u])
            got = O.materialize_side(dtype, w.head_dim, d["pool_" + side], d["idx_" + side], d["user_" + side], p0, L)
            assert np.array_equal(got, rows[p0:p0 + L])
            assert np.array_equal(O.materialize_side(dtype, w.head_dim, None, None, rows, p0, L), rows[p0:p0 + L])
