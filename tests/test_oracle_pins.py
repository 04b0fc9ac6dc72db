"""Pins of the CPU oracle against things other than itself.

Each test names the mistake it would catch.  None needs a GPU.
"""
import math
import os

import numpy as np
import pytest
import torch

import synth
from oracle import ckv_oracle as O
from oracle import ckv_oracle_np as N

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _call(dtype, mode, scale, d, **kw):
    return O.attend(dtype, mode, scale, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"],
                    d["idx_V"], d["user_K"], d["user_V"], d["q_off"], d["queries"], **kw)


def _tiny(dtype="f32", mode="softmax", **kw):
    base = synth.Workload("tiny", 3, 5, 3, 5, 4, (1, 17), 3, mode, dtype, None, 1.0, 1.0, 1234)
    w = synth.scaled(base, **kw)
    return w, synth.generate(w)


def _as_f64(a):
    return synth.bf16_bits_to_f32(a).astype(np.float64) if a.dtype == np.uint16 else a.astype(np.float64)


def _read_fixture(path):
    vals = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=")
        vals[k.strip()] = np.array([float(x) for x in v.split()])
    return vals


# ---------------------------------------------------------------- hand-worked fixture
def _fixture_inputs(golden_dir):
    f = _read_fixture(os.path.join(golden_dir, "hand_worked_two_positions.txt"))
    d = {
        "pool_K": f["pool_K"].reshape(1, 3, 2).astype(np.float32),
        "pool_V": f["pool_V"].reshape(1, 3, 2).astype(np.float32),
        "idx_K": f["idx_K"].reshape(2, 1).astype(np.int32),
        "idx_V": f["idx_V"].reshape(2, 1).astype(np.int32),
        "user_K": f["user_K"].reshape(2, 1, 1).astype(np.float32),
        "user_V": f["user_V"].reshape(2, 1, 1).astype(np.float32),
        "hist_off": np.array([0, 2], dtype=np.int64),
        "q_off": np.array([0, 1], dtype=np.int32),
        "queries": f["query"].reshape(1, 1, 3).astype(np.float32),
    }
    return f, d


def test_hand_worked_example_softmax(golden_dir):
    f, d = _fixture_inputs(golden_dir)
    out = _call("f32", "softmax", float(f["softmax_scale"][0]), d)
    np.testing.assert_allclose(out.reshape(3), f["softmax_out"], atol=1e-12)


def test_hand_worked_example_pointwise(golden_dir):
    f, d = _fixture_inputs(golden_dir)
    out = _call("f32", "silu_over_l", float(f["silu_scale"][0]), d)
    np.testing.assert_allclose(out.reshape(3), f["silu_out"], atol=2e-12)


def test_hand_worked_example_is_sensitive(golden_dir):
    """The fixture separates the plausible mistakes: K/V indices swapped, user part
    placed last, scale dropped, K pool used for V."""
    f, d = _fixture_inputs(golden_dir)
    s = float(f["softmax_scale"][0])
    good = f["softmax_out"]

    def differs(dd, scale=s):
        return np.abs(_call("f32", "softmax", scale, dd).reshape(3) - good).max() > 1e-3

    assert differs({**d, "idx_K": d["idx_V"], "idx_V": d["idx_K"]})
    assert differs({**d, "pool_K": d["pool_V"], "pool_V": d["pool_K"]})
    assert differs({**d, "user_K": d["user_V"], "user_V": d["user_K"]})
    assert differs(d, scale=1.0)
    # user part last instead of first == rotating the query the other way
    assert differs({**d, "queries": np.roll(d["queries"], -1, axis=-1)})


# ---------------------------------------------------------------- two formulations
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("d_user", [0, 1, 3])
def test_fused_definition_equals_materialise_then_attend(dtype, mode, d_user):
    w, d = _tiny(dtype, mode, d_user=d_user)
    a = _call(dtype, mode, 0.9, d)
    b = N.attend(mode, 0.9, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"], d["idx_V"],
                 d["user_K"], d["user_V"], d["q_off"], d["queries"])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def _materialize_loops(d, u):
    """Brute-force Python loops over (position, group, column)."""
    G, m, dg = d["pool_K"].shape
    du = d["user_K"].shape[2]
    p0, p1 = int(d["hist_off"][u]), int(d["hist_off"][u + 1])
    K = np.zeros((p1 - p0, G, du + dg), dtype=d["pool_K"].dtype)
    V = np.zeros_like(K)
    for i in range(p1 - p0):
        for g in range(G):
            for c in range(du):
                K[i, g, c] = d["user_K"][p0 + i, g, c]
                V[i, g, c] = d["user_V"][p0 + i, g, c]
            for c in range(dg):
                K[i, g, du + c] = d["pool_K"][g, d["idx_K"][p0 + i, g], c]
                V[i, g, du + c] = d["pool_V"][g, d["idx_V"][p0 + i, g], c]
    return K, V


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_materialize_is_bitwise_concat_of_pool_rows_and_user_part(dtype):
    w, d = _tiny(dtype)
    for u in range(w.n_users):
        p0, L = int(d["hist_off"][u]), int(d["hist_off"][u + 1] - d["hist_off"][u])
        K, V = O.materialize(dtype, d["pool_K"], d["pool_V"], d["idx_K"], d["idx_V"],
                             d["user_K"], d["user_V"], p0, L)
        Kb, Vb = _materialize_loops(d, u)
        assert K.tobytes() == Kb.tobytes() and V.tobytes() == Vb.tobytes()


# ---------------------------------------------------------------- library routine
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_softmax_branch_equals_torch_sdpa_on_materialised_kv(dtype):
    w, d = _tiny(dtype, "softmax", n_users=3, hist_len=(2, 33), n_queries=4)
    scale = 0.37
    out = _call(dtype, "softmax", scale, d)
    for u in range(w.n_users):
        K, V = _materialize_loops(d, u)
        q0, q1 = int(d["q_off"][u]), int(d["q_off"][u + 1])
        q = torch.from_numpy(_as_f64(d["queries"][q0:q1])).permute(1, 0, 2)   # [G, M, d]
        k = torch.from_numpy(_as_f64(K)).permute(1, 0, 2)
        v = torch.from_numpy(_as_f64(V)).permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=scale)
        np.testing.assert_allclose(out[q0:q1], ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_pointwise_branch_equals_scalar_restatement():
    w, d = _tiny("f32", "silu_over_l", n_users=2, hist_len=(1, 9), n_queries=2)
    out = _call("f32", "silu_over_l", 1.3, d)
    for u in range(w.n_users):
        K, V = _materialize_loops(d, u)
        L = K.shape[0]
        for r in range(int(d["q_off"][u]), int(d["q_off"][u + 1])):
            for g in range(w.n_groups):
                o = [0.0] * w.head_dim
                for i in range(L):
                    s = 1.3 * sum(float(d["queries"][r, g, c]) * float(K[i, g, c]) for c in range(w.head_dim))
                    wgt = s * (1.0 / (1.0 + math.exp(-s))) / L
                    for c in range(w.head_dim):
                        o[c] += wgt * float(V[i, g, c])
                np.testing.assert_allclose(out[r, g], o, rtol=1e-11, atol=1e-13)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_one_entry_pool_without_user_part_returns_the_value_row(dtype):
    """d_user = 0 and m = 1: every K row is P_k[0], so softmax weights are uniform and
    o = P_v[0] exactly, for every query and every history length."""
    w, d = _tiny(dtype, "softmax", d_user=0, n_entries=1, d_shared=8)
    out = _call(dtype, "softmax", 0.5, d)
    want = _as_f64(d["pool_V"])[:, 0, :]                      # [G, d]
    np.testing.assert_allclose(out, np.broadcast_to(want, out.shape), rtol=1e-13, atol=1e-15)


def test_one_entry_pool_pointwise_closed_form():
    w, d = _tiny("f32", "silu_over_l", d_user=0, n_entries=1, d_shared=8)
    out = _call("f32", "silu_over_l", 0.8, d)
    pk, pv, q = _as_f64(d["pool_K"])[:, 0], _as_f64(d["pool_V"])[:, 0], _as_f64(d["queries"])
    s = 0.8 * np.einsum("rgc,gc->rg", q, pk)
    want = (s / (1 + np.exp(-s)))[..., None] * pv[None]
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-14)


def test_equal_indices_and_zero_user_part():
    """All indices = j and all user parts zero: o = [0 .. 0 | P_v[j]]."""
    w, d = _tiny("f32", "softmax")
    j = 3
    d["idx_K"][:] = 1
    d["idx_V"][:] = j
    d["user_K"][:] = 0
    d["user_V"][:] = 0
    out = _call("f32", "softmax", 1.0, d)
    want = np.concatenate([np.zeros((w.n_groups, w.d_user)), _as_f64(d["pool_V"])[:, j]], axis=1)
    np.testing.assert_allclose(out, np.broadcast_to(want, out.shape), rtol=1e-13, atol=1e-15)


def test_single_position_history_returns_its_value_row():
    w, d = _tiny("bf16", "softmax", hist_len=(1, 1))
    out = _call("bf16", "softmax", 2.0, d)
    for u in range(w.n_users):
        K, V = _materialize_loops(d, u)
        for r in range(int(d["q_off"][u]), int(d["q_off"][u + 1])):
            np.testing.assert_allclose(out[r], _as_f64(V[0]), rtol=0, atol=0)


def test_large_scale_selects_the_argmax_position():
    w, d = _tiny("f32", "softmax", hist_len=(5, 12))
    out = _call("f32", "softmax", 1e4, d)
    for u in range(w.n_users):
        K, V = _materialize_loops(d, u)
        for r in range(int(d["q_off"][u]), int(d["q_off"][u + 1])):
            for g in range(w.n_groups):
                s = _as_f64(K[:, g]) @ _as_f64(d["queries"][r, g])
                np.testing.assert_allclose(out[r, g], _as_f64(V[int(np.argmax(s)), g]), atol=1e-9)


def test_empty_history_and_empty_query_list():
    w, d = _tiny("f32", "softmax", n_users=3, hist_len=(4, 4), n_queries=2)
    # user 1 gets an empty history, user 2 no queries
    keep = np.r_[0:4, 8:12]
    d2 = dict(d)
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d2[k] = np.ascontiguousarray(d[k][keep])
    d2["hist_off"] = np.array([0, 4, 4, 8], dtype=np.int64)
    d2["q_off"] = np.array([0, 2, 4, 4], dtype=np.int32)
    d2["queries"] = np.ascontiguousarray(d["queries"][:4])
    for mode in ("softmax", "silu_over_l"):
        out = _call("f32", mode, 1.0, d2)
        assert out.shape[0] == 4
        assert np.all(out[2:4] == 0.0)
        assert np.abs(out[0:2]).max() > 0


# ---------------------------------------------------------------- invariants
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
def test_permuting_positions_leaves_output_unchanged(mode):
    w, d = _tiny("f32", mode, n_users=1, hist_len=(13, 13))
    a = _call("f32", mode, 0.6, d)
    perm = np.random.default_rng(0).permutation(13)
    d2 = dict(d)
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d2[k] = np.ascontiguousarray(d[k][perm])
    b = _call("f32", mode, 0.6, d2)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
def test_output_is_linear_in_values(mode):
    w, d = _tiny("f32", mode)
    a = _call("f32", mode, 0.6, d)
    d2 = {**d, "pool_V": d["pool_V"] * 2, "user_V": d["user_V"] * 2}
    b = _call("f32", mode, 0.6, d2)
    np.testing.assert_allclose(b, 2 * a, rtol=1e-13, atol=0)


def test_softmax_is_shift_invariant_in_the_scores():
    """Adding the same constant to every <q, K[i]> (here: a constant user-K column met
    by a non-zero query entry) must not change a softmax output."""
    w, d = _tiny("f32", "softmax", d_user=1)
    d["user_K"][:] = 0.0
    a = _call("f32", "softmax", 1.0, d)
    d2 = {**d, "user_K": np.full_like(d["user_K"], 7.0)}
    b = _call("f32", "softmax", 1.0, d2)
    np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-12)


def test_key_indices_do_not_touch_values_and_vice_versa():
    """Changing I_v for one position changes only that position's V row; with a one-hot
    softmax (large scale) on another position the output must stay the same."""
    w, d = _tiny("f32", "softmax", n_users=1, hist_len=(6, 6), n_queries=1)
    a = _call("f32", "softmax", 1e4, d)
    K, V = _materialize_loops(d, 0)
    for g in range(w.n_groups):
        win = int(np.argmax(_as_f64(K[:, g]) @ _as_f64(d["queries"][0, g])))
        other = (win + 1) % 6
        d["idx_V"][other, g] = (d["idx_V"][other, g] + 1) % w.n_entries
    b = _call("f32", "softmax", 1e4, d)
    np.testing.assert_allclose(a, b, atol=1e-9)


def test_selection_returns_the_same_rows_as_the_full_run():
    w, d = _tiny("bf16", "softmax", n_users=6)
    full = _call("bf16", "softmax", 0.5, d)
    sel = [4, 1, 5]
    part = _call("bf16", "softmax", 0.5, d, sel=sel)
    rows = np.concatenate([np.arange(d["q_off"][u], d["q_off"][u + 1]) for u in sel])
    assert np.array_equal(part, full[rows])


def test_thread_count_does_not_change_results():
    w, d = _tiny("f32", "softmax", n_users=9)
    assert np.array_equal(_call("f32", "softmax", 0.5, d, n_threads=1),
                          _call("f32", "softmax", 0.5, d, n_threads=4))


def test_out_of_range_index_is_an_error():
    w, d = _tiny("f32", "softmax")
    d["idx_V"][2, 1] = w.n_entries
    with pytest.raises(IndexError):
        _call("f32", "softmax", 1.0, d)
    d["idx_V"][2, 1] = -1
    with pytest.raises(IndexError):
        O.materialize("f32", d["pool_K"], d["pool_V"], d["idx_K"], d["idx_V"], d["user_K"],
                      d["user_V"], 0, int(d["hist_off"][-1]))


# ---------------------------------------------------------------- storage accounting
def test_compression_rate_reproduces_table_1(golden_dir):
    for line in open(os.path.join(golden_dir, "table1_compression_rates.txt")):
        if line.startswith("#") or not line.strip():
            continue
        d_u, cr = line.split()
        assert round(O.compression_rate(256, int(d_u)), 3) == float(cr)
