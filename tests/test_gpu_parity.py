"""CUDA path vs CPU oracle, through the C ABI, on seeded synthetic inputs."""
import numpy as np
import pytest
import torch

import synth
from ckv_testlib import assert_close, gpu_attend, make_session, oracle_attend, to_dev
from oracle import ckv_oracle as O

pytestmark = pytest.mark.gpu

W = synth.WORKLOADS

# scaled-down copies of the five benchmark workloads: several tiles and a ragged tail each
SMALL = {
    "cfg1": synth.scaled(W["cfg1"], n_users=64),                                        # full size
    "cfg2": synth.scaled(W["cfg2"], n_users=6, hist_len=(1024, 1024)),
    "cfg2_ragged": synth.scaled(W["cfg2"], n_users=9, hist_len=(1, 700), n_queries=37),
    "cfg3": synth.scaled(W["cfg3"], n_users=3, hist_len=(1100, 1100)),
    "cfg3_ragged": synth.scaled(W["cfg3"], n_users=7, hist_len=(3, 333), n_queries=50),
    "cfg4": synth.scaled(W["cfg4"], n_users=12, hist_len=(1000, 9000)),
    "cfg5": synth.scaled(W["cfg5"], n_users=300, hist_len=(512, 512)),
    "cfg5_ragged": synth.scaled(W["cfg5"], n_users=80, hist_len=(1, 130)),
}


@pytest.mark.parametrize("name", sorted(SMALL))
def test_attend_matches_oracle(name):
    w = SMALL[name]
    d = synth.generate(w)
    got = gpu_attend(w, d)
    want = oracle_attend(w, d)
    assert_close(got, want, w.dtype, name)


@pytest.mark.parametrize("kernel", [1, 2, 3])
@pytest.mark.parametrize("name", ["cfg2", "cfg2_ragged", "cfg3", "cfg3_ragged", "cfg5_ragged"])
def test_every_kernel_family_matches_oracle(name, kernel):
    """1 = CUDA cores, 2 = warp-level MMA, 3 = tcgen05; all must agree with the oracle."""
    w = SMALL[name]
    d = synth.generate(w)
    s = make_session(w, d, kernel=kernel)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == kernel
    assert s.stat("device_errors") == 0
    s.close()
    assert_close(got, oracle_attend(w, d), w.dtype, f"{name} kernel {kernel}")


@pytest.mark.parametrize("kernel,loader", [(2, 1), (2, 2), (3, 0)])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("d_user", [0, 1, 2, 4, 8])
def test_tensor_core_kernels_user_widths_and_sharp_softmax(kernel, loader, mode, d_user):
    w = synth.Workload("tc", 3, 32 - d_user, d_user, 300, 5, (1, 700), 70, mode, "bf16", 1.1, 1 / 32, 1 / 32, 21)
    d = synth.generate(w)
    scale = 8.0 / np.sqrt(32) if mode == "softmax" else 1.0
    s = make_session(w, d, scale=scale, kernel=kernel, split_len=256, mma_loader=loader)
    got = gpu_attend(w, d, session=s)
    assert s.stat("split_items") > 0 and s.stat("device_errors") == 0
    s.close()
    assert_close(got, oracle_attend(w, d, scale=scale), "bf16", f"d_user={d_user}")


@pytest.mark.parametrize("name", ["cfg4", "cfg5", "cfg5_ragged", "cfg2_ragged", "cfg3_ragged"])
def test_warp_mma_kernel_loaders_agree_bit_for_bit(name):
    """The staging ring is filled by cp.async copies (loader 1) or TMA row gathers (loader 2); everything
    after that is the same code, so the outputs must be the same bits.  Loader 0 is the default (cp.async)."""
    w = SMALL[name]
    d = synth.generate(w)
    outs = {}
    for loader in (1, 2, 0):
        s = make_session(w, d, kernel=2, mma_loader=loader)
        outs[loader] = gpu_attend(w, d, session=s)
        again = gpu_attend(w, d, session=s)
        assert s.stat("kernel") == 2 and s.stat("device_errors") == 0
        assert s.stat("mma_loader") == (loader or 1)
        s.close()
        assert np.array_equal(outs[loader], again)
    assert np.array_equal(outs[1], outs[2]) and np.array_equal(outs[0], outs[1])
    assert_close(outs[2], oracle_attend(w, d), w.dtype, name)


@pytest.mark.parametrize("loader", [1, 2])
@pytest.mark.parametrize("n_queries", [1, 7, 20])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("d_user", [0, 1, 2, 4, 8])
def test_warp_mma_kernel_head_dim_64(n_queries, mode, d_user, loader):
    """64-wide heads run on the warp-level tensor-core kernel from one query per user on."""
    w = synth.Workload("tc64", 3, 64 - d_user, d_user, 500, 6, (1, 900), n_queries, mode, "bf16", 1.1, 1 / 32, 1 / 32, 22)
    d = synth.generate(w)
    scale = 8.0 / np.sqrt(64) if mode == "softmax" else 1.0
    s = make_session(w, d, scale=scale, split_len=256, mma_loader=loader, kernel=2)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 2 and s.stat("split_items") > 0 and s.stat("device_errors") == 0
    s.close()
    assert_close(got, oracle_attend(w, d, scale=scale), "bf16", f"d_user={d_user} M={n_queries}")


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("n_queries", [70, 150])
def test_persistent_tcgen05_kernel_many_units_per_sm(mode, n_queries):
    """More work units than SMs, one to six tiles each: every buffer of the kernel is reused
    across unit boundaries (tile stages, Q buffers, both accumulators)."""
    w = synth.Workload("many", 8, 30, 2, 500, 110, (1, 700), n_queries, mode, "bf16", 1.1, 1 / 32, 1 / 32, 41)
    d = synth.generate(w)
    s = make_session(w, d, kernel=3)
    got = gpu_attend(w, d, session=s)
    again = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 3 and s.stat("device_errors") == 0
    s.close()
    assert np.array_equal(got, again), "run-to-run bitwise reproducibility"
    assert_close(got, oracle_attend(w, d), "bf16", f"{mode} M={n_queries}")


def test_growing_maximum_triggers_rescale_in_tcgen05_kernel():
    """Keys sorted by increasing score: the scores climb by about 115 log2 units along the
    history, so every kernel has to move its running / reference maximum several times.
    Pool and user values keep the workloads' scale (variance 1/32): with unit-variance V the
    bf16 rounding of the weights alone leaves well under 1e-3 of margin to the tolerance."""
    w = synth.Workload("grow", 1, 30, 2, 512, 2, (1024, 1024), 128, "softmax", "bf16", None, 1 / 32, 1 / 32, 33)
    d = synth.generate(w)
    # history = pool rows in an order of growing norm along one direction: scale the user part
    ramp = np.linspace(-40.0, 40.0, 1024, dtype=np.float32)
    for u in range(2):
        d["user_K"][u * 1024:(u + 1) * 1024, 0, 0] = synth.f32_to_bf16_bits(ramp)
    d["queries"][:, 0, 0] = synth.f32_to_bf16_bits(np.full(d["queries"].shape[0], 1.0, np.float32))
    for kernel in (2, 3):
        s = make_session(w, d, scale=1.0, kernel=kernel)
        got = gpu_attend(w, d, session=s)
        assert s.stat("device_errors") == 0
        s.close()
        assert_close(got, oracle_attend(w, d, scale=1.0), "bf16", f"kernel {kernel}")


@pytest.mark.parametrize("name", ["cfg1", "cfg2_ragged", "cfg4", "cfg5_ragged"])
@pytest.mark.parametrize("scale_mul", [1.0, 4.0])
def test_attend_sharper_softmax(name, scale_mul):
    """The default logits are nearly flat (std ~0.2); a larger scale makes the softmax matter."""
    w = synth.scaled(SMALL[name], n_users=min(SMALL[name].n_users, 8))
    d = synth.generate(w)
    scale = scale_mul * 4.0 / np.sqrt(w.head_dim)
    assert_close(gpu_attend(w, d, scale=scale), oracle_attend(w, d, scale=scale), w.dtype, name)


@pytest.mark.parametrize("name", ["cfg1", "cfg2_ragged", "cfg3_ragged", "cfg4"])
def test_materialize_is_bit_exact(name):
    w = synth.scaled(SMALL[name], n_users=min(SMALL[name].n_users, 5))
    d = synth.generate(w)
    s = make_session(w, d)
    for u in range(w.n_users):
        K, V = s.materialize(int(d["users"][u]))
        p0, L = int(d["hist_off"][u]), int(d["hist_off"][u + 1] - d["hist_off"][u])
        Ko, Vo = O.materialize(w.dtype, d["pool_K"], d["pool_V"], d["idx_K"], d["idx_V"], d["user_K"],
                               d["user_V"], p0, L)
        view = torch.int16 if w.dtype == "bf16" else torch.int32
        npv = np.int16 if w.dtype == "bf16" else np.int32
        assert np.array_equal(K.view(view).cpu().numpy(), Ko.view(npv))
        assert np.array_equal(V.view(view).cpu().numpy(), Vo.view(npv))
    s.close()


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("split_len", [8, 64, 1000, 100000])
def test_split_count_does_not_change_the_result(mode, split_len):
    w = synth.scaled(W["cfg4"], n_users=6, hist_len=(1, 1500), n_queries=3, mode=mode)
    d = synth.generate(w)
    want = oracle_attend(w, d)
    s = make_session(w, d, split_len=split_len)
    a = gpu_attend(w, d, session=s)
    b = gpu_attend(w, d, session=s)
    assert np.array_equal(a, b), "run-to-run bitwise reproducibility"
    if split_len >= 100000:
        assert s.stat("split_items") == 0
    else:
        assert s.stat("split_items") > 0
    s.close()
    assert_close(a, want, w.dtype, f"split_len={split_len}")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("head", [(16, 0), (14, 2), (31, 1), (28, 4), (56, 8), (120, 8), (10, 22)])
@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
def test_head_shapes(dtype, head, mode):
    dg, du = head
    w = synth.Workload("shape", 3, dg, du, 97, 5, (1, 90), 5, mode, dtype, None, 1.0 / (dg + du),
                       1.0 / (dg + du), 77)
    d = synth.generate(w)
    assert_close(gpu_attend(w, d), oracle_attend(w, d), dtype, f"{head}")


def test_degenerate_one_entry_pool_and_no_user_part():
    w = synth.Workload("deg", 2, 32, 0, 1, 4, (1, 300), 2, "softmax", "bf16", None, 1 / 32, 1 / 32, 5)
    d = synth.generate(w)
    got = gpu_attend(w, d, out_dtype="f32")
    pv = synth.bf16_bits_to_f32(d["pool_V"])[:, 0].astype(np.float64)
    assert np.abs(got - pv[None]).max() <= 1e-6 * np.abs(pv).max() + 1e-7
    assert_close(got, oracle_attend(w, d), "bf16")


def test_wide_pool_uses_32_bit_indices():
    w = synth.Workload("wide", 1, 30, 2, 70000, 3, (50, 400), 2, "softmax", "bf16", None, 1 / 32, 1 / 32, 6)
    d = synth.generate(w)
    d["idx_K"][0, 0] = 69999
    d["idx_V"][1, 0] = 65536
    assert_close(gpu_attend(w, d), oracle_attend(w, d), "bf16")


@pytest.mark.parametrize("kernel", [1, 2, 3])
def test_empty_history_empty_query_list_and_repeated_user(kernel):
    w = synth.Workload("edge", 2, 30, 2, 64, 4, (40, 40), 3, "softmax", "bf16", None, 1 / 32, 1 / 32, 8)
    d = synth.generate(w)
    # user 1: empty history; request list: [u0, u1, u2 (no queries), u3, u0 again]
    keep = np.r_[0:40, 80:160]
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d[k] = np.ascontiguousarray(d[k][keep])
    d["hist_off"] = np.array([0, 40, 40, 80, 120], dtype=np.int64)
    s = make_session(w, d, kernel=kernel)
    req_users = d["users"][[0, 1, 2, 3, 0]]
    q_off = np.array([0, 3, 6, 6, 9, 12], dtype=np.int32)
    q = d["queries"]
    out = s.attend(req_users, q_off, to_dev(q, "bf16")).float().cpu().numpy().astype(np.float64)
    s.close()
    # oracle on the equivalent explicit layout
    o_all = O.attend("bf16", "softmax", w.default_scale, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"],
                     d["idx_V"], d["user_K"], d["user_V"], np.array([0, 3, 6, 6, 9]), d["queries"][:9])
    assert np.all(out[3:6] == 0.0)                       # empty history -> zero rows
    assert_close(out[0:3], o_all[0:3], "bf16")
    assert_close(out[6:9], o_all[6:9], "bf16")
    # the repeated user sees queries 9..11: compare against the oracle fed with those rows
    d2 = dict(d, queries=np.ascontiguousarray(d["queries"][9:12]))
    o_rep = O.attend("bf16", "softmax", w.default_scale, d["pool_K"], d["pool_V"], d["hist_off"], d["idx_K"],
                     d["idx_V"], d["user_K"], d["user_V"], np.array([0, 3, 3, 3, 3]), d2["queries"])
    assert_close(out[9:12], o_rep, "bf16")


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("head", [(64, 0), (63, 1), (62, 2), (60, 4), (56, 8), (28, 4), (29, 3)])
def test_pool_side_factorisation_matches_oracle(mode, head):
    """One query per user: score table T = P_k q and weight histogram w replace the row gathers (kernel 4)."""
    dg, du = head
    w = synth.Workload("fact", 3, dg, du, 333, 21, (1, 700), 1, mode, "bf16", 1.1, 1.0 / (dg + du), 1.0 / (dg + du), 31)
    d = synth.generate(w)
    scale = 8.0 / np.sqrt(dg + du) if mode == "softmax" else 1.0
    s = make_session(w, d, scale=scale, kernel=4)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 4 and s.stat("launches") == 3 and s.stat("split_items") == 0
    s.close()
    want = oracle_attend(w, d, scale=scale)
    assert_close(got, want, "bf16", f"{head} {mode}")
    # the gathering tensor-core kernel on the same inputs: both within tolerance of the oracle, and of each other
    other = gpu_attend(w, d, scale=scale, kernel=2)
    assert np.abs(got - other).max() <= 2.0 ** -7 * np.abs(want).max()


def test_pool_side_factorisation_is_chosen_when_it_pays_and_handles_edge_requests():
    import paper_2601_19178_b200 as ckv
    # one wave of (user, group) pairs with histories long against the pool: chosen by default
    w = synth.Workload("fact_long", 4, 60, 4, 512, 37, (1500, 3000), 1, "softmax", "bf16", None, 1 / 64, 1 / 64, 32)
    d = synth.generate(w)
    s = make_session(w, d)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 4
    assert_close(got, oracle_attend(w, d), "bf16", "auto")
    # a handful of pairs cannot fill the SMs with one CTA per pair: the gathering kernel stays
    few = s.attend(d["users"][:3], d["q_off"][:4], to_dev(d["queries"][:3], "bf16")).float().cpu().numpy().astype(np.float64)
    assert s.stat("kernel") == 2
    assert_close(few, got[:3], "bf16", "few pairs")
    # forced: request list with an empty query list and a repeated user: [u0, u1 (no query), u2, u0]
    s.set_option("kernel", 4)
    req = d["users"][[0, 1, 2, 0]]
    q_off = np.array([0, 1, 1, 2, 3], dtype=np.int32)
    q = to_dev(d["queries"][[0, 2, 0]], "bf16")
    out = s.attend(req, q_off, q).float().cpu().numpy().astype(np.float64)
    assert s.stat("kernel") == 4
    assert_close(out[0], got[0], "bf16")
    assert_close(out[1], got[2], "bf16")
    assert_close(out[2], got[0], "bf16")
    # more than one query for a user: the family cannot take it
    with pytest.raises(ckv.CkvError) as e:
        s.attend(d["users"][:2], np.array([0, 2, 3], dtype=np.int32), to_dev(d["queries"][:3], "bf16"))
    assert e.value.status == ckv.CKV_ERR_UNSUPPORTED
    s.close()
    # many pairs, but short histories against a large pool: the gathering kernel stays
    w2 = synth.Workload("fact_short", 4, 60, 4, 4096, 40, (10, 200), 1, "softmax", "bf16", None, 1 / 64, 1 / 64, 33)
    d2 = synth.generate(w2)
    s2 = make_session(w2, d2)
    assert_close(gpu_attend(w2, d2, session=s2), oracle_attend(w2, d2), "bf16", "short")
    assert s2.stat("kernel") == 2
    s2.close()


def test_pool_side_factorisation_empty_history_gives_zero_rows():
    w = synth.Workload("fact_empty", 2, 30, 2, 64, 3, (40, 40), 1, "softmax", "bf16", None, 1 / 32, 1 / 32, 8)
    d = synth.generate(w)
    keep = np.r_[0:40, 80:120]
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d[k] = np.ascontiguousarray(d[k][keep])
    d["hist_off"] = np.array([0, 40, 40, 80], dtype=np.int64)
    s = make_session(w, d, kernel=4)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 4
    s.close()
    assert np.all(got[1] == 0.0)
    assert_close(got, oracle_attend(w, d), "bf16", "empty history")


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4", "cfg5"])
def test_full_size_workloads_on_sampled_users(name):
    """The benchmark workloads at full size, default options (the launch configuration bench.py times):
    first, last, longest, shortest and two random users against the oracle."""
    w = W[name]
    d = synth.generate(w)
    s = make_session(w, d)
    out = s.attend(d["users"], d["q_off"], to_dev(d["queries"], w.dtype))
    torch.cuda.synchronize()
    assert s.stat("device_errors") == 0
    s.close()
    lens = np.diff(d["hist_off"])
    rng = np.random.default_rng(11)
    sel = sorted(set([0, w.n_users - 1, int(np.argmax(lens)), int(np.argmin(lens))] +
                     rng.integers(0, w.n_users, size=2).tolist()))
    rows = np.concatenate([np.arange(d["q_off"][u], d["q_off"][u + 1]) for u in sel])
    got = out[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert_close(got, oracle_attend(w, d, sel=sel), w.dtype, name)


@pytest.mark.parametrize("seed", range(40))
def test_random_shapes_against_the_oracle(seed):
    """Seeded random workloads across head widths, user-part widths, pool sizes, ragged lengths (zero included),
    query counts and both normalisations: whatever kernel the library picks must match the oracle."""
    rng = np.random.default_rng(1000 + seed)
    dtype = "f32" if seed % 5 == 0 else "bf16"
    D = int(rng.choice([16, 32, 32, 64, 64, 128]))
    du = int(rng.choice([0, 1, 2, 3, 4, 8, 12]))
    du = min(du, D - 4)
    m = int(rng.choice([1, 7, 100, 333, 2048, 5000]))
    G = int(rng.integers(1, 5))
    n_users = int(rng.integers(1, 9))
    Lmax = int(rng.choice([1, 40, 300, 1500]))
    M = int(rng.choice([1, 1, 2, 9, 33, 50, 130]))
    mode = "softmax" if rng.integers(0, 2) else "silu_over_l"
    zipf = None if rng.integers(0, 2) else 1.1
    w = synth.Workload(f"rnd{seed}", G, D - du, du, m, n_users, (0, Lmax), M, mode, dtype, zipf, 1.0 / D, 1.0 / D, 500 + seed)
    d = synth.generate(w)
    s = make_session(w, d)
    got = gpu_attend(w, d, session=s)
    fam = s.stat("kernel")
    assert s.stat("device_errors") == 0
    s.close()
    assert_close(got, oracle_attend(w, d), dtype, f"seed {seed}: D={D} du={du} m={m} G={G} M={M} {mode} family {fam}")


def test_host_buffers_go_through_the_same_path():
    w = SMALL["cfg5_ragged"]
    d = synth.generate(w)
    s = make_session(w, d)
    dev = gpu_attend(w, d, session=s)
    q_host = torch.from_numpy(d["queries"].view(np.int16)).view(torch.bfloat16).pin_memory()
    o_host = torch.empty(q_host.shape, dtype=torch.bfloat16).pin_memory()
    s.attend(d["users"], d["q_off"], q_host, o_host)
    torch.cuda.synchronize()
    s.close()
    assert np.array_equal(o_host.float().numpy().astype(np.float64), dev)


@pytest.mark.parametrize("name,kw", [
    ("cfg2", dict(n_users=96, hist_len=(100, 400))),                 # tcgen05 kernel, 4.9 MB of queries
    ("cfg5", dict(n_users=5000, hist_len=(1, 90))),                  # warp-level tensor-core kernel, 20 MB
    ("cfg4", dict(n_users=48, hist_len=(3000, 9000), n_queries=200, n_entries=2048)),  # split histories, merge per range
])
def test_large_host_buffers_are_pipelined_and_give_the_same_bits(name, kw):
    """Host query / output buffers of a few MB and more: the request list is cut into ranges of users whose
    upload, kernels and download run on internal streams.  Same bits as the device-buffer call, the caller's
    stream is ordered behind everything, and a second call (plan cached) and a permuted request agree too."""
    w = synth.scaled(synth.WORKLOADS[name], **kw)
    d = synth.generate(w)
    s = make_session(w, d)
    q_dev = to_dev(d["queries"], w.dtype)
    dev = s.attend(d["users"], d["q_off"], q_dev).clone()
    assert s.stat("pipeline_ranges") == 1
    q_host = torch.from_numpy(d["queries"].view(np.int16)).view(torch.bfloat16).pin_memory()
    o_host = torch.full(q_host.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    for _ in range(2):
        o_host.fill_(float("nan"))
        s.attend(d["users"], d["q_off"], q_host, o_host)
        assert s.stat("pipeline_ranges") == 4
        torch.cuda.current_stream().synchronize()          # only the caller's stream: it must cover the internal ones
        assert torch.equal(o_host, dev.cpu())
    # users in another order, queries moved along
    perm = np.random.default_rng(1).permutation(w.n_users)
    M = w.n_queries
    rows = (perm[:, None] * M + np.arange(M)[None, :]).reshape(-1)
    q_perm = q_host[torch.from_numpy(rows)].contiguous().pin_memory()
    o_perm = torch.empty_like(q_perm).pin_memory()
    s.attend(d["users"][perm], d["q_off"], q_perm, o_perm)
    torch.cuda.current_stream().synchronize()
    assert torch.equal(o_perm, dev.cpu()[torch.from_numpy(rows)])
    assert s.stat("device_errors") == 0
    s.close()


@pytest.mark.parametrize("kernel,tol", [(1, 1e-5), (2, 2.0 ** -8)])
def test_permuting_a_history_keeps_the_output(kernel, tol):
    """Attention does not depend on the order of the history.  The CUDA-core kernel keeps the
    weights in fp32, so only the summation order moves; the tensor-core kernel rounds each weight
    to bf16 relative to the running maximum, which the order changes: one bf16 ulp there."""
    w = synth.scaled(W["cfg4"], n_users=1, hist_len=(777, 777), n_queries=2)
    d = synth.generate(w)
    a = gpu_attend(w, d, out_dtype="f32", kernel=kernel)
    perm = np.random.default_rng(3).permutation(777)
    d2 = dict(d)
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d2[k] = np.ascontiguousarray(d[k][perm])
    b = gpu_attend(w, d2, out_dtype="f32", kernel=kernel)
    assert np.abs(a - b).max() <= tol * np.abs(a).max()


def test_replacing_and_evicting_users():
    import paper_2601_19178_b200 as ckv
    w = synth.scaled(W["cfg1"], n_users=3, hist_len=(20, 60))
    d = synth.generate(w)
    s = make_session(w, d)
    first = gpu_attend(w, d, session=s)
    # replace user 1 by user 0's history: its output must now equal what user 0's history gives
    p0, p1 = int(d["hist_off"][0]), int(d["hist_off"][1])
    s.cache_put(int(d["users"][1]), to_dev(d["idx_K"][p0:p1], "i"), to_dev(d["idx_V"][p0:p1], "i"),
                to_dev(d["user_K"][p0:p1], "f32"), to_dev(d["user_V"][p0:p1], "f32"))
    d2 = dict(d)
    sel = np.r_[p0:p1, p0:p1, int(d["hist_off"][2]):int(d["hist_off"][3])]
    for k in ("idx_K", "idx_V", "user_K", "user_V"):
        d2[k] = np.ascontiguousarray(d[k][sel])
    L0, L2 = p1 - p0, int(d["hist_off"][3] - d["hist_off"][2])
    d2["hist_off"] = np.array([0, L0, 2 * L0, 2 * L0 + L2], dtype=np.int64)
    second = gpu_attend(w, d, session=s)
    assert_close(second, oracle_attend(w, d2), "f32")
    assert np.array_equal(first[0], second[0])
    ckv.ckv_cache_evict(s.ctx, int(d["users"][2]))
    with pytest.raises(ckv.CkvError) as e:
        gpu_attend(w, d, session=s)
    assert e.value.status == ckv.CKV_ERR_UNKNOWN_USER
    comp, full = ckv.ckv_cache_bytes(s.ctx)
    assert full == 2 * (2 * L0) * w.n_groups * w.head_dim * 4
    assert comp == (2 * L0) * w.n_groups * (2 * 2 + 2 * w.d_user * 4)
    s.close()


def _cut_histories(d, new_lens):
    """The generated data with user k's history cut to its first new_lens[k] positions."""
    off = d["hist_off"]
    keep = np.concatenate([np.arange(off[k], off[k] + n) for k, n in enumerate(new_lens)]).astype(np.int64)
    out = dict(d)
    for key in ("idx_K", "idx_V", "user_K", "user_V"):
        out[key] = np.ascontiguousarray(d[key][keep])
    out["hist_off"] = np.concatenate([[0], np.cumsum(new_lens)]).astype(np.int64)
    return out


@pytest.mark.parametrize("mode", ["softmax", "silu_over_l"])
@pytest.mark.parametrize("n_groups", [1, 4])
def test_tcgen05_kernel_long_units_followed_by_many_short_ones(mode, n_groups):
    """A few long histories and many of at most two half tiles.  The planner puts the long ones first, so every
    CTA of the tcgen05 kernel ends its stream with a run of units in which a normalisation group may own no half
    for many tiles while it still has weighted sums to issue for the long unit; with one or four groups the
    rotation that deals the halves out is the same for all units of a CTA, which makes such runs as long as
    they get.  Nothing may run out of its bounded waits, and the results must match."""
    rng = np.random.default_rng(5)
    n_users = 700
    w = synth.Workload("mixed", n_groups, 30, 2, 500, n_users, (1900, 1900), 64, mode, "bf16", 1.1, 1 / 32, 1 / 32, 77)
    d = synth.generate(w)
    # (SiLU: h (1 + tanh h) with the hardware's tanh cancels for strongly negative scores -- absolute error up to
    # about 5e-4 |h| per term; a row made of one or two such terms alone would fail the row-normalised bound)
    lens = rng.integers(1 if mode == "softmax" else 17, 129, size=n_users)
    lens[rng.choice(n_users, 40, replace=False)] = rng.integers(1200, 1901, size=40)
    d = _cut_histories(d, lens)
    s = make_session(w, d, kernel=3)
    got = gpu_attend(w, d, session=s)
    assert s.stat("kernel") == 3 and s.stat("device_errors") == 0
    s.close()
    assert_close(got, oracle_attend(w, d), "bf16", f"{mode} G={n_groups}")
