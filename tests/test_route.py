"""Prefill router (Sec. 4.3): oracle pins on the CPU, CUDA kernel against the oracle on the GPU."""
import numpy as np
import pytest

import synth
from oracle import route_oracle as R


def _bf16(a):
    return synth.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def test_oracle_equals_scalar_loops_on_tiny_inputs():
    rng = np.random.default_rng(1)
    n, G, m, d = 5, 2, 7, 4
    x = rng.standard_normal((n, d)).astype(np.float32)
    W = rng.standard_normal((G, m, d)).astype(np.float32)
    b = rng.standard_normal((G, m)).astype(np.float32)
    want = np.zeros((n, G), dtype=np.int32)
    for i in range(n):
        for g in range(G):
            best, arg = -np.inf, -1
            for j in range(m):
                sc = float(b[g, j])
                for k in range(d):
                    sc += float(x[i, k]) * float(W[g, j, k])
                if sc > best:
                    best, arg = sc, j
            want[i, g] = arg
    assert np.array_equal(R.route(x, W, b), want)


def test_oracle_closed_forms():
    # entries are the coordinate axes: the position picks its largest coordinate
    d = 6
    W = np.eye(d, dtype=np.float32)[None]
    x = np.array([[0.1, 0.9, -3, 0.2, 0.3, 0.0], [5, 1, 1, 1, 1, 1], [-1, -2, -0.5, -4, -3, -9]], dtype=np.float32)
    assert R.route(x, W).ravel().tolist() == [1, 0, 2]
    # equal scores: the lowest index wins
    W2 = np.ones((1, 4, d), dtype=np.float32)
    assert R.route(x, W2).ravel().tolist() == [0, 0, 0]
    # a bias can overrule the product; the groups are independent routers
    b = np.zeros((1, d), dtype=np.float32)
    b[0, 4] = 100.0
    assert R.route(x, W, b).ravel().tolist() == [4, 4, 4]
    Wg = np.stack([np.eye(d, dtype=np.float32), np.eye(d, dtype=np.float32)[::-1]])
    out = R.route(x, Wg)
    assert out[:, 0].tolist() == [1, 0, 2] and out[:, 1].tolist() == [d - 1 - 1, d - 1 - 0, d - 1 - 2]
    # permuting the entries permutes the indices (no ties here)
    rng = np.random.default_rng(2)
    Wr = rng.standard_normal((1, 9, d)).astype(np.float32)
    perm = rng.permutation(9)
    base = R.route(x, Wr)[:, 0]
    assert np.array_equal(perm[R.route(x, Wr[:, perm])[:, 0]], base)
    # bfloat16 bit patterns are widened exactly
    assert np.array_equal(R.route(_bf16(x), _bf16(Wr)), R.route(synth.bf16_bits_to_f32(_bf16(x)), synth.bf16_bits_to_f32(_bf16(Wr))))


def _gpu_route(x_bits, W_bits, bias, variant=0):
    import torch
    import paper_2601_19178_b200 as ckv
    from paper_2601_19178_b200.session import as_device_tensor as dev
    n, d = x_bits.shape
    G, m, _ = W_bits.shape
    xd, Wd = dev(x_bits, "bf16"), dev(W_bits, "bf16")
    bd = torch.from_numpy(bias).cuda() if bias is not None else None
    out = torch.full((n, G), -1, dtype=torch.int32, device="cuda")
    ckv.ckv_route(0, n, G, d, m, xd, Wd, bd, out, variant)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _check(x_bits, W_bits, bias, what, variant=0):
    got = _gpu_route(x_bits, W_bits, bias, variant)
    M = R.scores(x_bits, W_bits, bias)                     # [G][n][m] float64
    want = np.argmax(M, axis=2).T
    n, G = want.shape
    assert got.min() >= 0 and got.max() < W_bits.shape[1], what
    # the kernel sums in fp32: where its choice differs from the float64 arg-max, the two scores must be equal
    # within the rounding of a d_in-term fp32 sum
    gi, ii = np.meshgrid(np.arange(G), np.arange(n))
    s_got, s_want = M[gi, ii, got], M[gi, ii, want]
    tol = 4 * x_bits.shape[1] * 2.0 ** -24 * np.abs(M).max()
    bad = (got != want) & (s_want - s_got > tol)
    assert not bad.any(), f"{what}: {int(bad.sum())} positions routed to a worse entry"
    assert (got != want).mean() < 0.01, what


@pytest.mark.gpu
@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("d_in", [32, 64, 128])
@pytest.mark.parametrize("n,m,G", [(1, 1, 1), (37, 5, 2), (300, 333, 3), (1000, 2048, 2), (513, 4100, 1)])
def test_gpu_router_matches_oracle(d_in, n, m, G, variant):
    rng = np.random.default_rng(d_in + n + m)
    x = _bf16(rng.standard_normal((n, d_in)) / np.sqrt(d_in))
    W = _bf16(rng.standard_normal((G, m, d_in)))
    b = (0.1 * rng.standard_normal((G, m))).astype(np.float32)
    _check(x, W, b, f"d_in={d_in} n={n} m={m} G={G} variant={variant}", variant)
    _check(x, W, None, f"no bias d_in={d_in} n={n} m={m} G={G} variant={variant}", variant)


@pytest.mark.gpu
def test_gpu_router_exact_cases_and_errors():
    import torch
    import paper_2601_19178_b200 as ckv
    d = 32
    # one-hot inputs against one-hot entries (scores are exactly 0 or 1): ties resolve to the lowest entry
    m = 200
    W = np.zeros((1, m, d), dtype=np.float32)
    for j in range(m):
        W[0, j, j % d] = 1.0
    x = np.eye(d, dtype=np.float32)[np.arange(70) % d]
    for variant in (1, 2):
        got = _gpu_route(_bf16(x), _bf16(W), None, variant)
        assert np.array_equal(got[:, 0], np.arange(70) % d)      # entries k, k + 32, ... tie: the first one
        assert np.array_equal(got, R.route(_bf16(x), _bf16(W)))
    # the output feeds ckv_cache_put as it is: indices in range, int32 [n][G]
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_route(0, 4, 1, 48, 8, torch.zeros(4, 48, dtype=torch.bfloat16, device="cuda"),
                      torch.zeros(1, 8, 48, dtype=torch.bfloat16, device="cuda"), None,
                      torch.zeros(4, 1, dtype=torch.int32, device="cuda"), 0)
    assert e.value.status == ckv.CKV_ERR_UNSUPPORTED
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_route(0, 4, 1, 32, 8, np.zeros((4, 32), np.uint16), torch.zeros(1, 8, 32, dtype=torch.bfloat16, device="cuda"),
                      None, torch.zeros(4, 1, dtype=torch.int32, device="cuda"), 0)
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG


def test_projection_oracle_equals_scalar_loops():
    rng = np.random.default_rng(3)
    n, G, dout, d = 4, 2, 3, 8
    x = rng.standard_normal((n, d)).astype(np.float32)
    W = rng.standard_normal((G, dout, d)).astype(np.float32)
    b = rng.standard_normal((G, dout)).astype(np.float32)
    want = np.zeros((n, G, dout))
    for i in range(n):
        for g in range(G):
            for c in range(dout):
                want[i, g, c] = float(b[g, c]) + sum(float(x[i, k]) * float(W[g, c, k]) for k in range(d))
    assert np.allclose(R.project(x, W, b), want, rtol=1e-12, atol=1e-12)
    # unit weights copy coordinates; without a bias a zero input gives zero
    E = np.zeros((1, 2, d), dtype=np.float32)
    E[0, 0, 5] = 1.0
    E[0, 1, 2] = -1.0
    y = R.project(x, E)
    assert np.array_equal(y[:, 0, 0], x[:, 5].astype(np.float64)) and np.array_equal(y[:, 0, 1], -x[:, 2].astype(np.float64))
    assert not R.project(np.zeros_like(x), W).any()


@pytest.mark.gpu
@pytest.mark.parametrize("d_in,d_out,G,n", [(8, 1, 1, 1), (64, 4, 4, 1000), (128, 8, 8, 777), (256, 16, 2, 300), (32, 2, 3, 5000)])
def test_gpu_projection_matches_oracle(d_in, d_out, G, n):
    import torch
    import paper_2601_19178_b200 as ckv
    from paper_2601_19178_b200.session import as_device_tensor as dev
    rng = np.random.default_rng(d_in + n)
    x = _bf16(rng.standard_normal((n, d_in)))
    W = _bf16(rng.standard_normal((G, d_out, d_in)) / np.sqrt(d_in))
    b = (0.1 * rng.standard_normal((G, d_out))).astype(np.float32)
    for bias in (b, None):
        out = torch.zeros((n, G, d_out), dtype=torch.bfloat16, device="cuda")
        ckv.ckv_project(0, n, G, d_in, d_out, dev(x, "bf16"), dev(W, "bf16"),
                        torch.from_numpy(bias).cuda() if bias is not None else None, out)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy().astype(np.float64)
        want = R.project(x, W, bias)
        # fp32 sums rounded to bf16: within one bf16 unit in the last place of the exact value
        assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-6), f"d_in={d_in} d_out={d_out}"
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_project(0, n, G, d_in, 17, dev(x, "bf16"), dev(W, "bf16"), None, out)
    assert e.value.status == ckv.CKV_ERR_UNSUPPORTED


@pytest.mark.gpu
def test_prefill_outputs_feed_the_decode_path():
    """Router indices and projected user parts go into ckv_cache_put as they are; attending over them matches the
    oracle fed with the oracle's own prefill results."""
    import torch
    import paper_2601_19178_b200 as ckv
    from paper_2601_19178_b200.session import as_device_tensor as dev
    from ckv_testlib import assert_close
    from oracle import ckv_oracle as O
    rng = np.random.default_rng(12)
    G, d_in, m, dg, du, U, M = 2, 64, 300, 60, 4, 5, 3
    lens = rng.integers(1, 200, size=U)
    hist_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    P = int(hist_off[-1])
    x = _bf16(rng.standard_normal((P, d_in)) / np.sqrt(d_in))
    Wr = {k: _bf16(rng.standard_normal((G, m, d_in))) for k in "KV"}
    Wu = {k: _bf16(rng.standard_normal((G, du, d_in)) / np.sqrt(d_in) * 0.2) for k in "KV"}
    pool = {k: _bf16(rng.standard_normal((G, m, dg)) / 8) for k in "KV"}
    q = _bf16(rng.standard_normal((U * M, G, dg + du)) / 8)
    q_off = (np.arange(U + 1) * M).astype(np.int32)
    users = np.arange(U, dtype=np.int64) + 10

    xd = dev(x, "bf16")
    idx, usr = {}, {}
    for k in "KV":
        idx[k] = torch.empty((P, G), dtype=torch.int32, device="cuda")
        usr[k] = torch.empty((P, G, du), dtype=torch.bfloat16, device="cuda")
        ckv.ckv_route(0, P, G, d_in, m, xd, dev(Wr[k], "bf16"), None, idx[k])
        ckv.ckv_project(0, P, G, d_in, du, xd, dev(Wu[k], "bf16"), None, usr[k])
    s = ckv.CollectiveKV(G, dg + du, torch.bfloat16, "softmax")
    s.pool_load(dev(pool["K"], "bf16"), dev(pool["V"], "bf16"))
    s.cache_put_batch(users, hist_off, idx["K"], idx["V"], usr["K"], usr["V"])
    got = s.attend(users, q_off, dev(q, "bf16")).float().cpu().numpy().astype(np.float64)
    s.close()

    o_idx = {k: R.route(x, Wr[k]) for k in "KV"}
    for k in "KV":
        assert np.array_equal(idx[k].cpu().numpy(), o_idx[k])          # no near-ties in this draw
    o_usr = {k: _bf16(R.project(x, Wu[k]).astype(np.float32)) for k in "KV"}   # the cache stores bf16
    for k in "KV":
        g_bits = usr[k].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.abs(g_bits.astype(np.int32) - o_usr[k].astype(np.int32)).max() <= 1   # fp32 sum vs exact: one ulp
    want = O.attend("bf16", "softmax", 1.0 / np.sqrt(dg + du), pool["K"], pool["V"], hist_off, o_idx["K"], o_idx["V"],
                    o_usr["K"], o_usr["V"], q_off, q)
    assert_close(got, want, "bf16", "prefill -> decode")
