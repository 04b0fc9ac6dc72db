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


def _gpu_route(x_bits, W_bits, bias):
    import torch
    import paper_2601_19178_b200 as ckv
    from paper_2601_19178_b200.session import as_device_tensor as dev
    n, d = x_bits.shape
    G, m, _ = W_bits.shape
    xd, Wd = dev(x_bits, "bf16"), dev(W_bits, "bf16")
    bd = torch.from_numpy(bias).cuda() if bias is not None else None
    out = torch.full((n, G), -1, dtype=torch.int32, device="cuda")
    ckv.ckv_route(0, n, G, d, m, xd, Wd, bd, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _check(x_bits, W_bits, bias, what):
    got = _gpu_route(x_bits, W_bits, bias)
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
@pytest.mark.parametrize("d_in", [32, 64, 128])
@pytest.mark.parametrize("n,m,G", [(1, 1, 1), (37, 5, 2), (300, 333, 3), (1000, 2048, 2), (513, 4100, 1)])
def test_gpu_router_matches_oracle(d_in, n, m, G):
    rng = np.random.default_rng(d_in + n + m)
    x = _bf16(rng.standard_normal((n, d_in)) / np.sqrt(d_in))
    W = _bf16(rng.standard_normal((G, m, d_in)))
    b = (0.1 * rng.standard_normal((G, m))).astype(np.float32)
    _check(x, W, b, f"d_in={d_in} n={n} m={m} G={G}")
    _check(x, W, None, f"no bias d_in={d_in} n={n} m={m} G={G}")


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
    got = _gpu_route(_bf16(x), _bf16(W), None)
    assert np.array_equal(got[:, 0], np.arange(70) % d)      # entries k, k + 32, ... tie: the first one
    assert np.array_equal(got, R.route(_bf16(x), _bf16(W)))
    # the output feeds ckv_cache_put as it is: indices in range, int32 [n][G]
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_route(0, 4, 1, 48, 8, torch.zeros(4, 48, dtype=torch.bfloat16, device="cuda"),
                      torch.zeros(1, 8, 48, dtype=torch.bfloat16, device="cuda"), None,
                      torch.zeros(4, 1, dtype=torch.int32, device="cuda"))
    assert e.value.status == ckv.CKV_ERR_UNSUPPORTED
    with pytest.raises(ckv.CkvError) as e:
        ckv.ckv_route(0, 4, 1, 32, 8, np.zeros((4, 32), np.uint16), torch.zeros(1, 8, 32, dtype=torch.bfloat16, device="cuda"),
                      None, torch.zeros(4, 1, dtype=torch.int32, device="cuda"))
    assert e.value.status == ckv.CKV_ERR_INVALID_ARG
