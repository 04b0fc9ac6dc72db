"""The seeded input generator: determinism, shapes, distributions, bf16 rounding."""
import numpy as np
import torch

import synth


def test_bf16_rounding_matches_torch_rne():
    x = np.random.default_rng(1).standard_normal(10000).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, -0.0, 3.0e38]      # ties to even, signed zero, large
    bits = synth.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    back = synth.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_generate_is_deterministic_and_shaped():
    w = synth.scaled(synth.WORKLOADS["cfg4"], n_users=7, hist_len=(10, 50))
    a, b = synth.generate(w), synth.generate(w)
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    P = int(a["hist_off"][-1])
    assert a["idx_K"].shape == (P, 4) and a["user_V"].shape == (P, 4, 4)
    assert a["pool_K"].shape == (4, 16384, 60) and a["pool_K"].dtype == np.uint16
    assert a["queries"].shape == (7, 4, 64)
    lens = np.diff(a["hist_off"])
    assert lens.min() >= 10 and lens.max() <= 50
    assert len(set(a["users"].tolist())) == 7
    assert not np.array_equal(a["idx_K"], a["idx_V"])


def test_value_distributions_follow_the_recipe():
    w = synth.scaled(synth.WORKLOADS["cfg3"], n_users=8, hist_len=(512, 512), n_queries=4)
    d = synth.generate(w)
    assert abs(synth.bf16_bits_to_f32(d["user_K"]).std() - np.sqrt(0.05)) < 0.01
    assert abs(synth.bf16_bits_to_f32(d["pool_K"]).std() - np.sqrt(1 / 32)) < 0.005
    assert abs(synth.bf16_bits_to_f32(d["queries"]).std() - 1.0) < 0.05
    assert d["idx_K"].min() >= 0 and d["idx_K"].max() < w.n_entries
    # Zipf(1.2): the most frequent row of a group carries ~ 1 / H(m, 1.2) of the mass
    col = d["idx_K"][:, 0]
    top = np.bincount(col, minlength=w.n_entries).max() / col.size
    h = (np.arange(1, w.n_entries + 1) ** -1.2).sum()
    assert abs(top - 1 / h) < 0.03
