"""The range-checked build of the library (build.py --bounds, -DCKV_BOUNDS): every pool index, arena unit,
query / output / partial row and shared-memory offset the kernels compute is compared with its bound, and a
violation lands in the context's error word instead of a wild access.  It stands in for a memory checker, which
cannot be run on the GPUs these tests use.  A sample of the parity cases (every kernel family, split histories,
the variants) runs on it in a process of its own; the kernels must report no violation and still match the oracle."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LIB = os.path.join(ROOT, "paper_2601_19178_b200", "libckv_bounds.so")

CHILD = r"""
import numpy as np, torch, synth
from ckv_testlib import assert_close, gpu_attend, make_session, oracle_attend, to_dev
import paper_2601_19178_b200 as ckv
assert ckv.LIB_PATH.endswith("libckv_bounds.so")
W = synth.WORKLOADS
cases = [
    ("cfg1", dict(n_users=9, hist_len=(1, 700), n_queries=3), 0),              # CUDA cores, fp32
    ("cfg2", dict(n_users=5, hist_len=(1, 900)), 0),                           # tcgen05, softmax, tails
    ("cfg3", dict(n_users=3, hist_len=(100, 1500)), 0),                        # tcgen05, SiLU
    ("cfg4", dict(n_users=6, hist_len=(1, 4000)), 2),                          # warp-level, 64-wide, split
    ("cfg4", dict(n_users=6, hist_len=(3000, 9000)), 4),                       # pool-side factorisation
    ("cfg5", dict(n_users=70, hist_len=(1, 700)), 0),                          # warp-level, 32-wide
    ("cfg5", dict(n_users=20, hist_len=(1, 300), n_queries=3), 1),             # CUDA cores, bf16
]
for name, kw, kernel in cases:
    w = synth.scaled(W[name], **kw)
    d = synth.generate(w)
    s = make_session(w, d, kernel=kernel, split_len=256)
    got = gpu_attend(w, d, session=s)
    assert s.stat("device_errors") == 0, (name, kernel, s.stat("device_errors"))
    # visible lengths on the same cache (CUDA-core and warp-level kernels)
    if kernel in (0, 1, 2):
        rng = np.random.default_rng(2)
        vis = np.concatenate([rng.integers(0, L + 1, size=w.n_queries) for L in np.diff(d["hist_off"])]).astype(np.int32)
        s.attend_visible(d["users"], d["q_off"], vis, to_dev(d["queries"], w.dtype))
        torch.cuda.synchronize()
        assert s.stat("device_errors") == 0, (name, "visible", s.stat("device_errors"))
    s.close()
    assert_close(got, oracle_attend(w, d), w.dtype, f"{name} kernel {kernel}")
print("BOUNDS_OK", len(cases))
"""


def test_sample_of_parity_cases_on_the_range_checked_build():
    if not os.path.exists(LIB):
        sys.path.insert(0, os.path.join(ROOT, "paper_2601_19178_b200"))
        import importlib.util
        spec = importlib.util.spec_from_file_location("_ckv_build", os.path.join(ROOT, "paper_2601_19178_b200", "build.py"))
        mod = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(mod)
        mod.build(bounds=True)
    env = dict(os.environ, CKV_LIBRARY=LIB, PYTHONPATH=os.pathsep.join([ROOT, os.path.join(ROOT, "tests")]))
    r = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, env=env, cwd=ROOT, timeout=900)
    assert r.returncode == 0 and "BOUNDS_OK" in r.stdout, (r.stdout[-2000:], r.stderr[-3000:])
