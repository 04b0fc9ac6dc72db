"""The benchmark's multi-rank plumbing on CPU (gloo, two ranks): users are sharded over ranks with
no collective on the decode path; only the timing and the counts are reduced."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    import bench
    import synth
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        w = synth.scaled(synth.WORKLOADS["cfg4"], n_users=6)
        data = synth.generate(w, seed=bench.rank_seed(w, rank))   # ragged: ranks hold different totals
        positions = int(data["hist_off"][-1])
        elapsed = 10.0 + 5.0 * rank                               # rank 1 is the slow one
        t, p, u = bench.reduce_over_ranks(elapsed, positions, w.n_users, dist, "cpu")
        with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
            json.dump({"t": t, "p": p, "u": u, "own": positions, "ids": data["users"][:3].tolist(),
                       "first_len": int(data["hist_off"][1])}, f)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_counts_by_sum(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = (json.load(open(tmp_path / f"r{k}.json")) for k in (0, 1))
    assert r0["t"] == r1["t"] == 15.0                      # the slowest rank sets the time
    assert r0["p"] == r1["p"] == r0["own"] + r1["own"]     # whole-job positions
    assert r0["u"] == r1["u"] == 12
    assert r0["own"] != r1["own"] or r0["first_len"] != r1["first_len"]   # ranks serve different users' histories


def test_single_process_reduce_is_identity():
    import bench
    assert bench.reduce_over_ranks(3.5, 100, 7) == (3.5, 100, 7)
    assert bench.rank_env() == (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                                int(os.environ.get("LOCAL_RANK", "0")))


def test_reference_arm_under_two_ranks_prints_one_line():
    """`bench.py --impl reference` under torchrun: rank 0 times the oracle, the other ranks exit 0 silently."""
    env = dict(os.environ)
    env.pop("RANK", None)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--impl", "reference",
           "--gpus", "2", "--workload", "cfg1", "--steps", "1", "--warmup", "0"]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
