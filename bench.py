#!/usr/bin/env python
"""Benchmark of the CollectiveKV decode path (one `ckv_attend` over all users of a workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|cfg2|...] [--impl ours|reference]

Prints ONE JSON line.  A step = one pass of the whole hot path (compressed-cache read, pool
gather, concat, scores, normalisation, weighted sum, split merge, store) over the workload,
with pool and caches resident in HBM.  `value` is cached history positions per second over all
ranks (device time, max over ranks); `e2e` is the same call fed with host buffers (query
upload and output download inside the timed region), `e2e_fresh_plan` the same with a request
list the library has not seen before on every call.  Under torchrun each rank serves its own
users (weak scaling, no collective on the data path).

With `--workload all` (the default) the four large workloads run one after the other in this
process; the line's top-level figures are those of the largest one (cfg5: most positions and
bytes) and `per_config` carries the figures of each.  Per workload: W warm-up steps, a sampled
parity check, then at least one second of back-to-back steps (the SM clock settles to what it
sustains under this load; every step is timed and the clock is sampled throughout), a
synchronise, and the K timed steps of the headline figure.

`--impl reference` times the CPU oracle, as it stands, on this machine's host cores.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "cached_history_positions_per_sec"
UNIT = "positions/s"
HBM_FALLBACK_GBS = 6650.0
ALL_WORKLOADS = ("cfg2", "cfg3", "cfg4", "cfg5")
HEADLINE = "cfg5"            # the largest single-GPU workload: most positions and most bytes
SUSTAIN_SECONDS = 1.0        # back-to-back load per workload before (and around) the timed steps
CPU_SECONDS = {"headline": 15.0, "other": 4.0}   # host time the oracle leg may take per workload
# transcendental evaluations per SM per clock (ex2 / tanh issue rate of the special-function unit)
XU_PER_SM_CLK = 16
# bytes per SM per clock through the L1 / shared-memory data pipe (one 128-byte wavefront per clock)
L1_PIPE_BYTES_PER_SM_CLK = 128
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "traffic.json")
CSRC = os.path.join(ROOT, "paper_2601_19178_b200", "csrc")
KERNEL_SOURCES = {1: ["kernels_simt.cu"], 2: ["kernels_mma.cu"], 3: ["kernels_umma.cu"], 4: ["kernels_fact.cu"]}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback"


def source_hash(family: int) -> str:
    """Hash of the source of a kernel family (and the shared device helpers): the DRAM-traffic record of a
    kernel is only valid for the source it was captured from."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES.get(family, []) + ["ptx_helpers.cuh", "ckv_internal.h"]:
        path = os.path.join(CSRC, name)
        if os.path.exists(path):
            h.update(open(path, "rb").read())
    return h.hexdigest()[:16]


def _traffic(entry: str, family: int, users: int):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the workload's attend kernel(s),
    from the record `--record-traffic` wrote after an ncu capture (profiles/traffic.json), scaled by the number
    of users when the capture ran on a cut of the workload (users are independent: traffic grows in proportion).
    None when there is no record or the kernel's source has changed since."""
    try:
        rec = json.load(open(TRAFFIC_JSON)).get(entry)
    except Exception:
        return None
    if not rec or rec.get("source_hash") != source_hash(family) or rec.get("kernel_family") != family:
        return None
    return rec["dram_bytes"] * users / rec["users"]


def record_traffic(args):
    """Reads an ncu CSV (`ncu -i <rep> --page raw --csv`, one row per launch, or the log of
    `ncu --metrics ...,dram__bytes_read.sum,dram__bytes_write.sum --csv`, one row per launch and metric) and stores
    the DRAM bytes of the captured attend launch(es) in profiles/traffic.json under the entry name given.
    Runs here, without a GPU."""
    import csv
    rows = list(csv.reader(open(args.record_traffic)))
    hdr = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    cols = rows[hdr]
    ci = {c: i for i, c in enumerate(cols)}
    scale = {"byte": 1.0, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9}
    wanted = ("attend_", "fact_", "combine_kernel")
    total, names = 0.0, []
    if "Metric Name" in ci:      # one row per (launch, metric)
        for r in rows[hdr + 1:]:
            if len(r) != len(cols) or not any(k in r[ci["Kernel Name"]] for k in wanted):
                continue
            if r[ci["Metric Name"]] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                total += float(r[ci["Metric Value"]].replace(",", "")) * scale[r[ci["Metric Unit"]].lower()]
                name = r[ci["Kernel Name"]].split("(")[0]
                if name not in names:
                    names.append(name)
    else:                        # one row per launch, units in the row below the header
        units = rows[hdr + 1]
        for r in rows[hdr + 2:]:
            if len(r) != len(cols) or not any(k in r[ci["Kernel Name"]] for k in wanted):
                continue
            for m in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                total += float(r[ci[m]].replace(",", "")) * scale[units[ci[m]].lower()]
            names.append(r[ci["Kernel Name"]].split("(")[0])
    w = synth.WORKLOADS[args.workload if args.workload != "all" else HEADLINE]
    data = {}
    if os.path.exists(TRAFFIC_JSON):
        data = json.load(open(TRAFFIC_JSON))
    data[args.entry] = {"workload": w.name, "users": args.users or w.n_users, "kernel_family": args.family,
                        "kernels": names, "dram_bytes": total, "source_hash": source_hash(args.family),
                        "from": os.path.basename(args.record_traffic)}
    json.dump(data, open(TRAFFIC_JSON, "w"), indent=1, sort_keys=True)
    print(json.dumps(data[args.entry]))


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the bench runs."""

    def __init__(self, uuid: str, period: float = 0.005):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period, [], set(), None
        self._stop_evt, self._on = threading.Event(), threading.Event()
        self.h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode() if not uuid.startswith("GPU-") else uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.h = None

    def run(self):
        if self.h is None:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            if self._on.is_set():
                try:
                    self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                    for bit, name in names.items():
                        if r & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(self.period)

    def on(self):
        self._on.set()

    def off(self):
        self._on.clear()

    def take(self):
        """Summary of the samples since the last call."""
        s, r = self.samples, sorted(self.reasons)
        self.samples, self.reasons = [], set()
        return {"sm_mhz": statistics.median(s) if s else None, "sm_min_mhz": min(s) if s else None,
                "sm_max_mhz": self.max_mhz, "reasons": r, "samples": len(s)}

    def finish(self):
        self._stop_evt.set()


def _oracle_rate(w, data, n_users: int, n_threads: int = 0):
    """Times the CPU oracle on the first n_users users; returns (positions/s, seconds, cores, users, positions)."""
    from oracle import ckv_oracle as O
    n_users = min(n_users, w.n_users)
    sel = np.arange(n_users, dtype=np.int64)
    t0 = time.perf_counter()
    O.attend(w.dtype, w.mode, w.default_scale, data["pool_K"], data["pool_V"], data["hist_off"], data["idx_K"],
             data["idx_V"], data["user_K"], data["user_V"], data["q_off"], data["queries"], sel=sel,
             n_threads=n_threads)
    dt = time.perf_counter() - t0
    pos = int(data["hist_off"][n_users])
    return pos / dt, dt, O.max_threads(), n_users, pos


def _oracle_sample(w, data, seconds: float):
    """The oracle on a bounded sample of the workload: the first users of it, as many as take about `seconds`
    (a short run sizes the next one; the last run is the one reported; the whole workload if that is quicker)."""
    n_users = max(1, min(w.n_users, 64))
    while True:
        rate, dt, cores, n_u, pos = _oracle_rate(w, data, n_users)
        if n_u >= w.n_users or dt >= 0.5 * seconds:
            break
        n_users = int(min(w.n_users, max(2 * n_u, n_u * seconds / max(dt, 1e-3))))
    return {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n_u} of {w.n_users} users ({pos} positions), {dt:.1f} s"}


def rank_env():
    """(rank, world size, local rank) of this process as torchrun exports them; (0, 1, 0) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(w, rank: int) -> int:
    """Weak scaling: every rank serves its own users of the same workload shape."""
    return w.seed + 1000 * rank


def reduce_over_ranks(elapsed, positions: int, users: int, dist=None, device="cpu"):
    """Whole-job figures from per-rank ones: the slowest rank's time, everybody's positions and users.
    No data of the decode path crosses ranks; this is the only communication of the benchmark."""
    if dist is None:
        return float(elapsed), int(positions), int(users)
    import torch
    t = torch.tensor([float(elapsed)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([int(positions), int(users)], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t.item()), int(c[0].item()), int(c[1].item())


def workload_list(args):
    names = ALL_WORKLOADS if args.workload == "all" else (args.workload,)
    ws = []
    for n in names:
        w = synth.WORKLOADS[n]
        if args.users:
            w = synth.scaled(w, n_users=min(args.users, w.n_users))
        ws.append(w)
    return ws


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of users of the headline
    workload (the same workload the CUDA arm puts at the top level of its line)."""
    rank, _, _ = rank_env()
    if rank != 0:
        return
    ws = workload_list(args)
    w = next((x for x in ws if x.name == HEADLINE), ws[-1])
    # the oracle only touches the users it computes: generate a cut that holds the per-step sample
    gen_users = min(w.n_users, 4096)
    wg = synth.scaled(w, n_users=gen_users)
    data = synth.generate(wg)
    # size the per-step sample from a short probe so the whole run stays within ~2 minutes
    probe_users = max(1, min(gen_users, 8))
    _, probe_dt, cores, _, _ = _oracle_rate(wg, data, probe_users)
    per_user = probe_dt / probe_users
    budget = 100.0 / max(1, args.steps + args.warmup)
    n_users = int(max(1, min(gen_users, budget / max(per_user, 1e-9))))
    for _ in range(args.warmup):
        _oracle_rate(wg, data, n_users)
    times, pos = [], 0
    for _ in range(args.steps):
        _, dt, cores, _, pos = _oracle_rate(wg, data, n_users)
        times.append(dt)
    total = sum(times)
    value = pos * args.steps / total
    sample = (f"first {n_users} of {w.n_users} users ({pos} positions) per step; a rate over a sample of the "
              f"workload, not a pass over all of it")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "describe": w.describe, "sample": sample},
        "users_per_sec": n_users * args.steps / total,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class Measured:
    """One workload loaded into a library context on this rank, and the measurements taken on it."""

    def __init__(self, args, w, rank, local, dist, sampler):
        import torch
        import paper_2601_19178_b200 as ckv
        from paper_2601_19178_b200.session import as_device_tensor as dev
        self.torch, self.ckv, self.args, self.w, self.rank, self.local = torch, ckv, args, w, rank, local
        self.dist, self.sampler = dist, sampler
        # weak scaling: every rank serves its own users of the same workload shape
        self.data = data = synth.generate(w, seed=rank_seed(w, rank))
        tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
        self.s = s = ckv.CollectiveKV(w.n_groups, w.head_dim, tdt, w.mode, device=local)
        s.pool_load(dev(data["pool_K"], w.dtype), dev(data["pool_V"], w.dtype))
        ik, iv = dev(data["idx_K"], "i"), dev(data["idx_V"], "i")
        uk, uv = dev(data["user_K"], w.dtype), dev(data["user_V"], w.dtype)
        s.cache_put_batch(data["users"], data["hist_off"], ik, iv, uk, uv)
        del ik, iv, uk, uv
        torch.cuda.empty_cache()
        if args.split_len:
            s.set_option("split_len", args.split_len)
        if args.mma_loader:
            s.set_option("mma_loader", args.mma_loader)
        if args.l2_persist >= 0:
            s.set_option("l2_persist", args.l2_persist)
        s.set_option("time_kernels", 1)
        self.users, self.q_off = data["users"], data["q_off"]
        self.q = dev(data["queries"], w.dtype)
        self.out = torch.empty_like(self.q)
        self.positions = int(data["hist_off"][-1])
        self.comp_bytes, self.full_bytes = ckv.ckv_cache_bytes(s.ctx)
        self.qo_bytes = self.q.numel() * self.q.element_size() + self.out.numel() * self.out.element_size()
        self.algo_bytes = self.comp_bytes + self.qo_bytes
        # L2 flush between timed iterations: overwrite a buffer twice the size of L2
        self.flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream()
        self.q_host = self.o_host = None

    def close(self):
        self.s.close()
        del self.q, self.out, self.flush, self.q_host, self.o_host, self.data
        self.torch.cuda.empty_cache()

    def step(self):
        self.s.attend(self.users, self.q_off, self.q, self.out)

    def parity(self):
        from oracle import ckv_oracle as O
        torch, w, data = self.torch, self.w, self.data
        rng = np.random.default_rng(0)
        lens = np.diff(data["hist_off"])
        sel = sorted(set([0, w.n_users - 1, int(np.argmax(lens)), int(np.argmin(lens))] +
                         rng.integers(0, w.n_users, size=4).tolist()))
        want = O.attend(w.dtype, w.mode, w.default_scale, data["pool_K"], data["pool_V"], data["hist_off"],
                        data["idx_K"], data["idx_V"], data["user_K"], data["user_V"], data["q_off"],
                        data["queries"], sel=sel)
        rows = np.concatenate([np.arange(self.q_off[u], self.q_off[u + 1]) for u in sel])
        got = self.out[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
        atol, rtol = (1e-5, 1e-5) if w.dtype == "f32" else (2e-3, 1e-2)
        err = np.abs(got - want)
        ok = bool((err <= atol + rtol * np.abs(want)).all())
        rown = float((err.max(axis=-1) / np.maximum(np.abs(want).max(axis=-1), 1e-30)).max())
        return {"users_checked": len(sel), "ok": ok, "max_abs_err": float(err.max()), "row_norm_err": rown}

    def timed_steps(self, n_steps):
        """n_steps back-to-back steps (L2 flushed before each), every step timed with CUDA events on the
        launching stream; the library's own events around the attend kernel are read every 32nd step."""
        torch, s = self.torch, self.s
        ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps)]
        ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps)]
        kern_ns, comb_ns, launches = [], [], 0
        for i in range(n_steps):
            self.flush.zero_()
            ev0[i].record(self.stream)
            self.step()
            ev1[i].record(self.stream)
            launches += s.stat("launches")
            if i % 32 == 31 or i == n_steps - 1:
                kern_ns.append(s.stat("main_kernel_ns"))
                comb_ns.append(s.stat("combine_kernel_ns"))
        torch.cuda.synchronize()
        step_ms = [a.elapsed_time(b) for a, b in zip(ev0, ev1)]
        return step_ms, kern_ns, comb_ns, launches

    def e2e(self, fresh_plans: bool):
        """Host query buffer in, host output buffer out, through the same C-ABI call; host wall clock around
        call + synchronise.  fresh_plans: every call carries a request list (a rotation through nine
        permutations of the users) that is not among the plans the library keeps."""
        torch, s = self.torch, self.s
        if self.q_host is None:
            self.q_host = torch.empty(self.q.shape, dtype=self.q.dtype).pin_memory()
            self.q_host.copy_(self.q)
            self.o_host = torch.empty(self.out.shape, dtype=self.out.dtype).pin_memory()
        lists = [(self.users, self.q_off)]
        if fresh_plans:
            # all users of a workload have the same number of queries, so q_off stays as it is
            rng = np.random.default_rng(11)
            lists = [(np.ascontiguousarray(self.users[rng.permutation(self.w.n_users)]), self.q_off) for _ in range(9)]
        n = max(3, min(self.args.steps, 20))
        if fresh_plans:
            n = max(n, len(lists))
        for k in range(2 if not fresh_plans else len(lists)):
            s.attend(lists[k % len(lists)][0], lists[k % len(lists)][1], self.q_host, self.o_host)
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        hits = allocs = 0
        t0 = time.perf_counter()
        for k in range(n):
            u, qo = lists[k % len(lists)]
            s.attend(u, qo, self.q_host, self.o_host)
            torch.cuda.synchronize()
            hits += s.stat("plan_cache_hit")
            allocs += s.stat("alloc_calls")
        secs, pos, _ = reduce_over_ranks(time.perf_counter() - t0, self.positions, self.w.n_users, self.dist, "cuda")
        return {"value": pos * n / secs, "unit": UNIT,
                "h2d_bytes_per_step": self.q_host.numel() * self.q_host.element_size() + self.users.nbytes + self.q_off.nbytes,
                "d2h_bytes_per_step": self.o_host.numel() * self.o_host.element_size(),
                "ms_per_step": 1e3 * secs / n, "steps": n, "plan_cache_hits": hits, "alloc_calls": allocs}

    def measure(self, entry: str, kernel: int, cpu_seconds: float):
        """The whole protocol for one kernel choice on the loaded workload; returns the entry of `per_config`."""
        torch, s, w, args = self.torch, self.s, self.w, self.args
        s.set_option("kernel", kernel)
        warm = max(args.warmup, 3)
        t_probe = []
        for _ in range(warm):
            self.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            self.step()
            e1.record(self.stream)
            t_probe.append((e0, e1))
        torch.cuda.synchronize()
        est_ms = max(1e-3, min(a.elapsed_time(b) for a, b in t_probe))
        parity = self.parity() if (self.rank == 0 and not args.no_check) else None

        # sustained load: at least SUSTAIN_SECONDS of back-to-back steps, then the K timed steps behind a synchronise
        n_sustain = max(args.steps, int(math.ceil(1e3 * args.sustain / est_ms)))
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()
        if self.sampler:
            self.sampler.take()
            self.sampler.on()
        sus_ms, sus_kern, sus_comb, sus_launches = self.timed_steps(n_sustain)
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()
        step_ms, kern_ns, comb_ns, launches = self.timed_steps(args.steps)
        if self.sampler:
            self.sampler.off()
        if self.dist is not None:
            self.dist.barrier()
        clocks = self.sampler.take() if self.sampler else None
        total_ms, job_pos, job_users = reduce_over_ranks(float(sum(step_ms)), self.positions, w.n_users, self.dist, "cuda")
        sus_total_ms, _, _ = reduce_over_ranks(float(sum(sus_ms)), self.positions, w.n_users, self.dist, "cuda")
        e2e = None if args.no_e2e else self.e2e(False)
        e2e_fresh = None if args.no_e2e else self.e2e(True)
        dev_err = s.stat("device_errors")
        if dev_err:
            raise SystemExit(f"{entry}: a kernel gave up on a bounded wait (device_errors = {dev_err})")
        if self.rank != 0:
            return None

        peak, peak_kind = _peaks()
        kern_s = statistics.mean(kern_ns) * 1e-9
        sus_kern_s = statistics.mean(sus_kern) * 1e-9
        family = s.stat("kernel")
        achieved = self.algo_bytes / kern_s / 1e9
        mhz = clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None
        cpu = None if args.no_cpu else _oracle_sample(w, self.data, cpu_seconds)
        # The roof that binds, reported beside the HBM roofline the metric asks for.
        # Many queries per user (tcgen05 kernel): one exp (softmax) or tanh (SiLU) per score on the
        # special-function unit.  Few queries (warp-level tensor-core kernel): every gathered pool row crosses
        # the SM's L1 / shared-memory data pipe twice, once copied into the staging ring and once read
        # out by ldmatrix; the pool rows come from L2, not HBM.
        binding = None
        n_sms = torch.cuda.get_device_properties(self.local).multi_processor_count
        max_mhz = clocks["sm_max_mhz"] if clocks and clocks.get("sm_max_mhz") else None
        if family == 2 and max_mhz:
            pipe_bytes = float(self.positions) * w.n_groups * 2 * (w.head_dim * 2) * 2
            peak_pipe = L1_PIPE_BYTES_PER_SM_CLK * n_sms * max_mhz * 1e6 / 1e9
            binding = {"bound": "l1_shared_data_pipe",
                       "what": "K and V pool rows into the shared-memory ring and out through ldmatrix",
                       "achieved": pipe_bytes / kern_s / 1e9, "peak": peak_pipe, "unit": "GB/s",
                       "frac": pipe_bytes / kern_s / 1e9 / peak_pipe}
        elif family == 3 and max_mhz:
            scores = float(self.positions) * w.n_groups * w.n_queries
            peak_xu = XU_PER_SM_CLK * n_sms * max_mhz * 1e6 / 1e9
            binding = {"bound": "alu", "what": "one ex2/tanh per score on the special-function unit",
                       "achieved": scores / kern_s / 1e9, "peak": peak_xu, "unit": "Gscore/s",
                       "frac": scores / kern_s / 1e9 / peak_xu}
        return {
            "entry": entry, "workload": w.name, "describe": w.describe, "users": w.n_users, "positions": self.positions,
            "value": job_pos * args.steps / (total_ms * 1e-3), "unit": UNIT,
            "users_per_sec": job_users * args.steps / (total_ms * 1e-3),
            "steps": args.steps, "ms_per_step": total_ms / args.steps,
            "sustained": {"steps": n_sustain, "seconds": sus_total_ms * 1e-3, "ms_per_step": sus_total_ms / n_sustain,
                          "value": job_pos * n_sustain / (sus_total_ms * 1e-3), "kernel_us": sus_kern_s * 1e6,
                          "what": "back-to-back steps directly before the timed ones, every step timed"},
            "kernel_family": family, "kernel_option": kernel, "mma_loader": s.stat("mma_loader"),
            "work_items": s.stat("work_items"), "split_items": s.stat("split_items"),
            "l2_window": s.stat("l2_window"),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": _traffic(entry, family, w.n_users), "peak_kind": peak_kind,
                         "algorithmic_bytes": self.algo_bytes, "kernel_us": kern_s * 1e6,
                         "kernel_us_x_sm_mhz": kern_s * 1e6 * mhz if mhz else None,
                         "combine_us": statistics.mean(comb_ns) * 1e-3, "frac_of_nominal_8TBs": achieved / 8000.0},
            "roofline_binding": binding,
            "clocks": clocks,
            "e2e": e2e, "e2e_fresh_plan": e2e_fresh,
            "gpu_launches": launches, "gpu_launches_sustained": sus_launches,
            "cpu_baseline": cpu,
            "parity": parity,
            "compression": {"compressed_bytes": self.comp_bytes, "full_width_bytes": self.full_bytes,
                            "ratio": self.comp_bytes / max(self.full_bytes, 1)},
        }


def run_ours(args):
    import torch

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sampler = None
    if rank == 0:
        try:
            sampler = ClockSampler(str(torch.cuda.get_device_properties(local).uuid))
            sampler.start()
        except Exception:
            sampler = None

    ws = workload_list(args)
    head_name = HEADLINE if any(w.name == HEADLINE for w in ws) else ws[-1].name
    per_config = []
    for w in ws:
        m = Measured(args, w, rank, local, dist, sampler)
        runs = [(w.name, args.kernel)]
        if w.name == "cfg4" and args.kernel == 0 and args.workload == "all":
            # the gathering tensor-core kernel on the same workload: the path that splits the long histories
            runs.append(("cfg4_gather", 2))
        for entry, kernel in runs:
            r = m.measure(entry, kernel, args.cpu_seconds or
                          (CPU_SECONDS["headline"] if w.name == head_name else CPU_SECONDS["other"]))
            if r is not None:
                per_config.append(r)
        m.close()
    if sampler:
        sampler.finish()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    head = next(r for r in per_config if r["entry"] == head_name)
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if synth.WORKLOADS[head["workload"]].dtype == "f32" else "bf16",
        "data": "synthetic",
        "config": {"workload": head["workload"], "describe": head["describe"], "users": head["users"],
                   "positions": head["positions"],
                   "l2": "flushed between timed steps (256 MiB overwrite)",
                   "protocol": f"per workload: warm-up, >= {args.sustain:g} s of back-to-back steps, synchronise, the timed steps",
                   "sustained_steps_before_timed": head["sustained"]["steps"],
                   "kernel_family": head["kernel_family"], "mma_loader": head["mma_loader"],
                   "work_items": head["work_items"], "split_items": head["split_items"],
                   "workloads_in_per_config": [r["entry"] for r in per_config]},
        "users_per_sec": head["users_per_sec"],
        "clocks": head["clocks"],
        "e2e": head["e2e"], "e2e_fresh_plan": head["e2e_fresh_plan"],
        "gpu_launches": sum(r["gpu_launches"] for r in per_config),
        "roofline": head["roofline"],
        "roofline_binding": head["roofline_binding"],
        "cpu_baseline": head["cpu_baseline"],
        "parity": head["parity"],
        "compression": head["compression"],
        "per_config": per_config,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# Table 2 of the paper (A100, SIM model, Kuaivideo): latency in ms against batch size, for context only
PAPER_TABLE2_A100_MS = {"batch": [1, 8, 32, 64, 128, 256, 512],
                        "kv_cache": [0.099, 1.030, 1.808, 3.418, 6.679, 15.216, 32.991],
                        "collectivekv": [0.084, 0.129, 0.136, 0.152, 0.222, 0.375, 0.695]}


def run_load_path(args, w):
    """Decode-stage load path (Sec. 4.4, Table 2): per request batch, the latency of bringing the
    batch's cache from pinned host memory to the GPU.  Classical cache: one copy of the full-width
    K/V bytes, T_load(s d_a).  Here: ckv_cache_import of the packed blob, T_load(s d_u + s), and
    import + ckv_attend, which contains the on-GPU indexing T_index fused with the attention."""
    import torch
    import paper_2601_19178_b200 as ckv
    from paper_2601_19178_b200.session import as_device_tensor as dev

    rank, _, local = rank_env()
    if rank != 0:
        return
    torch.cuda.set_device(local)
    batches = [b for b in (1, 8, 32, 64, 128, 256, 512) if b <= w.n_users]
    data = synth.generate(w)
    tdt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    e = 4 if w.dtype == "f32" else 2
    src = ckv.CollectiveKV(w.n_groups, w.head_dim, tdt, w.mode, device=local)
    src.pool_load(dev(data["pool_K"], w.dtype), dev(data["pool_V"], w.dtype))
    src.cache_put_batch(data["users"], data["hist_off"], dev(data["idx_K"], "i"), dev(data["idx_V"], "i"),
                        dev(data["user_K"], w.dtype), dev(data["user_V"], w.dtype))
    lens = np.diff(data["hist_off"]).astype(np.int32)
    blobs = {b: src.export_blob(data["users"][:b]) for b in batches}

    dst = ckv.CollectiveKV(w.n_groups, w.head_dim, tdt, w.mode, device=local)
    dst.pool_load(dev(data["pool_K"], w.dtype), dev(data["pool_V"], w.dtype))
    q = dev(data["queries"], w.dtype)
    out = torch.empty_like(q)
    full_max = int(data["hist_off"][batches[-1]]) * w.n_groups * 2 * w.head_dim * e
    host_full = torch.empty(full_max, dtype=torch.uint8).pin_memory()
    dev_full = torch.empty(full_max, dtype=torch.uint8, device="cuda")
    reps = max(args.steps, 5)

    def med_ms(fn):
        for _ in range(3):
            fn()
        ts = []
        for _ in range(reps):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            fn()
            torch.cuda.synchronize()
            ts.append(1e3 * (time.perf_counter() - t0))
        return statistics.median(ts)

    rows, ok = [], True
    for b in batches:
        users, L, blob = data["users"][:b], lens[:b], blobs[b]
        q_off = data["q_off"][:b + 1]
        nq = int(q_off[-1])
        positions = int(data["hist_off"][b])
        full_bytes = positions * w.n_groups * 2 * w.head_dim * e

        def load_full():
            dev_full[:full_bytes].copy_(host_full[:full_bytes], non_blocking=True)

        def load_packed():
            ckv.ckv_cache_clear(dst.ctx)
            dst.import_blob(users, L, blob)

        def load_and_attend():
            load_packed()
            dst.attend(users, q_off, q[:nq], out[:nq])

        row = {"batch": b, "positions": positions, "full_kv_bytes": full_bytes, "packed_bytes": blob.numel(),
               "kv_cache_load_ms": med_ms(load_full), "ckv_import_ms": med_ms(load_packed),
               "ckv_import_attend_ms": med_ms(load_and_attend)}
        # same users, same request shape: the resident cache gives the same result (the same bits from the
        # gathering kernels; the factorised path sums its histogram with atomics: up to a bf16 ulp apart)
        ref = src.attend(users, q_off, q[:nq]).float()
        ok = ok and bool((out[:nq].float() - ref).abs().max() <= 2.0 ** -7 * ref.abs().max())
        rows.append(row)
    dst.close()
    src.close()
    line = {"mode": "load_path", "metric": "decode_load_latency_ms", "unit": "ms", "higher_is_better": False,
            "n_gpus": 1, "repeats": reps, "timing": "host wall clock around call + device synchronise, median",
            "data": "synthetic", "dtype": "f32" if w.dtype == "f32" else "bf16",
            "config": {"workload": w.name, "describe": w.describe, "source": "pinned host memory"},
            "rows": rows, "outputs_match_resident_cache": ok, "paper_table2_a100_ms": PAPER_TABLE2_A100_MS}
    print(json.dumps(line), flush=True)


def run_route(args):
    """Prefill router (Sec. 4.3) on a prefill-sized batch: n positions scored against every pool entry of every
    group, arg-max per row.  Reported against the bf16 tensor-core peak (it is a dense contraction)."""
    import torch
    import paper_2601_19178_b200 as ckv
    from oracle import route_oracle as R

    rank, _, local = rank_env()
    if rank != 0:
        return
    torch.cuda.set_device(local)
    n, d_in, m, G = 1 << 20, 64, 16384, 4           # one million positions, the pool shape of cfg4
    rng = np.random.default_rng(7)
    x = synth.f32_to_bf16_bits((rng.standard_normal((n, d_in)) / np.sqrt(d_in)).astype(np.float32))
    W = synth.f32_to_bf16_bits(rng.standard_normal((G, m, d_in)).astype(np.float32))
    b = (0.1 * rng.standard_normal((G, m))).astype(np.float32)
    xd = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).cuda()
    Wd = torch.from_numpy(W.view(np.int16)).view(torch.bfloat16).cuda()
    bd = torch.from_numpy(b).cuda()
    out = torch.empty((n, G), dtype=torch.int32, device="cuda")
    steps, warm = max(args.steps, 3), max(args.warmup, 3)
    for _ in range(warm):
        ckv.ckv_route(local, n, G, d_in, m, xd, Wd, bd, out, args.kernel if args.kernel in (1, 2) else 0)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for e0, e1 in evs:
        e0.record()
        ckv.ckv_route(local, n, G, d_in, m, xd, Wd, bd, out, args.kernel if args.kernel in (1, 2) else 0)
        e1.record()
    torch.cuda.synchronize()
    ms = statistics.mean(e0.elapsed_time(e1) for e0, e1 in evs)
    # sampled parity: 512 positions against the float64 oracle (ties in fp32 may pick an equal-scoring entry)
    sel = rng.integers(0, n, size=512)
    M = R.scores(x[sel], W, b)
    want = np.argmax(M, axis=2).T
    got = out[torch.from_numpy(sel).cuda()].cpu().numpy()
    gi, ii = np.meshgrid(np.arange(G), np.arange(len(sel)))
    gap = M[gi, ii, want] - M[gi, ii, got]
    ok = bool((gap <= 4 * d_in * 2.0 ** -24 * np.abs(M).max()).all())
    flops = 2.0 * n * m * d_in * G
    peak_tf, kind = 1590.0, "fallback"
    pth = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pth):
        try:
            peak_tf, kind = float(json.load(open(pth))["bf16_tflops"]), "measured"
        except Exception:
            pass
    ach = flops / (ms * 1e-3) / 1e12
    line = {"mode": "route", "metric": "router_positions_per_sec", "value": n / (ms * 1e-3), "unit": "positions/s",
            "higher_is_better": True, "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms, "dtype": "bf16",
            "data": "synthetic",
            "config": {"positions": n, "d_in": d_in, "n_entries": m, "n_groups": G, "inputs": "larger than L2",
                       "variant": "warp-level mma" if args.kernel == 1 else "tcgen05"},
            "roofline": {"bound": "tensor", "achieved": ach, "peak": peak_tf, "unit": "TFLOP/s", "frac": ach / peak_tf,
                         "peak_kind": kind, "traffic": None},
            "parity": {"positions_checked": int(len(sel)), "ok": ok, "index_mismatches": int((got != want).sum())},
            "gpu_launches": steps}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="all", choices=["all"] + sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--users", type=int, default=0, help="override the user count (smaller captures)")
    ap.add_argument("--kernel", type=int, default=0)
    ap.add_argument("--split-len", type=int, default=0)
    ap.add_argument("--mma-loader", type=int, default=0, help="1 = cp.async (default), 2 = TMA gathers")
    ap.add_argument("--l2-persist", type=int, default=-1, help="0 / 1: the library's option of that name (default: leave it)")
    ap.add_argument("--sustain", type=float, default=SUSTAIN_SECONDS,
                    help="seconds of back-to-back steps before the timed ones (0: only the timed steps' own count)")
    ap.add_argument("--cpu-seconds", type=float, default=0.0, help="host time of the CPU-oracle leg per workload")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-check", action="store_true", help="skip the sampled parity check")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer legs (profiling runs)")
    ap.add_argument("--route", action="store_true", help="time the prefill router (Sec. 4.3) instead of the attend step")
    ap.add_argument("--load-path", action="store_true",
                    help="time the decode-stage load path per batch size (Sec. 4.4) instead of the attend step")
    ap.add_argument("--record-traffic", metavar="NCU_RAW_CSV",
                    help="no GPU work: store the DRAM bytes of the attend launches of an `ncu --page raw --csv` dump "
                         "in profiles/traffic.json (with --entry, --family, --workload, --users)")
    ap.add_argument("--entry", default="", help="per_config entry the traffic record belongs to (cfg2, cfg4_gather, ...)")
    ap.add_argument("--family", type=int, default=0, help="kernel family of the traffic record")
    args = ap.parse_args()
    if args.record_traffic:
        record_traffic(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.route:
        run_route(args)
    elif args.load_path:
        w = synth.WORKLOADS["cfg4" if args.workload == "all" else args.workload]
        if args.users:
            w = synth.scaled(w, n_users=args.users)
        run_load_path(args, w)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
