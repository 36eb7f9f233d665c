#!/usr/bin/env python
"""Benchmark of the evolutionary batch-size search: one step = one generation
(tournament selection + elites, fused crossover/mutation, scoring of the new
population) over the "large" workload (2048 jobs, population 65536).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is candidate-schedule evaluations per second over
all ranks with the population resident in HBM; `e2e` is the same metric when
every step also uploads the job table from host memory and reads the best
schedule back; `roofline` is the dominant kernel against the measured HBM copy
bandwidth; `cpu_baseline` is the single-threaded CPU oracle on a bounded sample.
With N > 1 every rank runs an independent search (replicas, no data-path
collective).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2108_03645_b200 import inputs  # noqa: E402

METRIC = "candidate_evals_per_s"
UNIT = "candidate-schedule evaluations/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
# multi-rank plumbing (replicas: no data-path collective, only the barrier and the timing reduction)
# ----------------------------------------------------------------------------------------------
def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank searches on its own random stream."""
    return base_seed + rank


def max_over_ranks(x: float, device="cpu") -> float:
    """The slowest rank's figure (all-reduce MAX); identity when not distributed."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, units_per_rank_step: int, steps: int, ms: float) -> float:
    """Units all ranks processed per second, over the slowest rank's time."""
    return world * units_per_rank_step * steps / (ms * 1e-3)


# ----------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.sm, self.reasons, self.sm_max = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    def _loop(self):
        nv = self._nvml
        while not self._stop.is_set():
            try:
                self.sm.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self._nvml is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


# ----------------------------------------------------------------------------------------------
# CPU oracle on a bounded sample of the workload
# ----------------------------------------------------------------------------------------------
def oracle_sample(w, pop_sample: int, gens: int):
    """Seconds for `gens` generations of a `pop_sample`-candidate population (single thread)."""
    import oracle
    p = w.params
    s = oracle.Search(w.jobs, w.capacity, pop_sample, elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut,
                      penalty=p.penalty, flags=p.flags)
    s.randomize(w.seed)
    s.evaluate()
    t0 = time.perf_counter()
    s.evolve(gens, w.seed)
    dt = time.perf_counter() - t0
    s.close()
    return dt


def cpu_baseline(w, pop_sample=8192, gens=None):
    pop_sample = min(pop_sample, w.pop)
    if w.params.flags & 16:
        # per-GPU genome: the oracle's reorder costs slots x jobs per row (about 3.5 ms at 4096 x 2048)
        pop_sample, gens = min(pop_sample, 1024), 4
    if gens is None:  # about 1e8 gene evaluations: seconds of single-thread work
        gens = int(min(2000, max(8, 1.3e8 / (pop_sample * w.n_jobs))))
    dt = oracle_sample(w, pop_sample, gens)
    return {"value": pop_sample * gens / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{gens} generations of a {pop_sample}-candidate population (of {w.pop}), "
                      f"{w.n_jobs} jobs, same job table and parameters; {dt:.1f} s"}


def run_reference(args, w):
    """The reference arm: the CPU oracle as it stands, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pop_sample = min(8192, w.pop)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, pop_sample, 1)
    steps = max(1, min(args.steps, 20))
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_sample(w, pop_sample, 1)
    dt = time.perf_counter() - t0
    value = pop_sample * steps / dt
    sample = (f"each step = 1 generation of a {pop_sample}-candidate population (of {w.pop}), {w.n_jobs} jobs, "
              f"single thread; {steps} steps timed (capped at 20)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * dt / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "jobs": w.n_jobs, "population": w.pop, "capacity": w.capacity},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# online loop: per-round search latency and simulated job completion time
# ----------------------------------------------------------------------------------------------
def run_online(args):
    import torch
    from paper_2108_03645_b200 import binding, online

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    trace = inputs.online_trace()

    def gpu_engine(jobs, capacity, pop, params, n_jobs_max):
        return binding.Search(jobs, capacity, pop, params, n_jobs_max=n_jobs_max)

    def cpu_engine(jobs, capacity, pop, params, n_jobs_max):
        import oracle
        return oracle.Search(jobs, capacity, pop, elitism=params.elitism, tournament=params.tournament,
                             p_mut=params.p_mut, penalty=params.penalty, flags=params.flags)

    online.simulate(trace, gpu_engine, max_rounds=20, sync=torch.cuda.synchronize)  # warm-up
    res = online.simulate(trace, gpu_engine, keep_schedules=True, sync=torch.cuda.synchronize)
    lat = np.array(res.latency_s) * 1e3
    line = {"metric": "online_round_latency_ms", "value": float(lat.mean()), "unit": "ms per scheduling round "
            "(ones_update_jobs + 50 generations of a 4096-candidate population + ones_best with repair)",
            "n_gpus": 1, "higher_is_better": False, "data": "synthetic", "dtype": "f64",
            "config": {"workload": "online", "trace_jobs": int(trace.jobs.shape[0]), "capacity": trace.capacity,
                       "population": trace.pop, "generations_per_round": trace.generations,
                       "period_s": trace.period_s},
            "rounds": res.rounds, "p50_ms": float(np.percentile(lat, 50)), "p99_ms": float(np.percentile(lat, 99)),
            "max_ms": float(lat.max()), "mean_active_jobs": float(np.mean(res.active)),
            "max_active_jobs": int(max(res.active)), "mean_jct_s": res.mean_jct,
            "jobs_finished": int(np.isfinite(res.jct).sum())}
    if not args.no_cpu_baseline:
        k = 12
        t0 = time.perf_counter()
        ref = online.simulate(trace, cpu_engine, max_rounds=k, keep_schedules=True)
        dt = time.perf_counter() - t0
        same = all(ia == ib and (ga == gb).all() for (_, ia, ga), (_, ib, gb) in zip(res.deployed, ref.deployed))
        line["cpu_baseline"] = {"value": 1e3 * float(np.mean(ref.latency_s)), "unit": "ms per scheduling round",
                                "cores": 1, "kind": "oracle",
                                "sample": f"first {k} rounds of the same trace; {dt:.1f} s",
                                "schedules_identical_to_gpu": bool(same)}
    print(json.dumps(line))


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of this
# benchmark's default workload at its full population (profiles/dram_traffic_large_pop65536.md).  They belong
# to the kernels as they were when the capture was taken: set an entry to None when its kernel changes.
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("large", 65536, "k_evolve_score"): 403.6e6 + 485.2e6,
    ("large", 65536, "k_evolve"): 401.6e6 + 483.0e6,
    ("large", 65536, "k_fitness"): 537.1e6 + 0.7e6,
}


# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(inputs.WORKLOADS) + ["online"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-events", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--pop", type=int, default=0, help="override the population size (profiling a smaller case)")
    ap.add_argument("--scheme", default="tournament", choices=["tournament", "truncation", "per_gpu"],
                    help="truncation = the paper's best-K-of-4K selection (ONES_FLAG_TRUNCATION); per_gpu = the "
                         "paper's one-slot-per-GPU genome with the reorder operation (ONES_FLAG_PER_GPU)")
    args = ap.parse_args()
    if args.workload == "online":
        if args.impl == "ours" and int(os.environ.get("RANK", "0")) == 0:
            run_online(args)
        return
    w = inputs.WORKLOADS[args.workload]()
    if args.pop:
        import dataclasses
        w = dataclasses.replace(w, pop=args.pop)
    if args.scheme != "tournament":
        import dataclasses
        bit = 4 if args.scheme == "truncation" else 16
        w = dataclasses.replace(w, params=dataclasses.replace(w.params, flags=w.params.flags | bit))
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2108_03645_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    warmup = max(args.warmup, 3)
    steps = max(args.steps, 1)

    base = cpu_baseline(w) if (rank == 0 and world == 1 and not args.no_cpu_baseline) else None

    seed = rank_seed(w.seed, rank)
    s = binding.Search(w.jobs, w.capacity, w.pop, w.params)
    s.randomize(seed)
    s.evolve(warmup, seed)
    torch.cuda.synchronize()

    # ---- device-resident timed region: K generations ----
    if not args.no_kernel_events:
        s.set_profiling(8 if steps >= 64 else 1)  # event pairs around every 8th generation's kernels
        s.stage_times()
    sampler = ClockSampler(local)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = s.kernel_launches
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    ev0.record()
    s.evolve(steps, seed)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    launches = s.kernel_launches - launches0
    stage_ms, stage_n = ({}, {})
    if not args.no_kernel_events:
        stage_ms, stage_n = s.stage_times()
        s.set_profiling(False)
    ms = max_over_ranks(ms, "cuda")

    # ---- end to end: every step uploads the job table and reads the best schedule back ----
    J, N, E = w.n_jobs, w.pop, w.params.elitism
    e2e_steps = 0 if args.no_e2e else min(steps, 100)
    identity = np.arange(J, dtype=np.int32)
    jobs_pinned = torch.from_numpy(w.jobs.view(np.uint8).reshape(-1).copy()).pin_memory()
    jobs_host = jobs_pinned.numpy().view(inputs.JOB_DTYPE)
    out = {"fitness": None}
    e2e_s = float("nan")
    if e2e_steps:
        for _ in range(3):
            s.update_jobs(jobs_host, identity, w.capacity)
            s.evolve(1, seed)
            s.best(False)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            s.update_jobs(jobs_host, identity, w.capacity)
            s.evolve(1, seed)
            out = s.best(False)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_s = max_over_ranks(e2e_s, "cuda")
    h2d = J * 48 + J * 4
    d2h = J * (4 + 4 + 8) + 24 + 4

    # ---- the two separate kernels (crossover/mutation, fitness) on the same workload ----
    sep = None
    if rank == 0 and world == 1 and not args.no_kernel_events and args.scheme == "tournament":
        import dataclasses
        s.close()
        del s
        torch.cuda.empty_cache()
        p2 = dataclasses.replace(w.params, flags=w.params.flags | binding.FLAG_UNFUSED)
        s2 = binding.Search(w.jobs, w.capacity, w.pop, p2)
        s2.randomize(seed)
        s2.evolve(warmup, seed)
        s2.set_profiling(True)
        s2.stage_times()
        s2.evolve(min(steps, 200), seed)
        sep = s2.stage_times()
        s2.set_profiling(False)
        # the score step on packed rows (one byte per gene); two copies read in turn so that a launch never
        # finds its rows in L2 from the launch before (2 x N x ld8 bytes against 126 MB of L2)
        packs = [s2.pack(), s2.pack()]
        outF, outG = s2.evaluate_packed(packs[0])
        reps = 20
        torch.cuda.synchronize()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        for i in range(reps):
            s2.evaluate_packed(packs[i & 1], out=(outF, outG))
        p1.record()
        torch.cuda.synchronize()
        packed_ms = p0.elapsed_time(p1) / reps
        packed_bytes = packs[0].shape[0] * (packs[0].shape[1] + 12)
        del packs
        s2.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    line = {
        "metric": METRIC, "value": whole_job_rate(world, N, steps, ms), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "jobs": J, "population": N, "capacity": w.capacity,
                   "elitism": E, "tournament": w.params.tournament, "p_mut": w.params.p_mut,
                   "genome_table_bytes": N * J * 4, "l2": "inputs larger than L2 (two 512 MiB population buffers)",
                   "parallelism": "replicas" if world > 1 else "single GPU"},
        "generations_per_s": world * steps / (ms * 1e-3),
        "gpu_launches": launches,
        "clocks": clocks,
        "e2e": None if not e2e_steps else {"value": world * N * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "what": "per step: ones_update_jobs(host job table) + ones_evolve(1) + ones_best(host outputs)",
                "best_fitness": out["fitness"]},
    }
    if args.scheme == "per_gpu":
        Wg = w.capacity
        line["config"]["scheme"] = f"per-GPU genome: {Wg} slots per candidate, reorder after crossover and mutation"
        if stage_n.get("evolve"):
            peak, peak_kind = measured_peak()
            rows = {"k_evolve": ("evolve", 8 * Wg * N),
                    "k_per_gpu<reorder, score>": ("fitness", N * (8 * Wg + 12)),
                    "k_select_stage": ("select", 8 * N)}
            line["kernels"] = {}
            for name, (stage, nbytes) in rows.items():
                t_ms = stage_ms[stage] / stage_n[stage]
                a = nbytes / (t_ms * 1e-3) / 1e9
                line["kernels"][name] = {"bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                                         "bytes_per_generation": nbytes, "ms_per_generation": t_ms}
            dom = max(line["kernels"].items(), key=lambda kv: kv[1]["ms_per_generation"])
            line["roofline"] = dict(dom[1], kernel=dom[0], peak_kind=f"of {peak_kind}", traffic=None)
    if args.scheme == "truncation":
        line["config"]["scheme"] = "truncation: pool of 4N rows, 3N new candidates scored per generation"
        line["new_candidates_per_s"] = 3 * line["value"]
        if stage_n.get("evolve"):
            peak, peak_kind = measured_peak()
            if stage_n.get("fitness"):  # children written first, scored by a separate pass
                rows = {"children (k_trunc_draws + k_trunc_children)": ("evolve", 6 * N * J * 4),
                        "k_fitness over the 3N new rows": ("fitness", 3 * N * (4 * J + 12))}
            else:  # 3N children written and scored in one pass: 3N row reads, 3N row writes, (F, G) of each
                rows = {"children + scores (k_trunc_draws + k_trunc_children_score)": ("evolve", 6 * N * J * 4 + 3 * N * 12)}
            rows["selection (radix threshold, compaction, k_trunc_gather)"] = ("select", 2 * N * J * 4 + 4 * N * 8 * 10)
            line["kernels"] = {}
            for name, (stage, nbytes) in rows.items():
                t_ms = stage_ms[stage] / stage_n[stage]
                a = nbytes / (t_ms * 1e-3) / 1e9
                line["kernels"][name] = {"bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                                         "bytes_per_generation": nbytes, "ms_per_generation": t_ms}
            dom = max(line["kernels"].items(), key=lambda kv: kv[1]["ms_per_generation"])
            line["roofline"] = dict(dom[1], kernel=dom[0], peak_kind=f"of {peak_kind}", traffic=None)
    if stage_n.get("evolve") and args.scheme == "tournament":
        ev_ms = stage_ms["evolve"] / stage_n["evolve"]
        sel_ms = stage_ms["select"] / stage_n["select"] if stage_n.get("select") else 0.0
        # algorithmic bytes per launch: one parent-row read and one child-row write per child gene (8 B),
        # the elite rows, the pair/elite indices, and F and G of every candidate (scored in the same kernel)
        evolve_bytes = 8 * J * (N - E) + 8 * J * E + 8 * ((N - E + 1) // 2) + 4 * E
        fused_bytes = evolve_bytes + 12 * N
        ach = fused_bytes / (ev_ms * 1e-3) / 1e9
        gens_per_launch = steps if launches < steps else 1  # the cluster path runs a whole call in one launch
        one_launch = launches <= steps
        kernel = "k_evolve_cluster" if launches < steps else ("k_generation" if one_launch else "k_evolve_score")
        ach = fused_bytes * gens_per_launch / (ev_ms * 1e-3) / 1e9
        line["roofline"] = {"kernel": kernel, "bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s",
                            "frac": ach / peak, "peak_kind": f"of {peak_kind}",
                            "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((w.name, N, kernel)),
                            "bytes_per_launch": fused_bytes * gens_per_launch, "ms_per_launch": ev_ms,
                            "generations_per_launch": gens_per_launch,
                            "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                            "note": "crossover + mutation + scoring of the children in one pass (dominant kernel of the "
                                    "generation); shapes that fit one cluster's shared memory are latency-bound, their "
                                    "fraction of the HBM rate is informational; the unfused kernels are under 'kernels'"}
        line["kernels"] = {"k_select_stage": {"ms_per_launch": sel_ms}} if sel_ms else {}
        if sep is not None:
            sep_ms, sep_n = sep
            e_ms = sep_ms["evolve"] / sep_n["evolve"]
            f_ms = sep_ms["fitness"] / sep_n["fitness"]
            fitness_bytes = 4 * J * N + 12 * N
            for name, nbytes, t_ms in (("k_evolve", evolve_bytes, e_ms), ("k_fitness", fitness_bytes, f_ms)):
                a = nbytes / (t_ms * 1e-3) / 1e9
                line["kernels"][name] = {"bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                                         "bytes_per_launch": nbytes, "ms_per_launch": t_ms,
                                         "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((w.name, N, name)),
                                         "frac_of_nominal_8TBs": a / NOMINAL_HBM_GBS,
                                         "how": "same workload with ONES_FLAG_UNFUSED (separate scoring pass)"}
            a = packed_bytes / (packed_ms * 1e-3) / 1e9
            line["kernels"]["k_fitness_packed"] = {
                "bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                "bytes_per_launch": packed_bytes, "ms_per_launch": packed_ms, "frac_of_nominal_8TBs": a / NOMINAL_HBM_GBS,
                "candidate_evals_per_s": N / (packed_ms * 1e-3),
                "how": "ones_evaluate_packed on the same population stored as one byte per gene (a variant beside the "
                       "int32 contract); 20 launches back to back, two packed copies read in turn"}
    if base is not None:
        line["cpu_baseline"] = base
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
