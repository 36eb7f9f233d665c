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
def host_info():
    """The host the CPU figures were taken on: logical cores and the CPU model string."""
    model = "unknown"
    try:
        with open("/proc/cpuinfo") as fh:
            for ln in fh:
                if ln.lower().startswith(("model name", "cpu model", "cpu\t")):
                    model = ln.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"host_cores": os.cpu_count(), "host_cpu": model}


def oracle_search(w, pop_sample: int):
    """An oracle handle over a `pop_sample`-candidate population, randomised and scored (set-up, not timed)."""
    import oracle
    p = w.params
    s = oracle.Search(w.jobs, w.capacity, pop_sample, elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut,
                      penalty=p.penalty, flags=p.flags)
    s.randomize(w.seed)
    s.evaluate()
    return s


def oracle_sample(w, pop_sample: int, gens: int):
    """Seconds for `gens` generations of a `pop_sample`-candidate population (single thread)."""
    s = oracle_search(w, pop_sample)
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
    if gens is None:  # about 3e8 gene evaluations: 10-20 s of single-thread work
        gens = int(min(2000, max(8, 3e8 / (pop_sample * w.n_jobs))))
    dt = oracle_sample(w, pop_sample, gens)
    return dict({"value": pop_sample * gens / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                 "sample": f"{gens} generations of a {pop_sample}-candidate population (of {w.pop}), "
                           f"{w.n_jobs} jobs, same job table and parameters; {dt:.1f} s"}, **host_info())


def run_reference(args, w):
    """The reference arm: the CPU oracle as it stands; each step is one generation of a bounded sample of the
    population.  Handle creation, the random initial population and its first scoring are set-up and stay
    outside the clock, as they do in the GPU arm and in `cpu_baseline`."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    pop_sample = min(8192, w.pop)
    s = oracle_search(w, pop_sample)
    warm = min(max(args.warmup, 0), 5)
    s.evolve(warm, w.seed)
    steps = max(1, min(args.steps, 40))
    t0 = time.perf_counter()
    s.evolve(steps, w.seed)
    dt = time.perf_counter() - t0
    s.close()
    value = pop_sample * steps / dt
    sample = (f"each step = 1 generation of a {pop_sample}-candidate population (of {w.pop}), {w.n_jobs} jobs, "
              f"single thread; {steps} steps timed (capped at 40), {warm} warm-up (capped at 5)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": 1e3 * dt / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, max(args.gpus, 1)),
            "cpu_baseline": dict({"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
                                 **host_info()),
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# online loop: per-round search latency and simulated job completion time
# ----------------------------------------------------------------------------------------------
def online_figures(oracle_rounds: int):
    """The 2000-job trace through the library (every round), and its first `oracle_rounds` rounds through the
    CPU oracle (0: skipped).  Returns the figures of the online workload as a dict."""
    import torch
    from paper_2108_03645_b200 import binding, online

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
    out = {"what": "ones_update_jobs + 50 generations of a 4096-candidate population + ones_best with repair, per "
                   "60 s scheduling round of the 2000-job trace on 256 GPUs (host wall clock around the three calls)",
           "rounds": res.rounds, "mean_ms": float(lat.mean()), "p50_ms": float(np.percentile(lat, 50)),
           "p99_ms": float(np.percentile(lat, 99)), "max_ms": float(lat.max()),
           "mean_active_jobs": float(np.mean(res.active)), "max_active_jobs": int(max(res.active)),
           "mean_jct_s": res.mean_jct, "jobs_finished": int(np.isfinite(res.jct).sum()),
           "trace_jobs": int(trace.jobs.shape[0]), "capacity": trace.capacity, "population": trace.pop,
           "generations_per_round": trace.generations, "period_s": trace.period_s}
    if oracle_rounds > 0:
        t0 = time.perf_counter()
        ref = online.simulate(trace, cpu_engine, max_rounds=oracle_rounds, keep_schedules=True)
        dt = time.perf_counter() - t0
        same = len(ref.deployed) == min(oracle_rounds, res.rounds) and all(
            ra == rb and ia == ib and (ga == gb).all() for (ra, ia, ga), (rb, ib, gb) in zip(res.deployed, ref.deployed))
        same = same and ref.best_fitness == res.best_fitness[:len(ref.best_fitness)]
        out["cpu_oracle"] = dict({"mean_ms": 1e3 * float(np.mean(ref.latency_s)), "rounds": ref.rounds, "cores": 1,
                                  "kind": "oracle", "sample": f"first {ref.rounds} rounds of the same trace; {dt:.1f} s",
                                  "schedules_identical_to_gpu": bool(same)}, **host_info())
    return out


def run_online(args):
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    f = online_figures(0 if args.no_cpu_baseline else 100)
    line = {"metric": "online_round_latency_ms", "value": f["mean_ms"], "unit": "ms per scheduling round "
            "(ones_update_jobs + 50 generations of a 4096-candidate population + ones_best with repair)",
            "n_gpus": 1, "higher_is_better": False, "data": "synthetic", "dtype": "f64",
            "config": {"workload": "online", "trace_jobs": f["trace_jobs"], "capacity": f["capacity"],
                       "population": f["population"], "generations_per_round": f["generations_per_round"],
                       "period_s": f["period_s"]},
            "rounds": f["rounds"], "p50_ms": f["p50_ms"], "p99_ms": f["p99_ms"], "max_ms": f["max_ms"],
            "mean_active_jobs": f["mean_active_jobs"], "max_active_jobs": f["max_active_jobs"],
            "mean_jct_s": f["mean_jct_s"], "jobs_finished": f["jobs_finished"]}
    if "cpu_oracle" in f:
        c = f["cpu_oracle"]
        line["cpu_baseline"] = dict(c, value=c["mean_ms"], unit="ms per scheduling round")
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# timing helpers
# ----------------------------------------------------------------------------------------------
def timed_repeats(run_steps, min_s: float, max_repeats: int = 4000):
    """Time `run_steps()` (which enqueues exactly K steps on the current stream) repeatedly: one untimed
    call sizes the repeat count so that the timed region lasts at least `min_s`, then every repeat is
    bracketed by its own pair of CUDA events.  Returns the per-repeat milliseconds."""
    import torch
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    run_steps()
    torch.cuda.synchronize()
    once = max(time.perf_counter() - t0, 1e-6)
    repeats = int(min(max_repeats, max(3, np.ceil(min_s / once))))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(repeats)]
    for e0, e1 in evs:
        e0.record()
        run_steps()
        e1.record()
    torch.cuda.synchronize()
    return [e0.elapsed_time(e1) for e0, e1 in evs]


def small_workload_figures(binding, name: str, min_s: float = 0.25):
    """Generations/s of one of the cache-resident workloads: repeats of its own generation count."""
    w = inputs.WORKLOADS[name]()
    s = binding.Search(w.jobs, w.capacity, w.pop, w.params)
    s.randomize(w.seed)
    s.evolve(w.generations, w.seed)
    l0 = s.kernel_launches
    ms = timed_repeats(lambda: s.evolve(w.generations, w.seed), min_s)
    launches = (s.kernel_launches - l0) / (len(ms) + 1)
    per_gen_ms = statistics.median(ms) / w.generations
    s.close()
    return {"jobs": w.n_jobs, "population": w.pop, "generations_per_call": w.generations,
            "us_per_generation": 1e3 * per_gen_ms, "generations_per_s": 1e3 / per_gen_ms,
            "candidate_evals_per_s": w.pop * 1e3 / per_gen_ms, "launches_per_call": launches,
            "timed_calls": len(ms), "hbm": "n/a (population resident in L2 or shared memory)"}


# The functions whose source the traffic figures below belong to: the five timed kernels and the device
# functions they call.  Their text (definition line to closing brace) is hashed, so that an edit elsewhere in the
# kernel file does not orphan the capture and an edit to any of them does.
TRAFFIC_FUNCTIONS = ("philox", "draw_gene", "slot_of", "sibling_gene", "sibling_int4", "ld_row", "ld_row_hint",
                     "l2_policy_evict_last", "l2_prefetch", "score4", "k_fitness", "k_fitness_packed", "k_evolve",
                     "mutate_gene", "sibling_pair", "score_int4", "k_evolve_score", "mutate_byte", "score_gene",
                     "score_word", "k_evolve_score_packed", "launch_evolve_score", "launch_evolve_score_packed",
                     "launch_evolve", "launch_fitness", "launch_fitness_packed")


def sha16(path: str) -> str:
    """Hash of the source text of TRAFFIC_FUNCTIONS in `path`; raises when one of them cannot be found."""
    import hashlib
    import re
    with open(path, "r", encoding="utf-8") as fh:
        text = fh.read()
    h = hashlib.sha256()
    for name in TRAFFIC_FUNCTIONS:
        # a definition: the name at the start of a line or after the return type, followed by its parameter list
        # and, later, a brace at the start of a line that closes it
        m = re.search(r"^(?:[^\n;{}()]*[ \*&])?" + re.escape(name) + r"\(", text, flags=re.M)
        if not m:
            raise OSError(f"{name}: definition not found")
        end = text.find("\n}\n", m.start())
        if end < 0:
            raise OSError(f"{name}: end not found")
        h.update(text[m.start():end + 3].encode())
    return h.hexdigest()[:16]


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from one ncu capture of this
# benchmark's default workload at its full population.  A figure belongs to the source it was captured on:
# `source_sha16` is sha16() of the kernel file at commit `captured_at` (the timed kernels, their device functions
# and their launchers), and the benchmark reports traffic as null whenever the file it runs gives another hash.
NCU_TRAFFIC = {
    "captured_at": "2810ec6",
    "source_sha16": "3a974a5302ea4351",
    "bytes_per_launch": {
        ("large", 65536, "k_evolve_score"): 379.4e6 + 481.2e6,
        ("large", 65536, "k_evolve"): 375.3e6 + 479.2e6,
        ("large", 65536, "k_fitness"): 537.1e6 + 0.7e6,
        ("large", 65536, "k_evolve_score_packed"): 45.3e6 + 73.7e6,
        ("large", 65536, "k_fitness_packed"): 134.5e6 + 0.3e6,
    },
}
KERNEL_SOURCE = os.path.join(ROOT, "paper_2108_03645_b200", "csrc", "ones_kernels.cu")


def ncu_traffic(workload: str, pop: int, kernel: str):
    """(bytes per launch or None, commit of the capture)."""
    try:
        current = sha16(KERNEL_SOURCE)
    except OSError:
        current = None
    if current != NCU_TRAFFIC["source_sha16"]:
        return None, NCU_TRAFFIC["captured_at"]
    return NCU_TRAFFIC["bytes_per_launch"].get((workload, pop, kernel)), NCU_TRAFFIC["captured_at"]


def roofline_entry(kernel, nbytes, t_ms, peak, peak_kind, traffic, captured_at, **more):
    """HBM roofline of one kernel: `achieved` counts the algorithmic bytes; where an ncu capture of the DRAM
    bytes of this very kernel exists, the rate on those bytes is reported beside it (`dram_*`)."""
    a = nbytes / (t_ms * 1e-3) / 1e9
    r = {"kernel": kernel, "bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
         "peak_kind": f"of {peak_kind}", "traffic": traffic, "traffic_captured_at": captured_at,
         "bytes_per_launch": nbytes, "ms_per_launch": t_ms, "frac_of_nominal_8TBs": a / NOMINAL_HBM_GBS}
    if traffic:
        d = traffic / (t_ms * 1e-3) / 1e9
        r.update({"dram_achieved": d, "dram_frac": d / peak, "dram_frac_of_nominal_8TBs": d / NOMINAL_HBM_GBS})
    r.update(more)
    return r


def config_of(w, world: int):
    return {"workload": w.name, "jobs": w.n_jobs, "population": w.pop, "capacity": w.capacity,
            "elitism": w.params.elitism, "tournament": w.params.tournament, "p_mut": w.params.p_mut,
            "genome_table_bytes": w.pop * w.n_jobs * 4,
            "l2": "inputs larger than L2 (two population buffers of genome_table_bytes each against 126 MB)"
                  if w.pop * w.n_jobs * 4 > 2 * 126e6 else "population fits L2: cache-resident",
            "parallelism": "replicas" if world > 1 else "single GPU"}


# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=sorted(inputs.WORKLOADS) + ["online"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-events", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the figures of the other workloads")
    ap.add_argument("--min-seconds", type=float, default=0.5,
                    help="the K timed steps are repeated until the timed region lasts this long")
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
    solo = rank == 0 and world == 1

    base = cpu_baseline(w) if (solo and not args.no_cpu_baseline) else None

    seed = rank_seed(w.seed, rank)
    s = binding.Search(w.jobs, w.capacity, w.pop, w.params)
    s.randomize(seed)
    s.evolve(warmup, seed)
    torch.cuda.synchronize()

    # ---- device-resident timed region: repeats of exactly K generations, each repeat between its own
    # pair of CUDA events on the handle's stream; no per-kernel events are recorded inside it ----
    sampler = ClockSampler(local, period_s=0.002)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = s.kernel_launches
    sampler.start()
    t_wall = time.perf_counter()
    rep_ms = timed_repeats(lambda: s.evolve(steps, seed), args.min_seconds)
    torch.cuda.synchronize()
    timed_region_s = time.perf_counter() - t_wall
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    launches = (s.kernel_launches - launches0) / (len(rep_ms) + 1)  # per K steps (one untimed sizing call)
    ms = max_over_ranks(statistics.median(rep_ms), "cuda")

    # ---- per-kernel durations: a separate pass with an event pair around every kernel ----
    stage_ms, stage_n = ({}, {})
    if not args.no_kernel_events:
        s.set_profiling(1)
        s.stage_times()
        s.evolve(max(steps, 100) if w.pop * w.n_jobs >= (1 << 24) else steps, seed)
        stage_ms, stage_n = s.stage_times()
        s.set_profiling(False)

    # ---- end to end: every step uploads the job table and reads the best schedule back ----
    J, N, E = w.n_jobs, w.pop, w.params.elitism
    identity = np.arange(J, dtype=np.int32)
    jobs_pinned = torch.from_numpy(w.jobs.view(np.uint8).reshape(-1).copy()).pin_memory()
    jobs_host = jobs_pinned.numpy().view(inputs.JOB_DTYPE)
    # two job tables that differ in their coefficients (what a round's progress report changes), taken in turn:
    # every step rebuilds the model tables and scores the population under them
    jobs_alt = w.jobs.copy()
    jobs_alt["a"] *= 1.0 + 2.0 ** -20
    jobs_pinned2 = torch.from_numpy(jobs_alt.view(np.uint8).reshape(-1).copy()).pin_memory()
    tables = [jobs_host, jobs_pinned2.numpy().view(inputs.JOB_DTYPE)]
    out = {"fitness": None}
    e2e_ms, e2e_reps = float("nan"), 0
    if not args.no_e2e:
        def e2e_steps():
            for i in range(steps):
                s.update_jobs(tables[(i + 1) & 1], identity, w.capacity)
                s.evolve(1, seed)
                out.update(s.best(False))
        e2e_steps()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        reps = []
        t_all = time.perf_counter()
        while len(reps) < 3 or (time.perf_counter() - t_all < 0.6 * args.min_seconds and len(reps) < 500):
            t0 = time.perf_counter()
            e2e_steps()  # ones_best synchronises: the host clock brackets the device work
            reps.append(time.perf_counter() - t0)
        e2e_ms = max_over_ranks(1e3 * statistics.median(reps), "cuda")
        e2e_reps = len(reps)
    h2d = J * 48  # the job rows (the column map stays on the host when every job keeps its column)
    d2h = J * (4 + 4 + 8) + 64

    # ---- the two separate kernels (crossover/mutation, fitness) on the same workload ----
    sep = None
    if solo and not args.no_kernel_events and args.scheme == "tournament":
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
        s2.evolve(min(max(steps, 50), 200), seed)
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
        del s2
        torch.cuda.empty_cache()

    # ---- the generation on one-byte genes (ONES_FLAG_PACKED): a variant beside the int32 contract ----
    packed_gen = None
    if solo and not args.no_kernel_events and args.scheme == "tournament":
        import dataclasses
        p3 = dataclasses.replace(w.params, flags=w.params.flags | binding.FLAG_PACKED)
        s3 = binding.Search(w.jobs, w.capacity, w.pop, p3)
        s3.randomize(seed)
        s3.evolve(warmup, seed)
        rep3 = timed_repeats(lambda: s3.evolve(steps, seed), 0.5 * args.min_seconds)
        s3.set_profiling(1)
        s3.stage_times()
        s3.evolve(max(steps, 50), seed)
        ms3, n3 = s3.stage_times()
        s3.set_profiling(False)
        packed_gen = (statistics.median(rep3) / steps, ms3["evolve"] / n3["evolve"], ms3["select"] / n3["select"], len(rep3))
        s3.close()
        del s3
        torch.cuda.empty_cache()

    # ---- the other workloads, measured in the same run ----
    others = None
    if solo and not args.no_workloads and args.scheme == "tournament" and not args.pop:
        others = {name: small_workload_figures(binding, name) for name in ("tiny", "paper", "mid") if name != w.name}
        others["online"] = online_figures(0 if args.no_cpu_baseline else 100)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    line = {
        "metric": METRIC, "value": whole_job_rate(world, N, steps, ms), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, world),
        "generations_per_s": world * steps / (ms * 1e-3),
        "gpu_launches": int(round(launches)),
        "timing": {"timed_repeats": len(rep_ms), "steps_per_repeat": steps, "ms_per_repeat_median": ms,
                   "ms_per_repeat_min": min(rep_ms), "ms_per_repeat_max": max(rep_ms),
                   "timed_region_s": timed_region_s,
                   "how": "the K steps are repeated back to back until the timed region lasts --min-seconds; each "
                          "repeat has its own CUDA-event pair on the launching stream, the median repeat is reported; "
                          "per-kernel events are recorded in a separate pass afterwards"},
        "clocks": clocks,
        "e2e": None if not e2e_reps else {
            "value": world * N * steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "ms_per_step": e2e_ms / steps, "timed_repeats": e2e_reps,
            "what": "per step: ones_update_jobs(host job table; two tables with different coefficients in turn, same "
                    "jobs in the same columns) + ones_evolve(1) + ones_best(host outputs); host wall clock, median repeat",
            "best_fitness": out["fitness"]},
    }
    if args.scheme == "per_gpu":
        Wg = w.capacity
        line["config"]["scheme"] = f"per-GPU genome: {Wg} slots per candidate, reorder after crossover and mutation"
        if stage_n.get("evolve"):
            rows = {"k_evolve": ("evolve", 8 * Wg * N),
                    "k_per_gpu<reorder, score>": ("fitness", N * (8 * Wg + 12)),
                    "k_select_stage": ("select", 8 * N)}
            line["kernels"] = {}
            for name, (stage, nbytes) in rows.items():
                line["kernels"][name] = roofline_entry(name, nbytes, stage_ms[stage] / stage_n[stage], peak, peak_kind,
                                                       None, None)
            dom = max(line["kernels"].values(), key=lambda kv: kv["ms_per_launch"])
            line["roofline"] = dict(dom)
    if args.scheme == "truncation":
        line["config"]["scheme"] = "truncation: pool of 4N rows, 3N new candidates scored per generation"
        line["new_candidates_per_s"] = 3 * line["value"]
        if stage_n.get("evolve"):
            if stage_n.get("fitness"):  # children written first, scored by a separate pass
                rows = {"children (k_trunc_draws + k_trunc_children)": ("evolve", 6 * N * J * 4),
                        "k_fitness over the 3N new rows": ("fitness", 3 * N * (4 * J + 12))}
            else:  # 3N children written and scored in one pass: 3N row reads, 3N row writes, (F, G) of each
                rows = {"children + scores (k_trunc_children_score)": ("evolve", 6 * N * J * 4 + 3 * N * 12)}
            if launches == 2 * steps:
                # fused handle: the pool is used in place, one cluster launch finds the threshold, the survivors'
                # places and the new row map (scores, GPU counts and the map: no candidate row moves)
                rows["selection in place (k_trunc_pick_place: threshold, places, row map)"] = \
                    ("select", 4 * N * 8 + N * 12 * 2 + 4 * N * 4 * 2)
            else:
                rows["selection (threshold search, compaction, k_trunc_gather)"] = ("select", 2 * N * J * 4 + 4 * N * 8 * 3)
            line["kernels"] = {}
            for name, (stage, nbytes) in rows.items():
                line["kernels"][name] = roofline_entry(name, nbytes, stage_ms[stage] / stage_n[stage], peak, peak_kind,
                                                       None, None)
            dom = max(line["kernels"].values(), key=lambda kv: kv["ms_per_launch"])
            line["roofline"] = dict(dom)
    if stage_n.get("evolve") and args.scheme == "tournament":
        ev_ms = stage_ms["evolve"] / stage_n["evolve"]
        sel_ms = stage_ms["select"] / stage_n["select"] if stage_n.get("select") else 0.0
        # algorithmic bytes per launch: one parent-row read and one child-row write per child gene (8 B),
        # the elite rows, the pair/elite indices, and F and G of every candidate (scored in the same kernel)
        evolve_bytes = 8 * J * (N - E) + 8 * J * E + 8 * ((N - E + 1) // 2) + 4 * E
        fused_bytes = evolve_bytes + 12 * N
        gens_per_launch = steps if launches < steps else 1  # the cluster path runs a whole call in one launch
        one_launch = launches <= steps
        kernel = "k_evolve_cluster" if launches < steps else ("k_generation" if one_launch else "k_evolve_score")
        traffic, at = ncu_traffic(w.name, N, kernel)
        line["roofline"] = roofline_entry(
            kernel, fused_bytes * gens_per_launch, ev_ms, peak, peak_kind, traffic, at,
            generations_per_launch=gens_per_launch,
            note="crossover + mutation + scoring of the children in one pass (dominant kernel of the generation), timed "
                 "with an event pair around every launch in a pass of its own; shapes that fit one cluster's shared "
                 "memory are latency-bound, their fraction of the HBM rate is informational; the unfused kernels are "
                 "under 'kernels'")
        line["kernels"] = {"k_select_stage": {"ms_per_launch": sel_ms}} if sel_ms else {}
        if sep is not None:
            sep_ms, sep_n = sep
            e_ms = sep_ms["evolve"] / sep_n["evolve"]
            f_ms = sep_ms["fitness"] / sep_n["fitness"]
            fitness_bytes = 4 * J * N + 12 * N
            for name, nbytes, t_ms in (("k_evolve", evolve_bytes, e_ms), ("k_fitness", fitness_bytes, f_ms)):
                traffic, at = ncu_traffic(w.name, N, name)
                line["kernels"][name] = roofline_entry(name, nbytes, t_ms, peak, peak_kind, traffic, at,
                                                       how="same workload with ONES_FLAG_UNFUSED (separate scoring pass)")
            line["kernels"]["k_fitness_packed"] = roofline_entry(
                "k_fitness_packed", packed_bytes, packed_ms, peak, peak_kind, *ncu_traffic(w.name, N, "k_fitness_packed"),
                candidate_evals_per_s=N / (packed_ms * 1e-3),
                how="ones_evaluate_packed on the same population stored as one byte per gene (a variant beside the "
                    "int32 contract); 20 launches back to back, two packed copies read in turn")
    if packed_gen is not None and "kernels" in line:
        gen_ms, k_ms, sel_ms3, reps3 = packed_gen
        # one parent byte read and one child byte written per child gene, the elite rows, indices, F and G
        pbytes = 2 * J * (N - E) + 2 * J * E + 8 * ((N - E + 1) // 2) + 4 * E + 12 * N
        line["kernels"]["k_evolve_score_packed"] = roofline_entry(
            "k_evolve_score_packed", pbytes, k_ms, peak, peak_kind, *ncu_traffic(w.name, N, "k_evolve_score_packed"),
            ms_per_generation=gen_ms, generations_per_s=1e3 / gen_ms, candidate_evals_per_s=N * 1e3 / gen_ms,
            timed_repeats=reps3,
            how="same workload on a handle with ONES_FLAG_PACKED (population kept as one byte per gene; identical "
                "children, scores and selections): ms_per_generation from repeats of the K steps without per-kernel "
                "events, ms_per_launch from an event pass of its own")
    if others is not None:
        line["workloads"] = others
    if base is not None:
        line["cpu_baseline"] = base
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
