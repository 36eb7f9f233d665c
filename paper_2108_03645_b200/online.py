"""Online scheduling loop around a search engine (host-side event simulation).

Every `period_s` simulated seconds the set of running jobs is rebuilt (arrived and
unfinished, in arrival order), the engine's population is carried over to the new
job set (`update_jobs`: finished jobs' columns dropped, new jobs at their smallest
batch), `generations` generations are run and the best schedule, repaired to the
cluster's capacity, is deployed until the next round (paper, Section 3.2.2
"Refresh" and "Update"; batch-size limit policies "Start" and "Scale-up" of
Section 3.3.3: a job is held at its smallest batch in its first round and its
limit doubles every round after that).

The simulator is engine-agnostic: it only calls `update_jobs`, `evolve` and `best`
on the object `make_engine` returns, and does no scoring of its own; job progress
between rounds uses the per-job throughput the engine reports for the deployed
schedule.
"""
from __future__ import annotations

import time
from dataclasses import dataclass, field

import numpy as np

from .inputs import JOB_DTYPE, Trace


def sruf_weights(y_processed, alpha, beta, rng: np.random.Generator) -> np.ndarray:
    """Per-job weights for the ONES_FLAG_SRUF score of one scheduling round.

    Alg. 1 draws one progress sample rho_j ~ Be(alpha_j, beta_j) per job, shared by every
    candidate of the round; Eq. 7 turns it into the remaining workload
    Y_j = Y_processed,j * (1/rho_j - 1), which is the job's weight in the score
    sum_j Y_j * c_j / X_j (Eq. 8).  alpha, beta >= 1 come from the caller's progress predictor.
    """
    y = np.asarray(y_processed, dtype=np.float64)
    a = np.maximum(np.asarray(alpha, dtype=np.float64), 1.0)
    b = np.maximum(np.asarray(beta, dtype=np.float64), 1.0)
    rho = np.clip(rng.beta(a, b), 1e-12, 1.0)
    return y * (1.0 / rho - 1.0)


@dataclass
class OnlineResult:
    jct: np.ndarray                 # seconds from arrival to completion, per job (nan if unfinished)
    rounds: int                     # search rounds run
    latency_s: list = field(default_factory=list)   # wall seconds of update + evolve + best, per round
    gpus_used: list = field(default_factory=list)   # GPU demand of the deployed schedule, per round
    active: list = field(default_factory=list)      # number of running jobs, per round
    best_fitness: list = field(default_factory=list)
    deployed: list = field(default_factory=list)    # (round, job ids, genome) when keep_schedules

    @property
    def mean_jct(self) -> float:
        return float(np.nanmean(self.jct))


def simulate(trace: Trace, make_engine, *, max_rounds: int | None = None, kmax_cap: int = 7,
             n_jobs_max: int = 256, keep_schedules: bool = False, sync=None) -> OnlineResult:
    """Run the online loop over `trace`.

    make_engine(jobs, capacity, pop, params, n_jobs_max) -> engine with
    update_jobs(jobs, remap, capacity), evolve(generations, seed), best(repair=True).
    `sync` (optional) is called before each latency timestamp (e.g. a device synchronise).
    """
    n = trace.jobs.shape[0]
    remaining = trace.length.astype(np.float64).copy()
    first_round = np.full(n, -1, dtype=np.int64)   # round in which the job was first scheduled
    done_at = np.full(n, np.nan)
    res = OnlineResult(jct=np.full(n, np.nan), rounds=0)
    engine = None
    prev_ids: list[int] = []
    rnd = 0
    t = 0.0
    arrival = trace.arrival_s
    while True:
        if max_rounds is not None and res.rounds >= max_rounds:
            break
        unfinished = np.isnan(done_at)
        if not unfinished.any():
            break
        ids = [int(j) for j in np.nonzero(unfinished & (arrival <= t))[0]]
        if not ids:
            # idle cluster: jump to the first round at or after the next arrival
            nxt = float(arrival[unfinished].min())
            rnd = max(rnd + 1, int(np.ceil(nxt / trace.period_s)))
            t = rnd * trace.period_s
            continue
        jobs = trace.jobs[ids].copy()
        for c, j in enumerate(ids):
            if first_round[j] < 0:
                first_round[j] = rnd
            jobs["kmin"][c] = 0
            jobs["kmax"][c] = min(kmax_cap, rnd - first_round[j], int(trace.jobs["kmax"][j]))
        where = {j: c for c, j in enumerate(prev_ids)}
        remap = np.array([where.get(j, -1) for j in ids], dtype=np.int32)

        if sync:
            sync()
        t0 = time.perf_counter()
        if engine is None or len(ids) > n_jobs_max:
            n_jobs_max = max(n_jobs_max, 2 * len(ids))
            engine = make_engine(jobs, trace.capacity, trace.pop, trace.params, n_jobs_max)
        else:
            engine.update_jobs(jobs, remap, trace.capacity)
        engine.evolve(trace.generations, rnd)
        best = engine.best(repair=True)
        if sync:
            sync()
        res.latency_s.append(time.perf_counter() - t0)
        res.rounds += 1
        res.gpus_used.append(int(best["total_gpus"]))
        res.active.append(len(ids))
        res.best_fitness.append(float(best["fitness"]))
        if keep_schedules:
            res.deployed.append((rnd, list(ids), best["genome"].copy()))

        # deploy until the next round: job j advances at the throughput of its gene (0 if it waits)
        rate = np.asarray(best["rate_per_job"], dtype=np.float64)
        for c, j in enumerate(ids):
            if rate[c] > 0.0:
                need = remaining[j] / rate[c]
                if need <= trace.period_s:
                    done_at[j] = t + need
                    remaining[j] = 0.0
                else:
                    remaining[j] -= rate[c] * trace.period_s
        prev_ids = ids
        rnd += 1
        t = rnd * trace.period_s
    res.jct = done_at - arrival
    return res
