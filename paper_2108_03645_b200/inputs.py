"""Seeded synthetic inputs for the ONES evolutionary batch-size search.

This module only *draws data*: job tables, search parameters, random genome
tables and the arrival trace of the online loop.  It contains none of the
method's arithmetic (no throughput model, no fitness, no operators) and is the
one module that both the CUDA library's callers and the CPU oracle's callers
may import.  It must stay importable without the CUDA extension.

The five workloads follow the shapes of the search described in the paper's
Section 3.2 (a population of candidate schedules over the set of jobs J on a
cluster of |C| GPUs, Table 1) at the paper's 64-GPU scale and beyond:

====  =======  =====  ======  =====  ===  ===  =====  ====
name  jobs J   GPUs   pop N   gens   E    T    p_mut  kmax
====  =======  =====  ======  =====  ===  ===  =====  ====
tiny      16     16      32     10    2    4   0.10     5
paper    100     64    1024    100    2    4   0.10     7
mid      512    512    8192    200    2    4   0.10     7
large   2048   4096   65536    200    2    8   0.02     7
online  trace   256    4096     50    2    4   0.10   0..7
====  =======  =====  ======  =====  ===  ===  =====  ====

All draws come from ``numpy.random.Generator(PCG64(seed))`` in the order
written below, so a (workload, seed) pair always yields the same bytes.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# One row of the job table as the C ABI sees it (48 bytes, natural alignment).
JOB_DTYPE = np.dtype(
    [
        ("b0", "<i4"),           # smallest global batch size of the job
        ("max_per_gpu", "<i4"),  # largest local batch one GPU can hold
        ("kmin", "<i4"),         # lowest admissible exponent
        ("kmax", "<i4"),         # highest admissible exponent (batch limit R_j = b0 << kmax)
        ("a", "<f8"),            # seconds per iteration, fixed part
        ("c", "<f8"),            # seconds per sample
        ("d", "<f8"),            # seconds per doubling of the worker count
        ("weight", "<f8"),       # per-job weight (1.0 unless the caller sets it)
    ],
    align=True,
)
assert JOB_DTYPE.itemsize == 48


@dataclass(frozen=True)
class SearchParams:
    """Search hyper-parameters (same fields as the C ABI's ``ones_params``)."""

    elitism: int = 2
    tournament: int = 4
    p_mut: float = 0.1
    penalty: float = 1e3
    flags: int = 0


@dataclass(frozen=True)
class Workload:
    name: str
    jobs: np.ndarray          # JOB_DTYPE[J]
    capacity: int             # |C|
    pop: int                  # N
    generations: int          # G
    params: SearchParams
    seed: int = 0             # seed handed to randomize()/evolve()
    extra: dict = field(default_factory=dict)

    @property
    def n_jobs(self) -> int:
        return int(self.jobs.shape[0])


def _draw_jobs(rng: np.random.Generator, n_jobs: int, kmax: int, *,
               log_uniform: bool, m_choices, pinned: int = 0) -> np.ndarray:
    """Draw ``n_jobs`` rows.  Order of draws: b0, max_per_gpu, a, c, d, pinned set."""
    jobs = np.zeros(n_jobs, dtype=JOB_DTYPE)
    jobs["b0"] = rng.choice(np.array([32, 64, 128], dtype=np.int32), size=n_jobs)
    jobs["max_per_gpu"] = rng.choice(np.asarray(m_choices, dtype=np.int32), size=n_jobs)
    if log_uniform:
        # two decades each, centred on the uniform ranges of the small workloads
        jobs["a"] = 10.0 ** rng.uniform(np.log10(0.005), np.log10(0.5), size=n_jobs)
        jobs["c"] = 10.0 ** rng.uniform(np.log10(1e-5), np.log10(1e-3), size=n_jobs)
        jobs["d"] = 10.0 ** rng.uniform(np.log10(0.002), np.log10(0.2), size=n_jobs)
    else:
        jobs["a"] = rng.uniform(0.01, 0.05, size=n_jobs)
        jobs["c"] = rng.uniform(1e-4, 1e-3, size=n_jobs)
        jobs["d"] = rng.uniform(0.005, 0.02, size=n_jobs)
    jobs["kmin"] = 0
    jobs["kmax"] = kmax
    jobs["weight"] = 1.0
    if pinned:
        # just-arrived jobs: held at their smallest batch (kmin = kmax = 0)
        who = rng.choice(n_jobs, size=pinned, replace=False)
        jobs["kmax"][who] = 0
    return jobs


_POW2_32_1024 = [32, 64, 128, 256, 512, 1024]


def tiny(seed: int = 0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    jobs = _draw_jobs(rng, 16, 5, log_uniform=False, m_choices=[64, 128, 256])
    return Workload("tiny", jobs, 16, 32, 10, SearchParams(2, 4, 0.1, 1e3), seed)


def paper_scale(seed: int = 0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    jobs = _draw_jobs(rng, 100, 7, log_uniform=False, m_choices=[64, 128, 256], pinned=20)
    return Workload("paper", jobs, 64, 1024, 100, SearchParams(2, 4, 0.1, 1e3), seed)


def mid(seed: int = 0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    jobs = _draw_jobs(rng, 512, 7, log_uniform=True, m_choices=_POW2_32_1024)
    return Workload("mid", jobs, 512, 8192, 200, SearchParams(2, 4, 0.1, 1e3), seed)


def large(seed: int = 0) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    jobs = _draw_jobs(rng, 2048, 7, log_uniform=True, m_choices=_POW2_32_1024)
    return Workload("large", jobs, 4096, 65536, 200, SearchParams(2, 8, 0.02, 1e3), seed)


def custom(n_jobs: int, capacity: int, pop: int, generations: int, *, seed: int = 0,
           kmax: int = 7, log_uniform: bool = False, pinned: int = 0,
           params: SearchParams | None = None, pow2: bool = True, kmin_max: int = 0) -> Workload:
    """A workload of arbitrary shape (ragged J, odd N, ...) for edge-case tests.

    ``pow2=False`` draws b0 and max_per_gpu from values that are not powers of
    two, so GPU counts are not powers of two either.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    m_choices = [64, 128, 256] if pow2 else [48, 96, 160, 224]
    jobs = _draw_jobs(rng, n_jobs, kmax, log_uniform=log_uniform, m_choices=m_choices,
                      pinned=pinned)
    if not pow2:
        jobs["b0"] = rng.choice(np.array([24, 40, 72, 100], dtype=np.int32), size=n_jobs)
    if kmin_max > 0:  # lower limits above the smallest batch (never above the job's upper limit)
        jobs["kmin"] = np.minimum(rng.integers(0, kmin_max + 1, size=n_jobs), jobs["kmax"]).astype(np.int32)
    return Workload("custom", jobs, capacity, pop, generations,
                    params or SearchParams(), seed)


WORKLOADS = {"tiny": tiny, "paper": paper_scale, "mid": mid, "large": large}


def random_genomes(jobs: np.ndarray, n: int, ld: int | None = None, seed: int = 0,
                   *, waiting_fraction: float = 0.0) -> np.ndarray:
    """``int32[n, ld]`` table of exponents, gene j uniform in [kmin_j, kmax_j].

    Padding columns (j >= J) are filled with a poison value so that a reader
    that touches them is caught.  ``waiting_fraction`` replaces that share of
    genes by -1 (a job that waits for the next schedule).
    """
    J = int(jobs.shape[0])
    ld = J if ld is None else int(ld)
    assert ld >= J
    rng = np.random.Generator(np.random.PCG64(seed ^ 0x5EED))
    lo = jobs["kmin"].astype(np.int64)[None, :]
    hi = jobs["kmax"].astype(np.int64)[None, :]
    g = np.full((n, ld), 0x7F7F7F7F, dtype=np.int32)
    g[:, :J] = rng.integers(lo, hi + 1, size=(n, J)).astype(np.int32)
    if waiting_fraction > 0.0:
        mask = rng.random((n, J)) < waiting_fraction
        g[:, :J][mask] = -1
    return g


# ---------------------------------------------------------------------------
# Online loop: arrival trace (Poisson arrivals, log-normal job lengths)
# ---------------------------------------------------------------------------

@dataclass(frozen=True)
class Trace:
    jobs: np.ndarray        # JOB_DTYPE[n]; kmax holds the final limit (7)
    arrival_s: np.ndarray   # float64[n], non-decreasing
    length: np.ndarray      # float64[n], samples to process until the job ends
    capacity: int = 256
    period_s: float = 60.0
    pop: int = 4096
    generations: int = 50
    params: SearchParams = SearchParams(2, 4, 0.1, 1e3)


def online_trace(n_jobs: int = 2000, seed: int = 0, *, mean_interarrival_s: float = 30.0,
                 median_length: float = 1e5, sigma: float = 1.5, capacity: int = 256,
                 pop: int = 4096, generations: int = 50) -> Trace:
    rng = np.random.Generator(np.random.PCG64(seed))
    jobs = _draw_jobs(rng, n_jobs, 7, log_uniform=False, m_choices=[64, 128, 256])
    gaps = rng.exponential(mean_interarrival_s, size=n_jobs)
    arrival = np.cumsum(gaps)
    length = rng.lognormal(np.log(median_length), sigma, size=n_jobs)
    return Trace(jobs, arrival, length, capacity=capacity, pop=pop, generations=generations)
