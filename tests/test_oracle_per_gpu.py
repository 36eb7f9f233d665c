"""Pins for the oracle's per-GPU genome (the paper's own encoding, Eq. 1-2) and the reorder operation."""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs
from util import example_jobs


def test_reorder_examples():
    # jobs in the order of their first occurrence, workers of a job adjacent, idle GPUs last
    assert list(oracle.reorder([2, 1, 2, 3, 1], 4)) == [2, 2, 1, 1, 3]
    assert list(oracle.reorder([0, 0, 0], 1)) == [0, 0, 0]
    assert list(oracle.reorder([-1, 3, -1, 3, 0], 4)) == [3, 3, 0, -1, -1]
    assert list(oracle.reorder([5, 9, 5], 6)) == [5, 5, -1]   # id 9 names no job: that GPU is idle
    assert list(oracle.reorder([], 3)) == []


def test_reorder_properties():
    rng = np.random.default_rng(1)
    for _ in range(50):
        W, J = int(rng.integers(1, 70)), int(rng.integers(1, 12))
        slots = rng.integers(-1, J, size=W)
        out = oracle.reorder(slots, J)
        assert sorted(out.tolist()) == sorted(slots.tolist())             # a permutation
        assert (oracle.reorder(out, J) == out).all()                      # idempotent
        seen = [j for i, j in enumerate(slots.tolist()) if j >= 0 and j not in slots[:i].tolist()]
        groups = [k for k, _ in itertools.groupby(out.tolist())]
        assert groups == seen + ([-1] if (slots < 0).any() else [])       # contiguous, first-occurrence order


def test_fitness_counts_gpus_and_picks_the_largest_batch_that_fits():
    jobs = example_jobs()  # job0: g = 1,1,2,4,8,16 for k = 0..5; job1: g = 2,4,8,16,32,64
    X = lambda j, k: oracle.model(jobs, j, k)[0]
    # job 0 on 5 GPUs -> k = 3 (4 GPUs used, one wasted); job 1 on 3 GPUs -> k = 0 (2 used)
    F, used, ks = oracle.fitness_per_gpu(jobs, [0, 0, 1, 0, 1, 0, 0, 1])
    assert list(ks) == [3, 0] and used == 6
    assert F == X(0, 3) + X(1, 0)
    # job 1 on one GPU cannot run its smallest batch (needs 2): it waits
    F, used, ks = oracle.fitness_per_gpu(jobs, [0, 1, -1, -1])
    assert list(ks) == [1, -1] and used == 1 and F == X(0, 1)
    # all idle
    assert oracle.fitness_per_gpu(jobs, [-1, -1, 7])[:2] == (0.0, 0)
    # lower limit: job 0 may not go below k = 2 (2 GPUs)
    jobs["kmin"][0] = 2
    assert list(oracle.fitness_per_gpu(jobs, [0, 1, 1, -1])[2]) == [-1, 0]
    assert list(oracle.fitness_per_gpu(jobs, [0, 0, 1, 1])[2]) == [2, 0]


def test_fitness_is_invariant_under_reorder_and_matches_the_per_job_score():
    w = inputs.paper_scale(3)
    rng = np.random.default_rng(2)
    for _ in range(10):
        slots = rng.integers(-1, w.n_jobs, size=64).astype(np.int32)
        F, used, ks = oracle.fitness_per_gpu(w.jobs, slots)
        F2, used2, ks2 = oracle.fitness_per_gpu(w.jobs, oracle.reorder(slots, w.n_jobs))
        assert F == F2 and used == used2 and (ks == ks2).all()
        assert used <= 64
        # the same schedule written as per-job exponents scores the same (no penalty: it fits)
        Fj, Gj = oracle.fitness(w.jobs, 64, 1e3, ks)
        assert Fj == F and Gj == used


def test_search_on_the_per_gpu_genome():
    w = inputs.custom(6, 12, 64, 30, seed=2, kmax=4)
    s = oracle.Search(w.jobs, w.capacity, w.pop, flags=oracle.FLAG_PER_GPU)
    P = s.get_population()
    assert P.shape == (64, 12) and (P == -1).all()       # starts with an idle cluster
    s.randomize(1)
    best = -math.inf
    for _ in range(12):
        s.evolve(1, 1)
        P = s.get_population()
        assert ((P >= -1) & (P < 6)).all()
        for row in P[:8]:
            assert (oracle.reorder(row, 6) == row).all()  # every candidate leaves a generation packed
        F, G = s.evaluate()
        assert F.max() >= best and (G <= 12).all()
        best = F.max()
    # exhaustive optimum over GPU counts per job (sum <= 12)
    opt = 0.0
    for counts in itertools.product(range(13), repeat=6):
        if sum(counts) <= 12:
            slots = [j for j, c in enumerate(counts) for _ in range(c)] + [-1] * (12 - sum(counts))
            opt = max(opt, oracle.fitness_per_gpu(w.jobs, slots)[0])
    s.evolve(40, 1)
    got = s.best()
    assert 0.9 * opt <= got["fitness"] <= opt
    assert got["total_gpus"] <= 12 and got["gpus_per_job"].sum() == got["total_gpus"]
    assert got["fitness"] == pytest.approx(math.fsum(got["rate_per_job"]), rel=1e-13)
    with pytest.raises(oracle.OracleError):
        s.update_jobs(w.jobs, np.arange(6, dtype=np.int32), 13)   # the cluster keeps its size
