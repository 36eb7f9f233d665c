"""Pins for the oracle's throughput model and fitness (CPU only)."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs
from util import example_jobs, golden_rows


def test_model_hand_values():
    jobs = example_jobs()
    rows = golden_rows("model")
    assert len(rows) == 12
    for j, k, B, g, t, frac, dec in rows:
        X, gg = oracle.model(jobs, int(j), int(k))
        assert gg == int(g)
        assert X == pytest.approx(float(Fraction(frac)), rel=1e-14)
        assert X == pytest.approx(float(dec), rel=1e-14)


def test_model_waiting_state():
    jobs = example_jobs()
    for k in (-1, -7, 6, 100):
        assert oracle.model(jobs, 0, k) == (0.0, 0)


def test_log2_of_powers_of_two_is_exact():
    # the model's log2 term must be an exact integer for power-of-two GPU counts
    for e in range(0, 31):
        assert math.log2(float(1 << e)) == float(e)
    jobs = example_jobs()
    jobs["a"] = 0.0
    jobs["c"] = 0.0
    jobs["d"] = 1.0
    # t = log2(g) alone: X = B / log2(g)
    X, g = oracle.model(jobs, 1, 3)
    assert g == 16 and X == 1024.0 / 4.0


def test_model_against_exact_rationals():
    """fp64 model vs exact arithmetic on the same binary coefficients (<= 4 roundings)."""
    w = inputs.mid(3)
    for j in range(0, w.n_jobs, 7):
        job = w.jobs[j]
        for k in range(int(job["kmax"]) + 1):
            b = int(job["b0"]) << k
            g = -(-b // int(job["max_per_gpu"]))
            assert g & (g - 1) == 0
            t = Fraction(float(job["a"])) + Fraction(float(job["c"])) * Fraction(b, g) \
                + Fraction(float(job["d"])) * (g.bit_length() - 1)
            exact = Fraction(b) / t
            X, gg = oracle.model(w.jobs, j, k)
            assert gg == g
            assert abs(Fraction(X) - exact) <= exact * Fraction(1, 10 ** 15)


def test_gpu_count_is_ceiling():
    w = inputs.custom(40, 64, 8, 1, seed=5, pow2=False)
    for j in range(w.n_jobs):
        for k in range(int(w.jobs["kmax"][j]) + 1):
            b = int(w.jobs["b0"][j]) << k
            m = int(w.jobs["max_per_gpu"][j])
            g = 0
            while g * m < b:  # smallest g with g*m >= b
                g += 1
            assert oracle.model(w.jobs, j, k)[1] == g


def test_fitness_hand_values():
    jobs = example_jobs()
    for k0, k1, cap, gpus, dec in golden_rows("fitness"):
        F, G = oracle.fitness(jobs, int(cap), 1e3, [int(k0), int(k1)])
        assert G == int(gpus)
        assert F == pytest.approx(float(dec), rel=1e-14)


def test_brute_force_optimum_matches_hand_table():
    jobs = example_jobs()
    for cap, b0, b1, gpus, dec in golden_rows("optimum"):
        best = max(itertools.product(range(6), repeat=2),
                   key=lambda ks: oracle.fitness(jobs, int(cap), 1e3, list(ks))[0])
        F, G = oracle.fitness(jobs, int(cap), 1e3, list(best))
        assert best == (int(b0), int(b1)) and G == int(gpus)
        assert F == pytest.approx(float(dec), rel=1e-14)


def test_penalty_is_per_gpu_over_capacity():
    w = inputs.tiny(1)
    g = inputs.random_genomes(w.jobs, 1, seed=2)[0]
    F_big, G = oracle.fitness(w.jobs, 10 ** 6, 1e3, g)
    for cap in (G + 3, G, G - 1, G - 5, 1):
        F, G2 = oracle.fitness(w.jobs, cap, 1e3, g)
        assert G2 == G
        assert F == pytest.approx(F_big - 1e3 * max(0, G - cap), rel=1e-15)
    # penalty coefficient scales linearly
    F2, _ = oracle.fitness(w.jobs, G - 5, 250.0, g)
    assert F2 == pytest.approx(F_big - 250.0 * 5, rel=1e-15)


@pytest.mark.parametrize("J", [1, 2, 3, 4, 5, 127, 128, 129, 300, 2048])
def test_fitness_sum_order_against_exact_sum(J):
    w = inputs.custom(J, 10 ** 6, 4, 1, seed=J, log_uniform=True)
    genomes = inputs.random_genomes(w.jobs, 4, seed=J + 1, waiting_fraction=0.1)
    for row in genomes:
        xs = [oracle.model(w.jobs, j, int(row[j])) for j in range(J)]
        exact = math.fsum(x for x, _ in xs)
        F, G = oracle.fitness(w.jobs, 10 ** 6, 1e3, row)
        assert G == sum(g for _, g in xs)
        assert F == pytest.approx(exact, rel=1e-13)
        if J <= 4:  # one partial only: plain left-to-right sum, bit for bit
            s = 0.0
            for x, _ in xs:
                s += x
            assert F == s


def test_fitness_ignores_nothing_and_reads_each_job_once():
    # moving one gene changes F by exactly that job's throughput difference
    w = inputs.paper_scale(2)
    row = inputs.random_genomes(w.jobs, 1, seed=9)[0]
    F0, G0 = oracle.fitness(w.jobs, 10 ** 6, 1e3, row)
    for j in (0, 1, 5, 63, 99):
        if w.jobs["kmax"][j] == 0:
            continue
        alt = row.copy()
        alt[j] = (row[j] + 1) % (int(w.jobs["kmax"][j]) + 1)
        F1, G1 = oracle.fitness(w.jobs, 10 ** 6, 1e3, alt)
        dx = oracle.model(w.jobs, j, int(alt[j]))[0] - oracle.model(w.jobs, j, int(row[j]))[0]
        dg = oracle.model(w.jobs, j, int(alt[j]))[1] - oracle.model(w.jobs, j, int(row[j]))[1]
        assert G1 - G0 == dg
        assert F1 - F0 == pytest.approx(dx, rel=1e-9)


def test_sruf_term():
    # Alg. 1 score term with weight = Y_processed*(1/rho - 1): weight * c_j / X_j, negated
    jobs = example_jobs()
    jobs["weight"] = [3.0e4, 7.5e3]
    t, g = oracle.term(jobs, 0, 4, oracle.FLAG_SRUF)
    assert g == 8
    assert t == pytest.approx(-3.0e4 * 8 / float(Fraction(512000, 57)), rel=1e-14)
    F, G = oracle.fitness(jobs, 64, 1e3, [4, 1], oracle.FLAG_SRUF)
    want = -(3.0e4 * 8 / float(Fraction(512000, 57)) + 7.5e3 * 4 / float(Fraction(128000, 77)))
    assert G == 12 and F == pytest.approx(want, rel=1e-14)
    # a waiting job holds no GPU and adds nothing
    assert oracle.term(jobs, 0, -1, oracle.FLAG_SRUF) == (0.0, 0)


def test_validation():
    jobs = example_jobs()
    assert oracle.validate_jobs(jobs) == 0
    for field, bad in [("b0", 0), ("max_per_gpu", -1), ("kmin", -1), ("kmax", 16), ("a", -0.1),
                       ("c", float("nan")), ("d", float("inf"))]:
        j = jobs.copy()
        j[field][1] = bad
        assert oracle.validate_jobs(j) < 0, field
    j = jobs.copy()
    j["kmin"][0] = 4
    j["kmax"][0] = 3
    assert oracle.validate_jobs(j) < 0
    j = jobs.copy()
    j["b0"][0] = 1 << 20
    j["kmax"][0] = 11  # 2^31 does not fit
    assert oracle.validate_jobs(j) < 0
    j = jobs.copy()
    j["a"][0] = j["c"][0] = j["d"][0] = 0.0  # t = 0
    assert oracle.validate_jobs(j) < 0


def test_summation_order_is_the_documented_one():
    # 2^53 next to a few ones: which ones survive the rounding depends on the order of the additions.
    # Documented order: 32 partial sums, job j to partial (j / 4) % 32 in increasing j, then a pairwise
    # tree with offsets 16, 8, 4, 2, 1.  Jobs 1-3 share partial 0 with the big value and are absorbed one
    # by one; jobs 4, 8, 12 sit in partials 1, 2, 3: 1 + 1 joins first, then 2^53 + 2 is exact.
    from paper_2108_03645_b200.inputs import JOB_DTYPE
    J = 16
    jobs = np.zeros(J, dtype=JOB_DTYPE)
    jobs["b0"] = 128
    jobs["max_per_gpu"] = 128
    jobs["a"] = 128.0            # X = 128 / a = 1
    jobs["a"][0] = 2.0 ** -46    # X = 2^53
    jobs["weight"] = 1.0
    genome = np.full(J, -1, dtype=np.int32)  # everybody else waits
    genome[[0, 1, 2, 3, 4, 8, 12]] = 0
    assert oracle.model(jobs, 0, 0) == (2.0 ** 53, 1) and oracle.model(jobs, 5, 0) == (1.0, 1)
    F, G = oracle.fitness(jobs, 10 ** 6, 1e3, genome)
    assert G == 7
    assert F == 2.0 ** 53 + 2.0
    # a left-to-right sum loses every one; one partial per job (j % 32) would give 2^53 + 6
    assert F != 2.0 ** 53 and F != 2.0 ** 53 + 6.0
