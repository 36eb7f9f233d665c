"""Pins for the oracle's (mu + lambda) truncation selection, the paper's own scheme (CPU only)."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs


def _search(w, **kw):
    p = w.params
    args = dict(elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut, penalty=p.penalty,
                flags=oracle.FLAG_TRUNCATION)
    args.update(kw)
    return oracle.Search(w.jobs, w.capacity, w.pop, **args)


def test_keep_best_against_sorted():
    rng = np.random.default_rng(4)
    for n, k in ((1, 1), (7, 0), (10, 10), (300, 77), (4096, 1024)):
        F = rng.integers(0, max(2, n // 5), size=n).astype(np.float64)  # many ties
        want = sorted(sorted(range(n), key=lambda i: (-F[i], i))[:k])
        assert list(oracle.keep_best(F, k)) == want


def test_generation_is_best_k_of_originals_children_and_mutants():
    w = inputs.custom(24, 40, 64, 1, seed=5, kmax=5, pinned=3)
    s = _search(w, p_mut=0.1)
    s.randomize(2)
    P0 = s.get_population()
    F0, _ = s.evaluate()
    s.evolve(1, 9)
    P1 = s.get_population()
    F1, G1 = s.evaluate()
    parents, _ = s.last_parents()
    K, J = 64, 24
    assert parents.shape == (K, 2)
    # rebuild the crossover children from the reported parents: complementary, no mutation
    pool = [P0[i] for i in range(K)]
    for q, (a, b) in enumerate(parents):
        flips = np.array([oracle.word(9, 0, 2 * q, j, oracle.STREAM_MUT) & 1 for j in range(J)], dtype=bool)
        pool.append(np.where(flips, P0[b], P0[a]))
        pool.append(np.where(flips, P0[a], P0[b]))
    thr = oracle.thr16(0.1)
    n_mut = 0
    for m in range(K):
        src = (oracle.word(9, 0, m, 0, 4) * K) >> 32  # stream 4: which candidate mutates
        row = P0[src].copy()
        for j in range(J):
            W = oracle.word(9, 0, m, j, 5)            # stream 5: the mutant's draws
            if (W & 0xFFFF) < thr:
                lo, hi = int(w.jobs["kmin"][j]), int(w.jobs["kmax"][j])
                frac = (W * 0x9E360001) & 0xFFFFFFFF
                row[j] = lo + ((frac * (hi - lo + 1)) >> 32)
                n_mut += 1
        pool.append(row)
    assert 0.5 * K * J * 0.1 < n_mut < 1.5 * K * J * 0.1
    pool = np.array(pool)
    Fp = np.array([oracle.fitness(w.jobs, w.capacity, 1e3, r)[0] for r in pool])
    keep = sorted(sorted(range(4 * K), key=lambda i: (-Fp[i], i))[:K])
    assert (P1 == pool[keep]).all()
    assert (F1 == Fp[keep]).all()
    # pinned genes never move, ranges hold
    assert (P1 >= w.jobs["kmin"][None, :]).all() and (P1 <= w.jobs["kmax"][None, :]).all()


def test_no_candidate_gets_worse():
    # the originals compete with their offspring, so neither the best nor the K-th best score can drop
    w = inputs.paper_scale(1)
    s = _search(w)
    s.randomize(0)
    lo, hi = -np.inf, -np.inf
    for _ in range(8):
        F, _ = s.evaluate()
        assert F.max() >= hi and F.min() >= lo
        lo, hi = F.min(), F.max()
        s.evolve(1, 0)


def test_never_beats_brute_force_optimum_and_is_deterministic():
    w = inputs.custom(3, 8, 32, 20, seed=1, kmax=5)
    best = max(oracle.fitness(w.jobs, 8, 1e3, list(ks))[0] for ks in itertools.product(range(6), repeat=3))
    a = _search(w); a.randomize(1); a.evolve(20, 1)
    b = _search(w); b.randomize(1); b.evolve(8, 1); b.evolve(12, 1)
    assert 0.99 * best <= a.best()["fitness"] <= best  # truncation converges fast; it may stop just short
    assert (a.get_population() == b.get_population()).all()


def test_identical_population_without_mutation_stays_put():
    w = inputs.tiny(0)
    s = _search(w, p_mut=0.0)
    row = inputs.random_genomes(w.jobs, 1, seed=3)[0]
    s.set_population(np.tile(row, (w.pop, 1)))
    s.evolve(2, 7)
    assert (s.get_population() == row[None, :]).all()
