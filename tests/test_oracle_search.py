"""Pins for the oracle's operators, selection, elitism, repair and remap (CPU only)."""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs
from util import example_jobs


def _search(w, **kw):
    p = w.params
    args = dict(elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut, penalty=p.penalty, flags=p.flags)
    args.update(kw)
    return oracle.Search(w.jobs, w.capacity, w.pop, **args)


def test_thr16():
    assert oracle.thr16(0.1) == 6554 and oracle.thr16(0.02) == 1311
    assert oracle.thr16(0.0) == 0 and oracle.thr16(1.0) == 65536


def test_create_starts_at_minimum_batch_and_randomize_keeps_row0():
    w = inputs.paper_scale(0)
    s = _search(w)
    assert (s.get_population() == w.jobs["kmin"][None, :]).all()
    s.randomize(4)
    P = s.get_population()
    assert (P[0] == w.jobs["kmin"]).all()
    assert (P >= w.jobs["kmin"][None, :]).all() and (P <= w.jobs["kmax"][None, :]).all()
    # uniform over the range of free genes (chi-square, 8 values)
    free = w.jobs["kmax"] == 7
    counts = np.bincount(P[1:, free].ravel(), minlength=8)
    exp = counts.sum() / 8
    assert ((counts - exp) ** 2 / exp).sum() < 40  # 7 dof, p ~ 1e-6


def test_genes_stay_in_range_and_pinned_never_move():
    w = inputs.paper_scale(1)
    s = _search(w)
    s.randomize(1)
    s.evolve(5, 1)
    P = s.get_population()
    assert (P >= w.jobs["kmin"][None, :]).all() and (P <= w.jobs["kmax"][None, :]).all()
    pinned = w.jobs["kmin"] == w.jobs["kmax"]
    assert pinned.sum() == 20
    assert (P[:, pinned] == 0).all()


def test_crossover_children_are_complementary_without_mutation():
    w = inputs.tiny(2)
    s = _search(w, p_mut=0.0)
    s.randomize(3)
    P0 = s.get_population()
    s.evolve(1, 3)
    P1 = s.get_population()
    parents, elites = s.last_parents()
    E = w.params.elitism
    took_first = 0
    total = 0
    for q, (a, b) in enumerate(parents):
        c0, c1 = P1[E + 2 * q], P1[E + 2 * q + 1]
        A, B = P0[a], P0[b]
        from_a = c0 == A
        from_b = c0 == B
        assert (from_a | from_b).all()
        differ = A != B
        took_first += int((c0[differ] == A[differ]).sum())
        total += int(differ.sum())
        # where the even child took A's gene the odd child holds B's, and the reverse
        assert ((c0 == A) & (c1 == B) | (c0 == B) & (c1 == A)).all()
    assert abs(took_first - total / 2) < 5 * (total / 4) ** 0.5  # fair coin per gene
    for r, e in enumerate(elites):
        assert (P1[r] == P0[e]).all()


def test_identical_parents_without_mutation_reproduce():
    w = inputs.tiny(0)
    s = _search(w, p_mut=0.0)
    row = inputs.random_genomes(w.jobs, 1, seed=8)[0]
    s.set_population(np.tile(row, (w.pop, 1)))
    s.evolve(3, 5)
    assert (s.get_population() == row[None, :]).all()


def test_mutation_rate_and_value_distribution():
    w = inputs.custom(64, 10 ** 6, 513, 1, seed=3, kmax=5)
    # identical rows: crossover has no effect, every change is a mutation
    row = np.zeros(64, dtype=np.int32)
    for p in (0.1, 0.02):
        s = _search(w, p_mut=p, elitism=1)
        s.set_population(np.tile(row, (w.pop, 1)))
        s.evolve(1, 11)
        kids = s.get_population()[1:]
        n = kids.size
        rate = oracle.thr16(p) / 65536 * (5 / 6)  # a redraw hits the old value 1 time in 6
        changed = int((kids != 0).sum())
        assert abs(changed - n * rate) < 5 * (n * rate * (1 - rate)) ** 0.5
    s = _search(w, p_mut=1.0, elitism=1)
    s.set_population(np.tile(row, (w.pop, 1)))
    s.evolve(1, 12)
    kids = s.get_population()[1:]
    counts = np.bincount(kids.ravel(), minlength=6)
    exp = kids.size / 6
    assert ((counts - exp) ** 2 / exp).sum() < 35  # 5 dof
    # each job's column is redrawn independently: per-column means agree
    assert np.abs(kids.mean(axis=0) - 2.5).max() < 6 * (35 / 12 / kids.shape[0]) ** 0.5


def test_tournament_size_one_is_uniform_and_large_picks_best():
    n = 16
    F = np.arange(n, dtype=np.float64)
    picks = np.array([oracle.tournament(F, 1, 77, 0, q, oracle.STREAM_SEL_A) for q in range(8000)])
    counts = np.bincount(picks, minlength=n)
    exp = picks.size / n
    assert ((counts - exp) ** 2 / exp).sum() < 60  # 15 dof
    F = np.random.default_rng(0).normal(size=n)
    best = int(np.argmax(F))
    assert all(oracle.tournament(F, 400, 5, 2, q, oracle.STREAM_SEL_B) == best for q in range(50))
    # size 2: the winner is the better of the two draws
    for q in range(200):
        d = [((oracle.word(9, 4, q, t, oracle.STREAM_SEL_A) * n) >> 32) for t in range(2)]
        want = max(d, key=lambda i: (F[i], -i))
        assert oracle.tournament(F, 2, 9, 4, q, oracle.STREAM_SEL_A) == want


def test_ties_go_to_the_lower_index():
    F = np.array([1.0, 5.0, 5.0, 0.0, 5.0])
    assert list(oracle.top(F, 4)) == [1, 2, 4, 0]
    flat = np.zeros(32)
    picks = [oracle.tournament(flat, 4, 1, 0, q, oracle.STREAM_SEL_A) for q in range(100)]
    for q, p in enumerate(picks):
        draws = [((oracle.word(1, 0, q, t, oracle.STREAM_SEL_A) * 32) >> 32) for t in range(4)]
        assert p == min(draws)


def test_top_matches_sort():
    rng = np.random.default_rng(2)
    F = rng.integers(0, 50, size=300).astype(np.float64)  # many ties
    order = sorted(range(300), key=lambda i: (-F[i], i))
    assert list(oracle.top(F, 17)) == order[:17]


def test_elitism_keeps_best_monotone_and_elites_verbatim():
    w = inputs.paper_scale(0)
    s = _search(w)
    s.randomize(0)
    best = -math.inf
    for g in range(12):
        P0 = s.get_population()
        F0, _ = s.evaluate()
        s.evolve(1, 0)
        P1 = s.get_population()
        F1, _ = s.evaluate()
        _, elites = s.last_parents()
        assert list(elites) == list(oracle.top(F0, 2))
        assert (P1[0] == P0[elites[0]]).all() and (P1[1] == P0[elites[1]]).all()
        assert F1.max() >= F0.max()
        assert F1.max() >= best
        best = F1.max()


def test_determinism_and_split_runs():
    w = inputs.tiny(0)
    a = _search(w); a.randomize(0); a.evolve(10, 0)
    b = _search(w); b.randomize(0); b.evolve(4, 0); b.evolve(6, 0)
    c = _search(w); c.randomize(0); c.evolve(10, 1)
    assert (a.get_population() == b.get_population()).all()
    assert not (a.get_population() == c.get_population()).all()
    assert a.generation == 10 and b.generation == 10


def test_odd_number_of_children():
    w = inputs.custom(7, 16, 10, 1, seed=1, kmax=4)
    s = _search(w, elitism=1)  # 9 children: the last even child has no sibling
    s.randomize(2)
    s.evolve(3, 2)
    P = s.get_population()
    assert P.shape == (10, 7)
    assert (P >= 0).all() and (P <= 4).all()
    parents, _ = s.last_parents()
    assert parents.shape == (5, 2)


def test_search_reaches_brute_force_optimum_on_tiny_instances():
    # 2-4 jobs, 8 GPUs, every assignment enumerated
    for J, seed in ((2, 0), (3, 1), (4, 2)):
        w = inputs.custom(J, 8, 32, 30, seed=seed, kmax=5)
        best = max(oracle.fitness(w.jobs, 8, 1e3, list(ks))[0]
                   for ks in itertools.product(range(6), repeat=J))
        s = _search(w)
        s.randomize(seed)
        for _ in range(30):
            s.evolve(1, seed)
            assert s.best()["fitness"] <= best
        assert s.best()["fitness"] == best


def _knapsack_optimum(w):
    """Exact optimum of sum_j X_j - penalty*max(0, G - cap): multiple-choice
    knapsack over the total GPU count, one exponent per job."""
    J = w.n_jobs
    opts = [[oracle.model(w.jobs, j, k) for k in range(int(w.jobs["kmin"][j]), int(w.jobs["kmax"][j]) + 1)]
            for j in range(J)]
    gmax = sum(max(g for _, g in o) for o in opts)
    best = np.full(gmax + 1, -np.inf)
    best[0] = 0.0
    for o in opts:
        nxt = np.full(gmax + 1, -np.inf)
        for x, g in o:
            nxt[g:] = np.maximum(nxt[g:], best[:gmax + 1 - g] + x)
        best = nxt
    G = np.arange(gmax + 1)
    return float(np.max(best - w.params.penalty * np.maximum(0, G - w.capacity)))


def test_search_never_beats_exact_optimum_and_gets_close():
    w = inputs.custom(40, 96, 256, 60, seed=4, kmax=5)
    opt = _knapsack_optimum(w)
    s = _search(w)
    s.randomize(0)
    s.evolve(60, 0)
    got = s.best()["fitness"]
    assert got <= opt * (1 + 1e-12)
    assert got >= 0.9 * opt
    # unlimited capacity: the problem separates per job
    w2 = inputs.custom(40, 10 ** 6, 256, 60, seed=4, kmax=5)
    sep = sum(max(oracle.model(w2.jobs, j, k)[0] for k in range(6)) for j in range(40))
    assert _knapsack_optimum(w2) == pytest.approx(sep, rel=1e-12)
    s = _search(w2)
    s.randomize(0)
    s.evolve(60, 0)
    assert 0.95 * sep <= s.best()["fitness"] <= sep * (1 + 1e-12)


def test_repair():
    w = inputs.paper_scale(0)  # 100 jobs need more than 64 GPUs even at their smallest batch
    rows = inputs.random_genomes(w.jobs, 6, seed=3)
    for row in rows:
        fixed = oracle.repair(w.jobs, w.capacity, row)
        F, G = oracle.fitness(w.jobs, w.capacity, 1e3, fixed)
        assert G <= w.capacity
        assert (oracle.repair(w.jobs, w.capacity, fixed) == fixed).all()  # idempotent
        parked = fixed < 0
        assert parked.any()
        # nothing is parked while some job could still shrink
        running = ~parked
        for j in np.nonzero(running)[0]:
            k = int(fixed[j])
            assert k <= row[j]
            if k > w.jobs["kmin"][j]:
                assert oracle.model(w.jobs, j, k)[1] == oracle.model(w.jobs, j, k - 1)[1]
        # parked jobs are the lowest-indexed ones that held GPUs
        assert parked[: int(parked.sum())].all()
    big = inputs.tiny(0)
    row = inputs.random_genomes(big.jobs, 1, seed=1)[0]
    G = oracle.fitness(big.jobs, 10 ** 6, 1e3, row)[1]
    assert (oracle.repair(big.jobs, G, row) == row).all()  # already fits: untouched
    fixed = oracle.repair(big.jobs, G - 1, row)
    assert oracle.fitness(big.jobs, G - 1, 1e3, fixed)[1] <= G - 1
    # the job holding the most GPUs (lowest index on ties) gives way first
    gs = [oracle.model(big.jobs, j, int(row[j]))[1] if row[j] > 0 and
          oracle.model(big.jobs, j, int(row[j]))[1] > oracle.model(big.jobs, j, int(row[j]) - 1)[1] else 0
          for j in range(big.n_jobs)]
    first = int(np.argmax(gs))
    assert fixed[first] < row[first]


def test_best_with_repair_fits_capacity():
    w = inputs.paper_scale(0)
    s = _search(w)
    s.randomize(0)
    s.evolve(3, 0)
    raw = s.best(False)
    F, G = s.evaluate()
    assert raw["index"] == int(oracle.top(F, 1)[0]) and raw["fitness"] == F[raw["index"]]
    assert raw["total_gpus"] == G[raw["index"]] == raw["gpus_per_job"].sum()
    fixed = s.best(True)
    assert fixed["total_gpus"] <= w.capacity
    assert fixed["gpus_per_job"].sum() == fixed["total_gpus"]
    assert fixed["fitness"] == pytest.approx(math.fsum(fixed["rate_per_job"]), rel=1e-13)
    assert (fixed["rate_per_job"][fixed["genome"] < 0] == 0).all()


def test_update_jobs_remaps_columns():
    w = inputs.tiny(0)
    s = _search(w)
    s.randomize(0)
    P = s.get_population()
    # jobs 3 and 7 finished; two jobs arrive; job 5's limit drops to 2
    keep = [j for j in range(16) if j not in (3, 7)]
    new = inputs.custom(2, 16, 32, 1, seed=9, kmax=3).jobs  # they may grow later, but start at their smallest batch
    jobs2 = np.concatenate([w.jobs[keep], new])
    jobs2["kmax"][keep.index(5)] = 2
    remap = np.array(keep + [-1, -1], dtype=np.int32)
    s.update_jobs(jobs2, remap, 20)
    Q = s.get_population()
    assert Q.shape == (32, 16)
    for jn, jo in enumerate(keep):
        want = np.clip(P[:, jo], jobs2["kmin"][jn], jobs2["kmax"][jn])
        assert (Q[:, jn] == want).all()
    assert (Q[:, 14:] == 0).all()
    F, G = s.evaluate()
    assert F[0] == oracle.fitness(jobs2, 20, 1e3, Q[0])[0]
    s.evolve(2, 1)  # still runs


def test_bad_arguments_are_reported():
    w = inputs.tiny(0)
    with pytest.raises(oracle.OracleError):
        oracle.Search(w.jobs, 0, 32)
    with pytest.raises(oracle.OracleError):
        oracle.Search(w.jobs, 16, 2, elitism=2)
    with pytest.raises(oracle.OracleError):
        oracle.Search(w.jobs, 16, 32, p_mut=1.5)
    with pytest.raises(oracle.OracleError):
        oracle.Search(w.jobs, 16, 32, tournament=0)


def test_sibling_children_mutate_independently():
    # p = 1: both children of a pair redraw every gene from one shared random word; the two new values
    # must still be jointly uniform over all pairs of values, and rates per child must agree
    w = inputs.custom(48, 10 ** 6, 1025, 1, seed=8, kmax=5)
    row = np.zeros(48, dtype=np.int32)
    s = _search(w, p_mut=1.0, elitism=1)
    s.set_population(np.tile(row, (w.pop, 1)))
    s.evolve(1, 21)
    kids = s.get_population()[1:]
    even, odd = kids[0::2].ravel(), kids[1::2].ravel()
    joint = np.bincount(even * 6 + odd, minlength=36)
    exp = even.size / 36
    assert ((joint - exp) ** 2 / exp).sum() < 80  # 35 dof, p ~ 2e-5
    for p in (0.1, 0.02):
        s = _search(w, p_mut=p, elitism=1)
        s.set_population(np.tile(row, (w.pop, 1)))
        s.evolve(1, 22)
        kids = s.get_population()[1:]
        rate = oracle.thr16(p) / 65536 * (5 / 6)
        for part in (kids[0::2], kids[1::2]):
            n = part.size
            assert abs(int((part != 0).sum()) - n * rate) < 5 * (n * rate * (1 - rate)) ** 0.5
        # a hit on one child says nothing about its sibling at the same gene
        both = int(((kids[0::2] != 0) & (kids[1::2] != 0)).sum())
        n = kids[0::2].size
        assert abs(both - n * rate * rate) < 6 * (n * rate * rate) ** 0.5 + 3
    # p = 0.1: where both siblings redraw the same gene (both 16-bit fields of the word are below the threshold,
    # a thin slice of the word's values) the two new values must still be jointly uniform.  Parents wait at
    # every gene (-1), so each redraw is visible.
    big = inputs.custom(48, 10 ** 6, 8193, 1, seed=8, kmax=5)
    s = _search(big, p_mut=0.1, elitism=1)
    s.set_population(np.full((big.pop, 48), -1, dtype=np.int32))
    s.evolve(1, 23)
    kids = s.get_population()[1:]
    even, odd = kids[0::2].ravel(), kids[1::2].ravel()
    hit = (even >= 0) & (odd >= 0)
    assert abs(int(hit.sum()) - even.size * 0.01) < 6 * (even.size * 0.01) ** 0.5   # both redraw: p * p
    joint = np.bincount(even[hit] * 6 + odd[hit], minlength=36)
    exp = int(hit.sum()) / 36
    assert exp > 40 and ((joint - exp) ** 2 / exp).sum() < 80  # 35 dof, p ~ 2e-5


def test_checkpoint_and_resume():
    w = inputs.paper_scale(0)
    a = _search(w); a.randomize(3); a.evolve(9, 3)
    b = _search(w); b.randomize(3); b.evolve(4, 3)
    saved, gen = b.get_population(), b.generation
    c = _search(w)  # a fresh handle picks the search up from the saved state
    c.set_population(saved)
    c.set_generation(gen)
    c.evolve(5, 3)
    assert (c.get_population() == a.get_population()).all() and c.generation == 9


def test_lower_limits_are_respected():
    w = inputs.custom(40, 10 ** 6, 200, 1, seed=12, kmax=6, kmin_max=4)
    assert w.jobs["kmin"].max() >= 3
    s = _search(w, p_mut=0.5)
    assert (s.get_population() == w.jobs["kmin"][None, :]).all()
    s.randomize(1)
    for _ in range(3):
        P = s.get_population()
        assert (P >= w.jobs["kmin"][None, :]).all() and (P <= w.jobs["kmax"][None, :]).all()
        s.evolve(1, 1)
    # every admissible value of a free job is reached, the lowest and the highest included
    j = int(np.argmax(w.jobs["kmax"] - w.jobs["kmin"]))
    seen = set(P[:, j].tolist())
    assert seen == set(range(int(w.jobs["kmin"][j]), int(w.jobs["kmax"][j]) + 1))
