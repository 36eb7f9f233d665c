"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element."""
import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL_TOL = 1e-12  # fp64 scores, fixed summation order (the build's stated bound; 0 ulp expected)


@pytest.fixture(scope="module")
def ones():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding
    binding.lib()
    return binding


def _pair(ones, w, **kw):
    p = w.params
    args = dict(elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut, penalty=p.penalty, flags=p.flags)
    args.update(kw)
    sp = inputs.SearchParams(**args)
    return ones.Search(w.jobs, w.capacity, w.pop, sp), oracle.Search(w.jobs, w.capacity, w.pop, **args)


def _rel_err(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    scale = np.maximum(np.abs(b), 1e-300)
    return float(np.max(np.abs(a - b) / scale)) if a.size else 0.0


def _same_state(g, o, exact_scores=True):
    assert (g.get_population() == o.get_population()).all()
    Fg, Gg = g.evaluate()
    Fo, Go = o.evaluate()
    assert (Gg.cpu().numpy() == Go).all()
    assert _rel_err(Fg.cpu().numpy(), Fo) <= REL_TOL
    if exact_scores:
        assert (Fg.cpu().numpy() == Fo).all()


# ---- a0: model tables ----------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "paper", "mid", "large"])
def test_model_table_bit_exact(ones, name):
    w = inputs.WORKLOADS[name]()
    s = ones.Search(w.jobs, w.capacity, 8, inputs.SearchParams())
    X, g = s.model_table()
    assert X.shape[0] == int(w.jobs["kmax"].max()) + 1
    for j in range(0, w.n_jobs, max(1, w.n_jobs // 64)):
        for k in range(X.shape[0]):
            Xo, go = oracle.model(w.jobs, j, k)
            assert g[k, j] == go and X[k, j] == Xo, (j, k)


def test_model_table_non_power_of_two_and_sruf(ones):
    w = inputs.custom(50, 64, 8, 1, seed=3, pow2=False)
    w.jobs["weight"] = np.linspace(1e3, 9e4, 50)
    for flags in (0, ones.FLAG_SRUF):
        s = ones.Search(w.jobs, w.capacity, 8, inputs.SearchParams(flags=flags))
        X, g = s.model_table()
        want = np.array([[oracle.term(w.jobs, j, k, flags) for j in range(50)] for k in range(X.shape[0])])
        assert (g == want[:, :, 1]).all()
        assert (X == want[:, :, 0]).all()  # log2 of a GPU count that is not a power of two comes from the host's library


# ---- a1: fitness ---------------------------------------------------------------------------------
@pytest.mark.parametrize("J,n,ld_extra", [(1, 5, 3), (3, 33, 1), (5, 64, 7), (16, 32, 0), (100, 1000, 4),
                                          (127, 257, 1), (128, 300, 0), (129, 300, 3), (512, 2051, 0),
                                          (2048, 5000, 0), (2050, 700, 2)])
def test_fitness_parity(ones, J, n, ld_extra):
    w = inputs.custom(J, max(8, 2 * J), 8, 1, seed=J, log_uniform=True)
    ld = ((J + 3) // 4) * 4 + 4 * ((ld_extra + 3) // 4)
    genomes = inputs.random_genomes(w.jobs, n, ld=ld, seed=n, waiting_fraction=0.05)
    genomes[0, :J] = w.jobs["kmax"] + 1  # above every limit: all jobs wait
    if n > 1:
        genomes[1, :J] = np.iinfo(np.int32).min
    g, o = _pair(ones, w)
    Fg, Gg = g.evaluate(torch.from_numpy(genomes).cuda())
    Fo, Go = o.evaluate(genomes)
    assert (Gg.cpu().numpy() == Go).all()
    assert _rel_err(Fg.cpu().numpy(), Fo) <= REL_TOL
    assert (Fg.cpu().numpy() == Fo).all()
    assert Fo[0] == 0.0 and Go[0] == 0


def test_fitness_summation_order_case(ones):
    # 2^53 next to a few ones: the documented order keeps exactly two of them (see the oracle's pin)
    jobs = np.zeros(16, dtype=inputs.JOB_DTYPE)
    jobs["b0"] = 128
    jobs["max_per_gpu"] = 128
    jobs["a"] = 128.0
    jobs["a"][0] = 2.0 ** -46
    jobs["weight"] = 1.0
    genome = np.full((3, 16), -1, dtype=np.int32)
    genome[:, [0, 1, 2, 3, 4, 8, 12]] = 0
    s = ones.Search(jobs, 10 ** 6, 3, inputs.SearchParams(1, 2, 0.1, 1e3))
    F, G = s.evaluate(torch.from_numpy(genome).cuda())
    assert F.cpu().tolist() == [2.0 ** 53 + 2.0] * 3 and G.cpu().tolist() == [7, 7, 7]
    s.set_population(genome)  # the evolve kernels score in the same order
    s.evolve(1, 0)
    F2, _ = s.evaluate()
    assert F2.cpu().tolist()[0] == 2.0 ** 53 + 2.0  # the elite row, copied and scored again


def test_fitness_zero_rows_and_sruf(ones):
    w = inputs.paper_scale(1)
    w.jobs["weight"] = np.random.default_rng(0).uniform(1e3, 1e6, w.n_jobs)
    g, o = _pair(ones, w, flags=ones.FLAG_SRUF)
    genomes = inputs.random_genomes(w.jobs, 77, seed=1)
    Fg, Gg = g.evaluate(torch.from_numpy(genomes).cuda())
    Fo, Go = o.evaluate(genomes)
    assert (Gg.cpu().numpy() == Go).all() and (Fg.cpu().numpy() == Fo).all()
    empty = torch.zeros((0, 100), dtype=torch.int32, device="cuda")
    Fe, Ge = g.evaluate(empty)
    assert Fe.numel() == 0


# ---- a2: top-e -----------------------------------------------------------------------------------
@pytest.mark.parametrize("n,e", [(1, 1), (5, 5), (32, 2), (1000, 7), (4097, 33), (65536, 2), (200000, 256)])
def test_select_top_parity(ones, n, e):
    rng = np.random.default_rng(n)
    F = rng.integers(0, max(2, n // 3), size=n).astype(np.float64) - 5.0  # many ties, both signs
    F[rng.integers(0, n)] = -0.0
    got = ones.select_top(torch.from_numpy(F).cuda(), e).cpu().numpy()
    want = np.array(sorted(range(n), key=lambda i: (-F[i], i))[:e])
    assert (got == want).all()
    if n <= 5000:
        assert (got == oracle.top(F, e)).all()


# ---- a3/a4/a5: one generation and many -------------------------------------------------------------
def test_randomize_parity(ones):
    for w in (inputs.tiny(), inputs.paper_scale(), inputs.custom(131, 64, 77, 1, seed=2, pinned=9)):
        g, o = _pair(ones, w)
        _same_state(g, o)  # all-minimum start
        g.randomize(12345678901234567)
        o.randomize(12345678901234567)
        _same_state(g, o)


@pytest.mark.parametrize("name,gens,flags", [("tiny", 10, 0), ("paper", 100, 0), ("paper", 100, 2), ("tiny", 10, 8),
                                             ("paper", 100, 8)])  # 0: one cluster launch, 8: launch per generation
def test_evolve_parity_named_workloads(ones, name, gens, flags):
    w = inputs.WORKLOADS[name]()
    g, o = _pair(ones, w, flags=flags)
    g.randomize(w.seed)
    o.randomize(w.seed)
    done = 0
    for step in (1, 1, 8, gens - 10):
        g.evolve(step, w.seed)
        o.evolve(step, w.seed)
        done += step
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
        assert g.generation == o.generation == done
    bg, bo = g.best(True), o.best(True)
    for key in ("genome", "gpus_per_job", "rate_per_job"):
        assert (bg[key] == bo[key]).all(), key
    assert bg["fitness"] == bo["fitness"] and bg["total_gpus"] == bo["total_gpus"] and bg["index"] == bo["index"]
    assert bg["total_gpus"] <= w.capacity


def test_evolve_parity_mid_all_generations(ones):
    """The mid workload for all of its 200 generations: parents, elites, genomes, GPU demand and scores against the
    oracle at generations 1, 2, 10, 50 and 200 (near-ties between fp64 scores decide tournaments, and only a long
    run at scale meets many of them)."""
    w = inputs.mid()
    g, o = _pair(ones, w)
    g.randomize(w.seed)
    o.randomize(w.seed)
    done = 0
    for upto in (1, 2, 10, 50, w.generations):
        g.evolve(upto - done, w.seed)
        o.evolve(upto - done, w.seed)
        done = upto
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all(), upto
        _same_state(g, o)
        assert g.generation == o.generation == done
    bg, bo = g.best(True), o.best(True)
    for key in ("genome", "gpus_per_job", "rate_per_job"):
        assert (bg[key] == bo[key]).all(), key
    assert bg["fitness"] == bo["fitness"] and bg["total_gpus"] == bo["total_gpus"] <= w.capacity


@pytest.mark.parametrize("kw", [dict(elitism=0), dict(elitism=1), dict(elitism=5, tournament=1),
                                dict(tournament=9), dict(p_mut=0.0), dict(p_mut=1.0), dict(p_mut=0.02, tournament=8),
                                dict(penalty=0.0), dict(penalty=37.5), dict(flags=2), dict(flags=2, p_mut=1.0),
                                dict(flags=3), dict(flags=8), dict(flags=8, elitism=0), dict(flags=8, p_mut=1.0)])
def test_evolve_parity_parameter_corners(ones, kw):
    w = inputs.custom(37, 48, 101, 6, seed=7, kmax=6, pinned=4, kmin_max=3)
    g, o = _pair(ones, w, **kw)
    g.randomize(5)
    o.randomize(5)
    for _ in range(3):
        g.evolve(2, 99)
        o.evolve(2, 99)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)


@pytest.mark.parametrize("elitism", [1, 2, 3, 4, 5, 9])
@pytest.mark.parametrize("N,flags", [(300, 2), (5000, 0), (1031, 2), (1031, 8), (2500, 8)])
def test_selection_stage_elites_with_ties(ones, elitism, N, flags):
    """Elites of the selection stage (register lists up to 4, block rounds above) on populations full of equal
    scores: slices with fewer distinct candidates than elites, ties decided by the row index."""
    w = inputs.custom(24, 40, N, 3, seed=N + elitism, kmax=5)
    g, o = _pair(ones, w, elitism=elitism, flags=flags)
    rows = inputs.random_genomes(w.jobs, 7, seed=3)[:, :24]
    pop = rows[np.random.default_rng(elitism).integers(0, 7, size=N)]   # only 7 distinct candidates
    g.set_population(pop)
    o.set_population(pop)
    for _ in range(3):
        g.evolve(1, 21)
        o.evolve(1, 21)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (eg == eo).all() and (pg == po).all()
        _same_state(g, o)


@pytest.mark.parametrize("flags", [0, 8])
@pytest.mark.parametrize("J,N", [(1, 2), (2, 3), (5, 4), (6, 4096), (127, 33), (129, 64), (260, 1025), (700, 2000)])
def test_evolve_parity_ragged_shapes(ones, J, N, flags):
    w = inputs.custom(J, max(4, J), N, 4, seed=J + N, kmax=7, params=inputs.SearchParams(1, 3, 0.1, 1e3))
    g, o = _pair(ones, w, flags=flags)
    g.randomize(1)
    o.randomize(1)
    g.evolve(4, 2 ** 40 + 17)
    o.evolve(4, 2 ** 40 + 17)
    _same_state(g, o)


@pytest.mark.parametrize("flags", [0, 32])
@pytest.mark.parametrize("J,N,kw", [(260, 12000, dict(elitism=3)), (700, 20001, {}), (129, 9474, dict(elitism=0, p_mut=1.0)),
                                    (512, 10000, dict(tournament=2))])
def test_evolve_parity_more_pairs_than_warps(ones, J, N, kw, flags):
    """Populations with more pairs of children than the persistent grid has warps (pairs beyond the first round are
    handed out through the work counter) on ragged rows: an odd and an even number of 128-gene blocks, a partial
    last block, an odd child count."""
    w = inputs.custom(J, max(4, J), N, 3, seed=J + N, kmax=6, kmin_max=1, pinned=J // 7)
    g, o = _pair(ones, w, flags=flags, **kw)
    g.randomize(4)
    o.randomize(4)
    for step in (1, 2):
        g.evolve(step, 77)
        o.evolve(step, 77)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)


@pytest.mark.parametrize("flags", [0, 2, 8, 32, 4])
def test_evolve_non_power_of_two_gpu_counts(ones, flags):
    """Batch sizes and per-GPU limits that are not powers of two: log2 of the GPU count is then not an integer.  The
    library takes it from the host's math library (the routine the oracle calls), so tables, scores and every
    selection stay identical over the generations, on every launch sequence."""
    for J, N in ((64, 256), (300, 6000)):
        w = inputs.custom(J, 2 * J, N, 1, seed=11, pow2=False, kmax=5)
        g, o = _pair(ones, w, flags=flags)
        X, gt = g.model_table()
        for j in range(0, J, 7):
            for k in range(X.shape[0]):
                Xo, go = oracle.model(w.jobs, j, k)
                assert gt[k, j] == go and X[k, j] == Xo, (j, k)
        assert (gt & (gt - 1)).any()  # some GPU count is not a power of two
        g.randomize(0)
        o.randomize(0)
        _same_state(g, o)
        for step in (1, 4):
            g.evolve(step, 9)
            o.evolve(step, 9)
            _same_state(g, o)
        jobs2 = np.concatenate([w.jobs[3:], inputs.custom(5, 8, 4, 1, seed=2, pow2=False, kmax=3).jobs])
        remap = np.concatenate([np.arange(3, J), np.full(5, -1)]).astype(np.int32)
        if not flags & 4:  # (the truncation scheme keeps its pool across a change of the job set as well)
            g2 = ones.Search(w.jobs, w.capacity, N, inputs.SearchParams(flags=flags), n_jobs_max=J + 8)
            o2 = oracle.Search(w.jobs, w.capacity, N, flags=flags & 1)
            for s in (g2, o2):
                s.randomize(1)
                s.evolve(2, 1)
                s.update_jobs(jobs2, remap, w.capacity)
                s.evolve(2, 2)
            _same_state(g2, o2)


@pytest.mark.parametrize("elitism", [0, 1, 2, 3, 4, 5, 7])
@pytest.mark.parametrize("J,N", [(16, 32), (100, 1024), (8, 4096), (40, 2048), (14, 999)])
def test_cluster_path_elites_over_many_generations(ones, J, N, elitism):
    """Populations that run all generations of a call inside one cluster launch: there the elites of a new population
    come from the old elites and the children that beat the old E-th best (lists of at most eight children per CTA
    and generation), and elite rows are copied with their scores.  Several generations per call, every number of
    elites on both sides of the four that the lists handle."""
    w = inputs.custom(J, max(4, 2 * J), N, 3, seed=J + N + elitism, kmax=6, kmin_max=1, pinned=J // 6)
    g, o = _pair(ones, w, elitism=elitism, tournament=3, p_mut=0.05)
    g.randomize(2)
    o.randomize(2)
    for gens in (1, 6, 13):
        g.evolve(gens, 5)
        o.evolve(gens, 5)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    bg, bo = g.best(True), o.best(True)
    assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"] and bg["index"] == bo["index"]


@pytest.mark.parametrize("elitism", [1, 2, 4])
@pytest.mark.parametrize("J,N", [(16, 32), (100, 1024), (8, 4096)])
def test_cluster_path_many_children_beat_the_elites(ones, J, N, elitism):
    """Every candidate starts as the same row and genes are redrawn at a high rate: where the common row is not
    already the best one, far more than eight children of a CTA beat the old elites from one generation to the next,
    so the lists overflow and every CTA falls back to the search over all scores inside the launch (seen on the 8 x
    4096 case with p_mut = 1 and on the 100 x 1024 case with p_mut = 0.3); later generations return to the lists."""
    w = inputs.custom(J, max(4, 2 * J), N, 3, seed=J + N, kmax=6)
    g, o = _pair(ones, w, elitism=elitism, tournament=2, p_mut=1.0)
    rows = np.tile(w.jobs["kmin"].astype(np.int32), (N, 1))
    g.set_population(rows)
    o.set_population(rows)
    for gens in (4, 3):
        g.evolve(gens, 9)
        o.evolve(gens, 9)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    g2, o2 = _pair(ones, w, elitism=elitism, tournament=2, p_mut=0.3)   # some generations with lists, some without
    for s_ in (g2, o2):
        s_.set_population(rows)
        s_.evolve(12, 3)
    _same_state(g2, o2)


def test_split_runs_and_determinism(ones):
    w = inputs.paper_scale()
    a, _ = _pair(ones, w)
    b, _ = _pair(ones, w)
    c, _ = _pair(ones, w)
    for s in (a, b, c):
        s.randomize(0)
    a.evolve(10, 0)
    b.evolve(4, 0)
    b.evolve(6, 0)
    c.evolve(10, 1)
    A, B = a.get_population(), b.get_population()
    assert (A == B).all() and not (A == c.get_population()).all()
    assert (a.evaluate()[0] == b.evaluate()[0]).all()


def test_checkpoint_and_resume(ones):
    w = inputs.paper_scale()
    a, o = _pair(ones, w)
    a.randomize(3)
    o.randomize(3)
    a.evolve(4, 3)
    o.evolve(9, 3)
    saved, gen = a.get_population(), a.generation
    b, _ = _pair(ones, w)  # a fresh handle picks the search up from the saved state
    b.set_population(saved)
    b.set_generation(gen)
    b.evolve(5, 3)
    assert b.generation == 9
    _same_state(b, o)


@pytest.mark.parametrize("flags,J,N", [(4, 130, 700), (4, 260, 20000), (0, 16, 32), (0, 8, 4096)])
def test_checkpoint_and_resume_of_mapped_and_cluster_states(ones, flags, J, N):
    """Saving and resuming where the handle keeps state of its own between generations: the truncation scheme's pool
    used in place (the saved population is the ordered one) and the cluster path (a resumed call starts without the
    lists of promising children).  Also: a change of the generation counter between two calls."""
    w = inputs.custom(J, 2 * J, N, 3, seed=J + N, kmax=6, pinned=J // 6)
    a, o = _pair(ones, w, flags=flags, p_mut=0.05)
    a.randomize(3)
    o.randomize(3)
    a.evolve(4, 3)
    a.evolve(3, 3)
    o.evolve(12, 3)
    saved, gen = a.get_population(), a.generation
    b, _ = _pair(ones, w, flags=flags, p_mut=0.05)
    b.set_population(saved)
    b.set_generation(gen)
    b.evolve(5, 3)
    assert b.generation == 12
    _same_state(b, o)
    a.set_generation(gen)      # the first handle goes on from its own (mapped) state as well
    a.evolve(5, 3)
    _same_state(a, o)
    a.set_generation(3)        # back in time: the draws of generations 3 and 4 on the current population
    o.set_generation(3)
    a.evolve(2, 3)
    o.evolve(2, 3)
    _same_state(a, o)


def test_set_get_population_roundtrip(ones):
    w = inputs.custom(30, 64, 50, 1, seed=1)
    g, o = _pair(ones, w)
    rows = inputs.random_genomes(w.jobs, 50, ld=36, seed=4)
    g.set_population(rows)
    o.set_population(rows)
    _same_state(g, o)
    assert (g.get_population(ld=40)[:, :30] == rows[:, :30]).all()
    dev = torch.from_numpy(rows).cuda()
    g.set_population(dev)
    back = g.get_population(on_device=True, ld=32).cpu().numpy()
    assert (back[:, :30] == rows[:, :30]).all()
    g.evolve(3, 4)
    o.evolve(3, 4)
    _same_state(g, o)


# ---- the paper's truncation selection (originals + crossover children + mutants, best K survive) -------
@pytest.mark.parametrize("J,N,kw", [(16, 32, {}), (100, 1024, {}), (37, 101, dict(p_mut=1.0)), (5, 3, dict(p_mut=0.0)),
                                    (130, 257, dict(p_mut=0.02)), (1, 3, {}), (512, 4096, {}),
                                    (130, 257, dict(flags=6)), (37, 101, dict(p_mut=1.0, flags=6)),   # separate scoring pass
                                    (2048, 700, dict(p_mut=0.02)),
                                    (130, 257, dict(flags=12)), (512, 4096, dict(flags=12))])  # survivors gathered
def test_truncation_selection_parity(ones, J, N, kw):
    w = inputs.custom(J, max(4, J), N, 4, seed=J + N, kmax=7, pinned=J // 5, kmin_max=2)
    kw = dict(kw)
    g, o = _pair(ones, w, flags=kw.pop("flags", 4), **kw)
    g.randomize(2)
    o.randomize(2)
    for step in (1, 1, 3):
        g.evolve(step, 11)
        o.evolve(step, 11)
        pg, _ = g.last_parents()
        po, _ = o.last_parents()
        assert pg.shape == (N, 2) and (pg == po).all()
        _same_state(g, o)
    bg, bo = g.best(True), o.best(True)
    assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"]


def test_truncation_selection_parity_large_job_table(ones):
    """The paper's scheme on the benchmark's job table with a pool larger than L2 (4 x 32768 rows of 2048 genes =
    1 GiB per buffer): every survivor, score and GPU count of one generation against the oracle."""
    import dataclasses
    w = dataclasses.replace(inputs.large(), pop=32768)
    g, o = _pair(ones, w, flags=4)
    g.randomize(w.seed)
    o.randomize(w.seed)
    g.evolve(1, w.seed)
    o.evolve(1, w.seed)
    pg, _ = g.last_parents()
    po, _ = o.last_parents()
    assert (pg == po).all()
    _same_state(g, o)


@pytest.mark.parametrize("J,N", [(16, 32), (130, 257), (300, 5000), (2048, 700)])
def test_truncation_pool_in_place_over_many_generations(ones, J, N):
    """The fused handle keeps the pool in place between generations (a row map instead of a gather).  Several
    generations per call, the best candidate read through the map before anything orders the rows, a change of the
    job set on the mapped pool, and the handle that gathers the survivors every generation as a second witness."""
    w = inputs.custom(J, max(4, J), N, 4, seed=3 * J + N, kmax=6, pinned=J // 6, kmin_max=2)
    g = ones.Search(w.jobs, w.capacity, N, inputs.SearchParams(p_mut=0.03, flags=4), n_jobs_max=J + 8)
    h = ones.Search(w.jobs, w.capacity, N, inputs.SearchParams(p_mut=0.03, flags=12), n_jobs_max=J + 8)
    o = oracle.Search(w.jobs, w.capacity, N, p_mut=0.03, flags=4)
    for s_ in (g, o, h):
        s_.randomize(6)
        s_.evolve(7, 21)
    for rep in (True, False):
        bg, bh, bo = g.best(rep), h.best(rep), o.best(rep)   # g: still mapped, the row is found through the map
        for b in (bg, bh):
            assert (b["genome"] == bo["genome"]).all() and b["fitness"] == bo["fitness"] and b["index"] == bo["index"]
    for s_ in (g, o, h):
        s_.evolve(5, 22)
    _same_state(g, o)
    _same_state(h, o)
    for s_ in (g, o, h):
        s_.evolve(2, 23)   # from the ordered pool, then mapped again when the job set changes
    jobs2 = np.concatenate([w.jobs[2:], inputs.custom(4, 8, 4, 1, seed=2, kmax=3).jobs])
    remap = np.concatenate([np.arange(2, J), np.full(4, -1)]).astype(np.int32)
    for s_ in (g, o, h):
        s_.update_jobs(jobs2, remap, w.capacity)   # g: the candidates are put in order before their columns move
        s_.evolve(3, 24)
    _same_state(g, o)
    _same_state(h, o)


def test_truncation_pool_in_place_large_pool(ones):
    """A pool of 80000 rows (five rows per thread of the selection cluster, the 16-rows-per-thread build of the
    kernel) used in place over several generations: the second and later generations read their parents through
    the row map that the selection before them wrote."""
    J, N = 260, 20000
    w = inputs.custom(J, 2 * J, N, 4, seed=77, kmax=6, pinned=J // 6, kmin_max=2)
    g = ones.Search(w.jobs, w.capacity, N, inputs.SearchParams(p_mut=0.03, flags=4))
    h = ones.Search(w.jobs, w.capacity, N, inputs.SearchParams(p_mut=0.03, flags=12))
    o = oracle.Search(w.jobs, w.capacity, N, p_mut=0.03, flags=4)
    for s_ in (g, o, h):
        s_.randomize(3)
    for gens in (1, 3, 2):
        for s_ in (g, o, h):
            s_.evolve(gens, 8)
        pg, _ = g.last_parents()
        po, _ = o.last_parents()
        assert (pg == po).all()
        bg, bo = g.best(False), o.best(False)   # read through the map
        assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"] and bg["index"] == bo["index"]
        _same_state(g, o)
        _same_state(h, o)


def test_truncation_selection_with_many_ties(ones):
    # identical candidates: every score ties, survivors are decided by row order alone
    w = inputs.tiny()
    g, o = _pair(ones, w, flags=4, p_mut=0.05)
    rows = np.tile(inputs.random_genomes(w.jobs, 1, seed=5)[0], (w.pop, 1))
    g.set_population(rows)
    o.set_population(rows)
    for _ in range(4):
        g.evolve(1, 3)
        o.evolve(1, 3)
        _same_state(g, o)


# ---- the paper's per-GPU genome with the reorder operation -------------------------------------------
@pytest.mark.parametrize("J,gpus,N,kw", [(6, 12, 64, {}), (100, 64, 1024, {}), (37, 130, 101, dict(p_mut=1.0)),
                                         (5, 3, 4, dict(p_mut=0.0)), (300, 257, 129, dict(elitism=0)),
                                         (2048, 4096, 300, dict(p_mut=0.02, tournament=8)), (40, 4100, 33, {}),
                                         (1500, 1027, 40, {})])
def test_per_gpu_genome_parity(ones, J, gpus, N, kw):
    w = inputs.custom(J, gpus, N, 4, seed=J + N, kmax=6, kmin_max=1)
    g, o = _pair(ones, w, flags=16, **kw)
    assert (g.get_population() == -1).all() and g.get_population().shape == (N, gpus)
    _same_state(g, o)  # an idle cluster scores 0
    g.randomize(3)
    o.randomize(3)
    _same_state(g, o)
    for step in (1, 2):
        g.evolve(step, 13)
        o.evolve(step, 13)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    bg, bo = g.best(), o.best()
    for key in ("genome", "gpus_per_job", "rate_per_job"):
        assert (bg[key] == bo[key]).all(), key
    assert bg["fitness"] == bo["fitness"] and bg["total_gpus"] == bo["total_gpus"] <= gpus
    # scoring rows from outside, with idle and invalid ids and padding columns
    rng = np.random.default_rng(J)
    ld = (gpus + 3) // 4 * 4 + 4
    rows = np.full((50, ld), 0x7F7F7F7F, dtype=np.int32)
    rows[:, :gpus] = rng.integers(-2, J + 2, size=(50, gpus))
    Fg, Gg = g.evaluate(torch.from_numpy(rows).cuda())
    Fo, Go = o.evaluate(rows)
    assert (Fg.cpu().numpy() == Fo).all() and (Gg.cpu().numpy() == Go).all()
    with pytest.raises(ones.OnesError):
        g.update_jobs(w.jobs, np.arange(J, dtype=np.int32), gpus + 1)  # the cluster keeps its size


def test_per_gpu_genome_wide_batches(ones):
    """Batch sizes and per-GPU limits so large that GPUs x max_per_gpu passes 2^31: the 64-bit exponent search."""
    w = inputs.custom(50, 600, 80, 2, seed=8, kmax=4, kmin_max=1)
    w.jobs["b0"] = (w.jobs["b0"].astype(np.int64) << 14).astype(np.int32)          # up to 2^21, << kmax 4 stays below 2^31
    w.jobs["max_per_gpu"] = (w.jobs["max_per_gpu"].astype(np.int64) << 15).astype(np.int32)   # 2^21 .. 2^23
    assert 600 * int(w.jobs["max_per_gpu"].max()) >= 2 ** 31
    g, o = _pair(ones, w, flags=16)
    g.randomize(1)
    o.randomize(1)
    _same_state(g, o)
    g.evolve(3, 5)
    o.evolve(3, 5)
    _same_state(g, o)
    bg, bo = g.best(), o.best()
    assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"]


def _changed_job_set(rng, jobs, n_leave, n_new, seed, kmax_new=0, shuffle=False):
    """Some jobs finish, limits move by -1..+1 exponents, new jobs join; returns (jobs, remap)."""
    J = jobs.shape[0]
    keep = sorted(rng.choice(J, size=J - n_leave, replace=False).tolist())
    fresh = inputs.custom(max(n_new, 1), 8, 4, 1, seed=seed, kmax=kmax_new, kmin_max=min(1, kmax_new)).jobs[:n_new]
    new = np.concatenate([jobs[keep], fresh])
    new["kmax"][:len(keep)] = np.clip(new["kmax"][:len(keep)] + rng.integers(-1, 2, len(keep)), 0, 7)
    new["kmin"] = np.minimum(new["kmin"], new["kmax"])
    remap = np.array(keep + [-1] * n_new, dtype=np.int32)
    if shuffle:  # new jobs anywhere in the table
        order = rng.permutation(new.shape[0])
        new, remap = new[order], remap[order]
    return new, remap


@pytest.mark.parametrize("J,gpus,N,leave,arrive,kw", [
    (6, 12, 64, 2, 2, {}),                                   # small: finished jobs, new jobs, refill
    (100, 64, 300, 13, 20, {}),                              # more new jobs than GPUs free up: GPUs are taken
    (37, 130, 101, 5, 3, dict(flags=1)),                     # SRUF terms: gains of either sign
    (5, 3, 9, 1, 6, {}),                                     # more new jobs than GPUs
    (300, 257, 129, 0, 0, {}),                               # only the limits move
    (64, 1027, 40, 60, 1, {}),                               # the cluster empties: one big refill
    (2048, 4096, 150, 200, 150, dict(p_mut=0.02)),           # benchmark shape
    (40, 4100, 33, 7, 9, {}),                                # rows above 4096 slots
    (200, 300, 50, 20, 10, {}),                              # sort lengths 256, 1024 and 4096 (1, 4, 16 records
    (700, 900, 40, 100, 30, {}),                             # per thread in registers)
    (2500, 1500, 24, 300, 100, dict(p_mut=0.02)),
])
def test_per_gpu_refresh_parity(ones, J, gpus, N, leave, arrive, kw):
    """ones_update_jobs on per-GPU candidates = the oracle's Refresh + Reorder, row by row."""
    flags = 16 | kw.pop("flags", 0)
    w = inputs.custom(J, gpus, N, 4, seed=J + N, kmax=6, kmin_max=1)
    p = inputs.SearchParams(flags=flags, **kw)
    g = ones.Search(w.jobs, gpus, N, p, n_jobs_max=J + 3 * arrive + 8)
    o = oracle.Search(w.jobs, gpus, N, elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut, penalty=p.penalty,
                      flags=flags)
    g.randomize(3)
    o.randomize(3)
    g.evolve(2, 13)
    o.evolve(2, 13)
    rng = np.random.default_rng(J + gpus)
    jobs = w.jobs
    for rnd in range(3):
        if rnd == 1:
            # rows from outside: unpacked, with idle and out-of-range ids (ranks are then counted, not derived)
            rows = rng.integers(-2, jobs.shape[0] + 2, size=(N, gpus)).astype(np.int32)
            rows[: N // 3] = np.sort(rows[: N // 3], axis=1)
            g.set_population(rows)
            o.set_population(rows)
        jobs2, remap = _changed_job_set(rng, jobs, min(leave, jobs.shape[0] - 1), arrive, seed=50 + rnd,
                                        kmax_new=rnd, shuffle=rnd == 2)
        g.update_jobs(jobs2, remap, gpus)
        o.update_jobs(jobs2, remap, gpus)
        assert (g.get_population() == o.get_population()).all(), rnd
        _same_state(g, o)
        g.evolve(2, rnd)
        o.evolve(2, rnd)
        _same_state(g, o)
        jobs = jobs2
    bg, bo = g.best(), o.best()
    assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"]


def test_per_gpu_refresh_rejected_update_leaves_the_search_untouched(ones):
    w = inputs.custom(9, 20, 40, 2, seed=6, kmax=3)
    g, o = _pair(ones, w, flags=16)
    g.randomize(4)
    o.randomize(4)
    g.evolve(2, 4)
    o.evolve(2, 4)
    bad = w.jobs.copy()
    bad["a"][2] = bad["c"][2] = bad["d"][2] = 0.0          # zero seconds per iteration: no throughput
    with pytest.raises(ones.OnesError) as err:
        g.update_jobs(bad, np.arange(9, dtype=np.int32), 20)
    assert err.value.code == -2
    _same_state(g, o)                                      # population, scores and tables as before
    g.evolve(2, 5)
    o.evolve(2, 5)
    _same_state(g, o)


def test_per_gpu_refresh_limits(ones):
    w = inputs.custom(6, 12, 8, 1, seed=1, kmax=3)
    g = ones.Search(w.jobs, 12, 8, inputs.SearchParams(flags=16), n_jobs_max=8)
    with pytest.raises(ones.OnesError) as err:   # more jobs than the workspace was sized for
        g.update_jobs(np.concatenate([w.jobs] * 4), np.full(24, -1, dtype=np.int32), 12)
    assert err.value.code == -5
    g.update_jobs(w.jobs[:4], np.array([0, 1, 1, -1], dtype=np.int32), 12)   # two rows claim old job 1
    assert ((g.get_population() >= -1) & (g.get_population() < 4)).all()


# ---- packed candidates: one byte per gene --------------------------------------------------------------
def _pack_numpy(rows, J):
    """The packed layout restated: tiles of 512 genes, byte 16*l + 4*b + s = gene 128*b + 4*l + s of the tile."""
    n = rows.shape[0]
    ld8 = (J + 511) // 512 * 512
    genes = np.full((n, ld8), 255, dtype=np.int64)
    genes[:, :J] = np.where((rows[:, :J] < 0) | (rows[:, :J] > 254), 255, rows[:, :J])
    j = np.arange(ld8)
    tile, r = j // 512, j % 512
    b, q = r // 128, r % 128
    where = tile * 512 + 16 * (q // 4) + 4 * b + q % 4
    out = np.zeros((n, ld8), dtype=np.uint8)
    out[:, where] = genes[:, j].astype(np.uint8)
    return out


@pytest.mark.parametrize("J,N", [(1, 3), (5, 9), (127, 40), (129, 33), (511, 20), (513, 70), (700, 5000), (2048, 300)])
def test_packed_candidates_score_like_int32_rows(ones, J, N):
    w = inputs.custom(J, max(4, J), N, 1, seed=J + N, kmax=7, kmin_max=2)
    g, o = _pair(ones, w)
    ld = (J + 3) // 4 * 4 + 8
    rows = inputs.random_genomes(w.jobs, N, ld=ld, seed=J, waiting_fraction=0.05)
    rows[0, :J] = 9                      # above every job's limit: a zero table entry, not a waiting job
    rows[N // 2, J // 2] = 300           # out of the byte range: stored as "waits"
    dev = torch.from_numpy(rows).cuda()
    packed = g.pack(dev)
    assert packed.shape == (N, (J + 511) // 512 * 512)
    assert (packed.cpu().numpy() == _pack_numpy(rows, J)).all()
    Fp, Gp = g.evaluate_packed(packed)
    Fi, Gi = g.evaluate(dev)
    Fo, Go = o.evaluate(rows)
    assert (Fp.cpu().numpy() == Fi.cpu().numpy()).all() and (Gp.cpu().numpy() == Gi.cpu().numpy()).all()
    assert (Gp.cpu().numpy() == Go).all() and _rel_err(Fp.cpu().numpy(), Fo) <= REL_TOL
    assert (Fp.cpu().numpy() == Fo).all()
    # the handle's own population
    g.randomize(3)
    o.randomize(3)
    F2, G2 = g.evaluate_packed(g.pack())
    assert (F2.cpu().numpy() == o.evaluate()[0]).all() and (G2.cpu().numpy() == o.evaluate()[1]).all()


def test_packed_candidates_errors(ones):
    w = inputs.tiny()
    g = ones.Search(w.jobs, w.capacity, w.pop)
    bad = torch.zeros((4, 1000), dtype=torch.uint8, device="cuda")    # stride not a multiple of 512
    with pytest.raises(ones.OnesError) as err:
        g.evaluate_packed(bad)
    assert err.value.code == -4
    p = ones.Search(w.jobs, w.capacity, w.pop, inputs.SearchParams(flags=16))
    with pytest.raises(ones.OnesError) as err:
        p.pack()
    assert err.value.code == -3


# ---- the generation on one-byte genes (ONES_FLAG_PACKED) ------------------------------------------------
@pytest.mark.parametrize("J,N,kw", [(1, 3, {}), (5, 4, {}), (127, 33, {}), (129, 64, {}), (513, 70, dict(p_mut=1.0)),
                                    (700, 2000, {}), (2048, 300, dict(p_mut=0.02, tournament=8)),
                                    (100, 1024, dict(elitism=0)), (260, 1025, dict(elitism=5, tournament=1)),
                                    (512, 9000, dict(p_mut=0.0)), (37, 101, dict(flags=33))])
def test_packed_generation_parity(ones, J, N, kw):
    """ones_evolve on packed rows: parents, elites, genomes, GPU demand and scores equal the oracle's after 1, 2
    and 10 generations, and the packed rows equal the packed form of the oracle's population byte for byte."""
    w = inputs.custom(J, max(4, J), N, 4, seed=J + N, kmax=7, kmin_max=2, pinned=J // 5)
    kw = dict(kw)
    if kw.get("flags", 0) & 1:
        w.jobs["weight"] = np.random.default_rng(J).uniform(1e3, 1e6, J)
    flags = kw.pop("flags", 32)
    g, o = _pair(ones, w, flags=flags, **kw)
    _same_state(g, o)  # every job at its smallest batch
    g.randomize(1)
    o.randomize(1)
    _same_state(g, o)
    for step in (1, 1, 8):
        g.evolve(step, 2 ** 33 + 5)
        o.evolve(step, 2 ** 33 + 5)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    assert (g.pack().cpu().numpy() == _pack_numpy(o.get_population(), J)).all()
    for repair in (False, True):
        bg, bo = g.best(repair), o.best(repair)
        # (with the SRUF score the library reports the per-job score terms, the oracle the throughputs)
        for key in ("genome", "gpus_per_job") + (() if flags & 1 else ("rate_per_job",)):
            assert (bg[key] == bo[key]).all(), (key, repair)
        assert bg["fitness"] == bo["fitness"] and bg["total_gpus"] == bo["total_gpus"] and bg["index"] == bo["index"]


def test_packed_generation_waiting_genes_and_job_set_change(ones):
    """Waiting jobs (-1) are inherited through crossover on packed rows, and a job-set change converts, remaps and
    packs again."""
    w = inputs.custom(300, 256, 1500, 2, seed=5, kmax=6, kmin_max=1)
    p = inputs.SearchParams(flags=32)
    g = ones.Search(w.jobs, w.capacity, w.pop, p, n_jobs_max=400, guard_bytes=4096)
    o = oracle.Search(w.jobs, w.capacity, w.pop, elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut,
                      penalty=p.penalty)
    rows = inputs.random_genomes(w.jobs, w.pop, seed=9, waiting_fraction=0.1)
    g.set_population(rows)
    o.set_population(rows)
    _same_state(g, o)
    g.evolve(3, 7)
    o.evolve(3, 7)
    _same_state(g, o)
    assert (g.get_population() == -1).any()
    rng = np.random.default_rng(3)
    jobs = w.jobs
    for rnd in range(2):
        jobs2, remap = _changed_job_set(rng, jobs, 40, 55, seed=60 + rnd, kmax_new=rnd)
        g.update_jobs(jobs2, remap, w.capacity)
        o.update_jobs(jobs2, remap, w.capacity)
        _same_state(g, o)
        g.evolve(2, rnd)
        o.evolve(2, rnd)
        _same_state(g, o)
        jobs = jobs2
    assert g.guards_intact()
    with pytest.raises(ones.OnesError) as err:   # not combinable with the truncation scheme
        ones.Search(w.jobs, w.capacity, 64, inputs.SearchParams(flags=32 | 4))
    assert err.value.code == -3


def test_packed_generation_large_config(ones):
    """The large workload on packed rows: two generations against the oracle, then 60 more against the int32 rows
    of a second handle (same seeds: populations, scores and selections must stay identical)."""
    w = inputs.large()
    g, o = _pair(ones, w, flags=32)
    h, _ = _pair(ones, w)
    for s in (g, o, h):
        s.randomize(w.seed)
    for _ in range(2):
        g.evolve(1, w.seed)
        o.evolve(1, w.seed)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    h.evolve(2, w.seed)
    g.evolve(60, w.seed)
    h.evolve(60, w.seed)
    assert torch.equal(g.evaluate()[0], h.evaluate()[0]) and torch.equal(g.evaluate()[1], h.evaluate()[1])
    assert torch.equal(g.get_population(on_device=True), h.get_population(on_device=True))
    pg, eg = g.last_parents()
    ph, eh = h.last_parents()
    assert (pg == ph).all() and (eg == eh).all()


# ---- a6: best and repair ---------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "paper", "mid"])
def test_best_and_repair_parity(ones, name):
    w = inputs.WORKLOADS[name]()
    g, o = _pair(ones, w)
    g.randomize(7)
    o.randomize(7)
    g.evolve(2, 7)
    o.evolve(2, 7)
    for repair in (False, True):
        bg, bo = g.best(repair), o.best(repair)
        for key in ("genome", "gpus_per_job", "rate_per_job"):
            assert (bg[key] == bo[key]).all(), (key, repair)
        assert bg["fitness"] == bo["fitness"] and bg["total_gpus"] == bo["total_gpus"]
        assert bg["index"] == bo["index"]
        if repair:
            assert bg["total_gpus"] <= w.capacity


def test_repair_tight_capacity(ones):
    w = inputs.custom(40, 3, 16, 1, seed=2, kmax=5)  # 40 jobs on 3 GPUs: most must wait
    g, o = _pair(ones, w)
    g.randomize(1)
    o.randomize(1)
    bg, bo = g.best(True), o.best(True)
    assert (bg["genome"] == bo["genome"]).all() and bg["total_gpus"] == bo["total_gpus"] <= 3
    assert (bg["genome"] < 0).sum() >= 37


# ---- a7: warm start across a changed job set --------------------------------------------------------
def test_update_jobs_parity(ones):
    w = inputs.paper_scale()
    p = w.params
    g = ones.Search(w.jobs, w.capacity, w.pop, p, n_jobs_max=160)
    o = oracle.Search(w.jobs, w.capacity, w.pop, elitism=p.elitism, tournament=p.tournament, p_mut=p.p_mut,
                      penalty=p.penalty)
    g.randomize(0)
    o.randomize(0)
    g.evolve(3, 0)
    o.evolve(3, 0)
    rng = np.random.default_rng(0)
    jobs = w.jobs
    for rnd in range(3):
        keep = sorted(rng.choice(jobs.shape[0], size=jobs.shape[0] - 13, replace=False).tolist())
        fresh = inputs.custom(20 + rnd, 64, 8, 1, seed=100 + rnd, kmax=0).jobs
        jobs2 = np.concatenate([jobs[keep], fresh])
        jobs2["kmax"][:len(keep)] = np.minimum(7, jobs2["kmax"][:len(keep)] + rng.integers(-1, 2, len(keep))).clip(0)
        jobs2["kmin"] = np.minimum(jobs2["kmin"], jobs2["kmax"])
        remap = np.array(keep + [-1] * fresh.shape[0], dtype=np.int32)
        g.update_jobs(jobs2, remap, 64 + rnd)
        o.update_jobs(jobs2, remap, 64 + rnd)
        _same_state(g, o)
        g.evolve(3, rnd)
        o.evolve(3, rnd)
        _same_state(g, o)
        jobs = jobs2
    with pytest.raises(ones.OnesError) as err:
        g.update_jobs(np.concatenate([jobs] * 3), np.full(3 * jobs.shape[0], -1, dtype=np.int32), 64)
    assert err.value.code == -5


@pytest.mark.parametrize("flags", [0, 32])
def test_update_jobs_same_columns(ones, flags):
    """A job-set change that keeps every job in its column: nothing moves when no range of exponents shrinks (the
    library then only rebuilds its tables), and the full pass still runs when a range shrinks or when the caller's
    own genes may lie outside the limits."""
    w = inputs.custom(300, 256, 6000, 2, seed=4, kmax=5, kmin_max=1)
    g, o = _pair(ones, w, flags=flags)
    ident = np.arange(300, dtype=np.int32)
    g.randomize(2)
    o.randomize(2)
    g.evolve(2, 2)
    o.evolve(2, 2)
    for s in (g, o):
        s.update_jobs(w.jobs, ident, w.capacity)           # the same table again
    _same_state(g, o)
    jobs2 = w.jobs.copy()
    jobs2["a"] *= 1.25
    jobs2["weight"] = 3.0
    jobs2["kmax"] = np.minimum(jobs2["kmax"] + 1, 7)        # limits grow ("Scale-up")
    for s in (g, o):
        s.update_jobs(jobs2, ident, w.capacity + 7)         # capacity moves too
    _same_state(g, o)
    g.evolve(2, 3)
    o.evolve(2, 3)
    _same_state(g, o)
    jobs3 = jobs2.copy()
    jobs3["kmax"] = np.maximum(jobs3["kmax"] - 2, jobs3["kmin"])   # limits shrink: genes are clamped
    for s in (g, o):
        s.update_jobs(jobs3, ident, w.capacity)
    _same_state(g, o)
    rows = inputs.random_genomes(jobs2, w.pop, seed=8)      # genes up to the old, larger limits
    for s in (g, o):
        s.set_population(rows)
        s.update_jobs(jobs3, ident, w.capacity)             # same table as in force, but the genes must be clamped
    _same_state(g, o)
    g.evolve(2, 4)
    o.evolve(2, 4)
    _same_state(g, o)
    bad = jobs3.copy()
    bad["a"][7] = bad["c"][7] = bad["d"][7] = 0.0            # no throughput: rejected on the host, nothing changes
    with pytest.raises(ones.OnesError) as err:
        g.update_jobs(bad, ident, w.capacity)
    assert err.value.code == -2
    _same_state(g, o)


# ---- no kernel writes outside the memory it was given ------------------------------------------------
@pytest.mark.parametrize("flags,J,gpus,N", [(0, 37, 48, 101), (0, 300, 256, 6000), (2, 129, 64, 257), (8, 260, 128, 1025),
                                            (4, 130, 64, 257), (16, 37, 130, 101), (16, 300, 257, 129), (1, 64, 64, 500), (32, 300, 256, 6000),
                                            (32, 37, 48, 101)])
def test_workspace_and_output_guards(ones, flags, J, gpus, N):
    """Every launch sequence with the workspace and the caller's output arrays between guard areas."""
    w = inputs.custom(J, gpus, N, 2, seed=J + N, kmax=6, kmin_max=1)
    g = ones.Search(w.jobs, gpus, N, inputs.SearchParams(flags=flags), n_jobs_max=J + 40, guard_bytes=4096)
    g.randomize(1)
    g.evolve(3, 1)
    g.best(repair=not flags & 16)
    jobs2 = np.concatenate([w.jobs[5:], inputs.custom(9, gpus, 4, 1, seed=3, kmax=2).jobs])
    remap = np.concatenate([np.arange(5, J), np.full(9, -1)]).astype(np.int32)
    g.update_jobs(jobs2, remap, gpus)
    g.evolve(2, 2)
    g.best()
    # outputs of ones_evaluate between guards of their own
    W = g.W
    ld = (W + 3) // 4 * 4
    rows = g.get_population(on_device=True, ld=ld)
    Fbig = torch.full((N + 64,), 7.25, dtype=torch.float64, device="cuda")
    Gbig = torch.full((N + 64,), -77, dtype=torch.int32, device="cuda")
    g.evaluate(rows, out=(Fbig[32:32 + N], Gbig[32:32 + N]))
    torch.cuda.synchronize()
    assert (Fbig[:32] == 7.25).all() and (Fbig[32 + N:] == 7.25).all()
    assert (Gbig[:32] == -77).all() and (Gbig[32 + N:] == -77).all()
    if not flags & 16:
        packed = g.pack()
        g.evaluate_packed(packed, out=(Fbig[32:32 + N], Gbig[32:32 + N]))
        torch.cuda.synchronize()
        assert (Fbig[:32] == 7.25).all() and (Fbig[32 + N:] == 7.25).all()
    assert g.guards_intact()


# ---- errors ------------------------------------------------------------------------------------
def test_errors_are_codes_not_faults(ones):
    w = inputs.tiny()
    bad = w.jobs.copy()
    bad["a"][3] = bad["c"][3] = bad["d"][3] = 0.0
    with pytest.raises(ones.OnesError) as err:
        ones.Search(bad, 16, 32)
    assert err.value.code == -2
    for kw, code in ((dict(elitism=40), -3), (dict(tournament=0), -3), (dict(p_mut=-0.1), -3),
                     (dict(p_mut=2.0 ** -18), -3)):   # a rate below the 16-bit resolution would switch mutation off
        with pytest.raises(ones.OnesError) as err:
            ones.Search(w.jobs, 16, 32, inputs.SearchParams(**kw))
        assert err.value.code == code
    s = ones.Search(w.jobs, 16, 32)
    odd = torch.zeros((4, 18), dtype=torch.int32, device="cuda")
    with pytest.raises(ones.OnesError) as err:
        s.evaluate(odd)  # ld % 4 != 0
    assert err.value.code == -4
    with pytest.raises(ones.OnesError) as err:
        s.evaluate(torch.zeros((4, 12), dtype=torch.int32, device="cuda"))  # ld < jobs
    assert err.value.code == -3
    s.evolve(1, 0)  # the handle still works


# ---- full size, in the configuration the benchmark times --------------------------------------------
@pytest.mark.parametrize("flags,gens", [(0, 3), (2, 1)])  # children scored inside the evolve kernel / by a separate pass
def test_large_config_parity_full_population(ones, flags, gens):
    w = inputs.large()
    g, o = _pair(ones, w, flags=flags)
    g.randomize(w.seed)
    o.randomize(w.seed)
    assert (g.get_population() == o.get_population()).all()
    for _ in range(gens):
        g.evolve(1, w.seed)
        o.evolve(1, w.seed)
        pg, eg = g.last_parents()
        po, eo = o.last_parents()
        assert (pg == po).all() and (eg == eo).all()
        _same_state(g, o)
    # invariants that hold at any size
    P = g.get_population()
    assert (P >= w.jobs["kmin"][None, :]).all() and (P <= w.jobs["kmax"][None, :]).all()
    b0 = g.best()["fitness"]
    g.evolve(5, w.seed)
    assert g.best()["fitness"] >= b0
    rep = g.best(True)
    assert rep["total_gpus"] <= w.capacity


def test_large_config_generation_200_recomputed_from_generation_199(ones):
    """The last generation of the large workload (2048 jobs, population 65536, 200 generations), in the launch
    sequence the benchmark times.  The random draws are keyed by (seed, generation, row, job), so any generation
    can be recomputed on its own: the oracle is given the GPU's population of generation 199 and the generation
    counter, scores it, and derives generation 200, which must equal the GPU's row for row (every tournament,
    elite, child gene, GPU demand and score).  On top, sampled pairs are re-derived from the oracle's stateless
    steps alone (tournament over the GPU's scores of generation 199; score of the GPU's child rows)."""
    w = inputs.large()
    p = w.params
    g, o = _pair(ones, w)
    g.randomize(w.seed)
    g.evolve(w.generations - 1, w.seed)
    P199 = g.get_population()
    F199 = g.evaluate()[0].cpu().numpy()
    o.set_population(P199)
    o.set_generation(w.generations - 1)
    Fo, _ = o.evaluate()
    assert (F199 == Fo).all()
    # after 199 generations the search has moved well away from its start
    g0, _ = _pair(ones, w)
    g0.randomize(w.seed)
    assert F199.max() > g0.evaluate()[0].max().item()
    g.evolve(1, w.seed)
    o.evolve(1, w.seed)
    assert g.generation == o.generation == w.generations
    pg, eg = g.last_parents()
    po, eo = o.last_parents()
    assert (pg == po).all() and (eg == eo).all()
    _same_state(g, o)
    # stateless re-derivation of sampled pairs
    P200 = g.get_population()
    F200, G200 = (t.cpu().numpy() for t in g.evaluate())
    rng = np.random.default_rng(200)
    pairs = pg.shape[0]
    for q in [0, pairs - 1] + rng.integers(0, pairs, size=254).tolist():
        for side, stream in ((0, oracle.STREAM_SEL_A), (1, oracle.STREAM_SEL_B)):
            assert pg[q, side] == oracle.tournament(F199, p.tournament, w.seed, w.generations - 1, q, stream)
        for row in (p.elitism + 2 * q, p.elitism + 2 * q + 1):
            Fr, Gr = oracle.fitness(w.jobs, w.capacity, p.penalty, P200[row])
            assert F200[row] == Fr and G200[row] == Gr
            assert np.isin(P200[row], [0, 1, 2, 3, 4, 5, 6, 7]).all()
    for r in range(p.elitism):
        assert (P200[r] == P199[eg[r]]).all()
