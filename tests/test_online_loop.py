"""The online scheduling loop (host simulation) driven by the CPU oracle, and by the CUDA library."""
import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs, online


def oracle_engine(jobs, capacity, pop, params, n_jobs_max):
    return oracle.Search(jobs, capacity, pop, elitism=params.elitism, tournament=params.tournament,
                         p_mut=params.p_mut, penalty=params.penalty, flags=params.flags)


def small_trace(seed=0, n=40, capacity=16, pop=64, gens=6):
    return inputs.online_trace(n, seed, mean_interarrival_s=20.0, median_length=2e5, sigma=1.0,
                               capacity=capacity, pop=pop, generations=gens)


def test_online_loop_invariants_with_oracle():
    tr = small_trace()
    res = online.simulate(tr, oracle_engine, keep_schedules=True)
    assert np.isfinite(res.jct).all() and (res.jct > 0).all()          # every job finishes
    assert max(res.gpus_used) <= tr.capacity                           # repair holds the capacity
    assert len(res.latency_s) == res.rounds == len(res.deployed)
    # limits: a job is at its smallest batch in its first round and may double each round after
    first = {}
    for rnd, ids, genome in res.deployed:
        for c, j in enumerate(ids):
            first.setdefault(j, rnd)
            assert genome[c] <= min(7, rnd - first[j])
    # no job can finish faster than at its best throughput over all exponents
    for j in range(tr.jobs.shape[0]):
        best_rate = max(oracle.model(tr.jobs, j, k)[0] for k in range(8))
        assert res.jct[j] >= tr.length[j] / best_rate * (1 - 1e-12)
    # deterministic
    again = online.simulate(tr, oracle_engine)
    assert (again.jct == res.jct).all() and again.best_fitness == res.best_fitness


def test_online_loop_skips_idle_time_and_respects_max_rounds():
    tr = inputs.online_trace(6, 3, mean_interarrival_s=2000.0, median_length=1e4, sigma=0.5, capacity=8, pop=32,
                             generations=3)
    res = online.simulate(tr, oracle_engine)
    assert np.isfinite(res.jct).all()
    assert res.rounds < 40  # idle stretches between far-apart arrivals are jumped over
    cut = online.simulate(tr, oracle_engine, max_rounds=2)
    assert cut.rounds == 2 and np.isnan(cut.jct).any()


def test_online_loop_regrows_engine_when_job_set_outgrows_it():
    tr = inputs.online_trace(30, 1, mean_interarrival_s=25.0, median_length=5e6, sigma=0.3, capacity=8, pop=32,
                             generations=2)
    made = []

    def eng(jobs, capacity, pop, params, n_jobs_max):
        made.append((jobs.shape[0], n_jobs_max))
        return oracle_engine(jobs, capacity, pop, params, n_jobs_max)

    res = online.simulate(tr, eng, n_jobs_max=2, max_rounds=8)
    assert len(made) >= 2 and all(n <= m for n, m in made)
    assert max(res.gpus_used) <= 8


def test_sruf_weights_follow_eq7():
    class Fixed:
        def __init__(self, rho):
            self.rho = np.asarray(rho, dtype=np.float64)

        def beta(self, a, b):
            return self.rho

    y = np.array([1000.0, 4000.0, 50.0])
    w = online.sruf_weights(y, [2, 3, 1], [2, 1, 5], Fixed([0.5, 0.25, 1.0]))
    assert (w == np.array([1000.0, 12000.0, 0.0])).all()  # Y * (1/rho - 1)
    rng = np.random.default_rng(0)
    many = np.array([online.sruf_weights([1.0], [4.0], [2.0], rng)[0] for _ in range(4000)])
    # E[1/rho - 1] for Be(4, 2) is (a + b - 1)/(a - 1) - 1 = 2/3
    assert abs(many.mean() - 2 / 3) < 0.05


def test_sruf_search_prefers_fewer_gpus_for_poorly_scaling_jobs():
    # the paper's objective (Eq. 3): with a large per-doubling cost d, holding many GPUs is wasteful
    w = inputs.custom(12, 10 ** 6, 128, 40, seed=3, kmax=5)
    jobs = w.jobs.copy()
    jobs["d"] = 0.5
    jobs["weight"] = online.sruf_weights(np.full(12, 1e5), np.full(12, 3.0), np.full(12, 3.0),
                                         np.random.default_rng(1))
    s = oracle.Search(jobs, w.capacity, w.pop, flags=oracle.FLAG_SRUF)
    s.randomize(0)
    s.evolve(40, 0)
    best = s.best()
    # exhaustive per-job optimum of weight * g / X (the score separates over jobs without a capacity limit)
    want = [min(range(6), key=lambda k: oracle.model(jobs, j, k)[1] / oracle.model(jobs, j, k)[0]) for j in range(12)]
    assert list(best["genome"]) == want


@pytest.mark.gpu
def test_sruf_evolve_gpu_matches_oracle():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding
    w = inputs.paper_scale(4)
    jobs = w.jobs.copy()
    jobs["weight"] = online.sruf_weights(np.random.default_rng(2).uniform(1e3, 1e6, 100), np.full(100, 2.0),
                                         np.full(100, 4.0), np.random.default_rng(3))
    p = inputs.SearchParams(2, 4, 0.1, 1e3, binding.FLAG_SRUF)
    g = binding.Search(jobs, w.capacity, w.pop, p)
    o = oracle.Search(jobs, w.capacity, w.pop, flags=oracle.FLAG_SRUF)
    g.randomize(1)
    o.randomize(1)
    g.evolve(20, 1)
    o.evolve(20, 1)
    assert (g.get_population() == o.get_population()).all()
    Fg, Gg = g.evaluate()
    Fo, Go = o.evaluate()
    assert (Fg.cpu().numpy() == Fo).all() and (Gg.cpu().numpy() == Go).all()
    bg, bo = g.best(True), o.best(True)
    assert (bg["genome"] == bo["genome"]).all() and bg["fitness"] == bo["fitness"]


@pytest.mark.gpu
def test_online_loop_gpu_matches_oracle():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding

    def gpu_engine(jobs, capacity, pop, params, n_jobs_max):
        return binding.Search(jobs, capacity, pop, params, n_jobs_max=n_jobs_max)

    tr = small_trace(seed=2, n=60, capacity=24, pop=256, gens=8)
    a = online.simulate(tr, gpu_engine, keep_schedules=True, n_jobs_max=16, sync=torch.cuda.synchronize)
    b = online.simulate(tr, oracle_engine, keep_schedules=True, n_jobs_max=16)
    assert a.rounds == b.rounds and a.gpus_used == b.gpus_used and a.active == b.active
    assert a.best_fitness == b.best_fitness
    for (ra, ia, ga), (rb, ib, gb) in zip(a.deployed, b.deployed):
        assert ra == rb and ia == ib and (ga == gb).all()
    assert (a.jct == b.jct).all()


@pytest.mark.gpu
def test_online_loop_full_trace_gpu_matches_oracle():
    """The online workload as specified: 2000 jobs, 256 GPUs, population 4096, 50 generations per round, every
    round of the trace.  Deployed schedules, GPU totals, best score per round and the completion time of every
    job must equal the oracle's."""
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2108_03645_b200 import binding

    def gpu_engine(jobs, capacity, pop, params, n_jobs_max):
        return binding.Search(jobs, capacity, pop, params, n_jobs_max=n_jobs_max)

    tr = inputs.online_trace()
    assert tr.jobs.shape[0] == 2000 and tr.capacity == 256 and tr.pop == 4096 and tr.generations == 50
    a = online.simulate(tr, gpu_engine, keep_schedules=True, sync=torch.cuda.synchronize)
    b = online.simulate(tr, oracle_engine, keep_schedules=True)
    assert a.rounds == b.rounds > 900 and a.active == b.active
    assert a.gpus_used == b.gpus_used and max(a.gpus_used) <= tr.capacity
    assert a.best_fitness == b.best_fitness
    for (ra, ia, ga), (rb, ib, gb) in zip(a.deployed, b.deployed):
        assert ra == rb and ia == ib and (ga == gb).all(), ra
    assert np.isfinite(a.jct).all() and (a.jct == b.jct).all()
