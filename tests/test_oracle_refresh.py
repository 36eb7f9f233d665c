"""Pins for the oracle's "Refresh" of per-GPU candidates (Section 3.2.2, Fig. 5): hand-worked rows, a
restatement in plain Python on random cases, and invariants."""
import numpy as np
import pytest

import oracle
from paper_2108_03645_b200 import inputs


def _jobs(speed, kmin=0, kmax=2):
    """Jobs whose GPU need is 2**k (b0 = max_per_gpu) and whose throughput scales with `speed`."""
    jobs = np.zeros(len(speed), dtype=inputs.JOB_DTYPE)
    for j, s in enumerate(speed):
        jobs[j] = (64, 64, kmin, kmax, 0.02 / s, 0.0005 / s, 0.001 / s, 1.0)
    return jobs


def _gain(jobs, j, count):
    """Score gained by job j from growing to its batch-size limit, from the model alone."""
    ks = [k for k in range(jobs["kmin"][j], jobs["kmax"][j] + 1) if oracle.model(jobs, j, k)[1] <= count]
    now = oracle.model(jobs, j, ks[-1])[0] if ks else 0.0
    return oracle.model(jobs, j, int(jobs["kmax"][j]))[0] - now


def test_fig5_like_example_finished_job_new_job_and_refill():
    # old jobs 0, 1, 2; job 1 has finished; new table: 0 <- old 0, 1 <- old 2, 2 = a new job; 8 GPUs
    jobs = _jobs([1.0, 1.0, 10.0])           # the new job is ten times faster: largest gain
    row = [0, 0, 1, 1, 1, 1, 2, 2]
    out = oracle.refresh(jobs, row, inv=[0, -1, 1], is_new=[0, 0, 1])
    # (1) [0,0,-,-,-,-,1,1]  (3) new job 2 on the lowest idle GPU: [0,0,2,-,-,-,1,1]
    # (4) job 2 gains most and takes the 3 GPUs it needs for its limit of 4: the cluster is full
    assert list(out) == [0, 0, 2, 2, 2, 2, 1, 1]
    # with the old jobs faster, job 0 (tie with job 1: lower index) grows to 4 and one GPU is left for job 1
    jobs = _jobs([10.0, 10.0, 1.0])
    assert _gain(jobs, 0, 2) == _gain(jobs, 1, 2) > _gain(jobs, 2, 1)
    out = oracle.refresh(jobs, row, inv=[0, -1, 1], is_new=[0, 0, 1])
    assert list(out) == [0, 0, 2, 0, 0, 1, 1, 1]


def test_new_job_takes_the_last_gpu_of_the_longest_present_job_when_nothing_is_idle():
    jobs = _jobs([1.0, 1.0, 1.0])
    out = oracle.refresh(jobs, [0, 0, 1, 1], inv=[0, 1], is_new=[0, 0, 1])
    assert list(out) == [0, 2, 1, 1]
    # a new job whose smallest batch needs two GPUs takes two: job 0 is emptied before job 1 is touched
    jobs = _jobs([1.0, 1.0, 1.0])
    jobs["kmin"][2] = 1
    out = oracle.refresh(jobs, [0, 1, 1, 0], inv=[0, 1], is_new=[0, 0, 1])
    assert list(out) == [2, 1, 1, 2]
    # two new jobs, one GPU held by old jobs: the second new job finds nothing to take
    out = oracle.refresh(_jobs([1.0, 1.0, 1.0]), [0], inv=[0], is_new=[0, 1, 1])
    assert list(out) == [1]


def test_scale_down_frees_the_last_gpus_beyond_the_limit():
    jobs = _jobs([1.0, 1.0])
    jobs["kmax"][0] = 1                       # limit now 2 GPUs, the candidate gives job 0 four
    jobs["kmax"][1] = 0                       # job 1 at its limit of one GPU: cannot use more
    out = oracle.refresh(jobs, [0, 1, 0, 0, 0], inv=[0, 1], is_new=[0, 0])
    assert list(out) == [0, 1, 0, -1, -1]     # nobody can use the two freed GPUs
    jobs["kmax"][1] = 2
    out = oracle.refresh(jobs, [0, 1, 0, 0, 0], inv=[0, 1], is_new=[0, 0])
    assert list(out) == [0, 1, 0, 1, 1]       # job 1 takes them on its way to its limit of 4


def test_nothing_to_do_leaves_the_row_alone():
    jobs = _jobs([1.0, 2.0, 3.0])
    row = [2, 2, 0, 1, 1, 1, 1, 0, 2, 2]      # 10 GPUs, limits 4: jobs 1 and 2 full, job 0 has 2, no idle GPU
    assert list(oracle.refresh(jobs, row, inv=[0, 1, 2], is_new=[0, 0, 0])) == row


def _refresh_py(jobs, row, inv, is_new):
    """The four steps restated with Python lists and the model only."""
    J = len(jobs)
    g = lambda j, k: oracle.model(jobs, j, k)[1]
    row = [inv[o] if 0 <= o < len(inv) else -1 for o in row]
    limit = [g(j, int(jobs["kmax"][j])) for j in range(J)]
    for j in range(J):
        pos = [i for i, x in enumerate(row) if x == j]
        for i in pos[limit[j]:]:
            row[i] = -1
    for j in range(J):
        if is_new[j]:
            for _ in range(g(j, int(jobs["kmin"][j]))):
                idle = [i for i, x in enumerate(row) if x < 0]
                if idle:
                    row[idle[0]] = j
                    continue
                old = [v for v in range(J) if not is_new[v] and v in row]
                if not old:
                    break
                row[max(i for i, x in enumerate(row) if x == old[0])] = j
    while -1 in row:
        open_ = [j for j in range(J) if row.count(j) < limit[j]]
        if not open_:
            break
        pick = max(open_, key=lambda j: (_gain(jobs, j, row.count(j)), -j))
        for _ in range(min(limit[pick] - row.count(pick), row.count(-1))):
            row[row.index(-1)] = pick
    return row


def test_refresh_against_the_python_restatement_and_invariants():
    rng = np.random.default_rng(5)
    for case in range(60):
        J_old, J, W = int(rng.integers(1, 9)), int(rng.integers(1, 9)), int(rng.integers(1, 40))
        w = inputs.custom(J, W, 4, 1, seed=case, kmax=int(rng.integers(0, 5)), kmin_max=1,
                          pow2=bool(case % 2))
        jobs = w.jobs
        # a random injective partial map old -> new; new jobs are those nobody maps to
        inv = np.full(J_old, -1, dtype=np.int32)
        targets = rng.permutation(J)[: int(rng.integers(0, min(J, J_old) + 1))]
        inv[rng.permutation(J_old)[: len(targets)]] = targets
        is_new = np.ones(J, dtype=np.int8)
        is_new[targets] = 0
        row = rng.integers(-1, J_old + 1, size=W)
        out = oracle.refresh(jobs, row, inv, is_new)
        assert list(out) == _refresh_py(jobs, list(row), list(inv), list(is_new)), case
        count = np.bincount(out[out >= 0], minlength=J)
        limit = np.array([oracle.model(jobs, j, int(jobs["kmax"][j]))[1] for j in range(J)])
        assert ((out >= -1) & (out < J)).all()
        assert (count <= limit).all()                       # nobody holds GPUs it cannot use
        assert (out >= 0).all() or (count == limit).all()   # an idle GPU only when every job is at its limit


def test_search_refreshes_every_candidate_at_a_job_set_change():
    w = inputs.custom(6, 16, 32, 5, seed=4, kmax=3)
    s = oracle.Search(w.jobs, w.capacity, w.pop, flags=oracle.FLAG_PER_GPU)
    s.randomize(2)
    s.evolve(3, 2)
    before = s.get_population()
    # jobs 1 and 4 finish, two new jobs arrive at the end of the table
    keep = [0, 2, 3, 5]
    w2 = inputs.custom(6, 16, 32, 5, seed=9, kmax=3)
    jobs = np.concatenate([w.jobs[keep], w2.jobs[:2]])
    remap = np.array(keep + [-1, -1], dtype=np.int32)
    s.update_jobs(jobs, remap, 16)
    after = s.get_population()
    inv = np.full(6, -1, dtype=np.int32)
    inv[keep] = np.arange(4)
    for i in range(32):
        want = oracle.reorder(oracle.refresh(jobs, before[i], inv, [0, 0, 0, 0, 1, 1]), 6)
        assert (after[i] == want).all()
    F, G = s.evaluate()
    for i in (0, 7, 31):
        assert (F[i], G[i]) == oracle.fitness_per_gpu(jobs, after[i])[:2]
    s.evolve(3, 2)                                          # and the search goes on
    assert ((s.get_population() >= -1) & (s.get_population() < 6)).all()
    with pytest.raises(oracle.OracleError):
        s.update_jobs(jobs, np.arange(6, dtype=np.int32), 17)   # the cluster keeps its size
