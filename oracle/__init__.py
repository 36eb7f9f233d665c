"""ctypes front-end of the CPU oracle (``ones_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this package.  It never imports the CUDA package
and the CUDA package never imports it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ones_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

FLAG_SRUF = 1
FLAG_TRUNCATION = 4
FLAG_PER_GPU = 16
STREAM_INIT, STREAM_SEL_A, STREAM_SEL_B, STREAM_MUT = 0, 1, 2, 3

JOB_DTYPE = np.dtype(
    [("b0", "<i4"), ("max_per_gpu", "<i4"), ("kmin", "<i4"), ("kmax", "<i4"),
     ("a", "<f8"), ("c", "<f8"), ("d", "<f8"), ("weight", "<f8")], align=True)


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"oracle: {where} failed with code {code}")
        self.code = code


class _Params(C.Structure):
    _fields_ = [("elitism", C.c_int32), ("tournament", C.c_int32), ("p_mut", C.c_double),
                ("penalty", C.c_double), ("flags", C.c_uint32)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (one rounding per operation: no FMA contraction)."""
    hdr = os.path.join(_HERE, "ones_oracle.h")
    if not force and os.path.exists(_LIB):
        if os.path.getmtime(_LIB) >= max(os.path.getmtime(_SRC), os.path.getmtime(hdr)):
            return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _configure(L: C.CDLL) -> C.CDLL:
    vp, i32, i64, u32, u64, dbl = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_double
    L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
    L.oracle_philox4x32_10.restype = None
    L.oracle_word.argtypes = [u64, u64, u32, u32, u32]
    L.oracle_word.restype = u32
    L.oracle_model.argtypes = [vp, i32, vp, vp]
    L.oracle_term.argtypes = [vp, i32, u32, vp, vp]
    L.oracle_fitness.argtypes = [vp, i32, i32, dbl, u32, vp, vp, vp]
    L.oracle_validate_jobs.argtypes = [vp, i32]
    L.oracle_repair.argtypes = [vp, i32, i32, vp]
    L.oracle_tournament.argtypes = [vp, i32, i32, u64, u64, u32, u32]
    L.oracle_tournament.restype = i32
    L.oracle_top.argtypes = [vp, i32, i32, vp]
    L.oracle_keep_best.argtypes = [vp, i32, i32, vp]
    L.oracle_fitness_per_gpu.argtypes = [vp, i32, i32, u32, vp, vp, vp, vp]
    L.oracle_reorder.argtypes = [vp, i32, i32]
    L.oracle_refresh.argtypes = [vp, i32, u32, vp, i32, vp, vp, i32]
    L.oracle_thr16.argtypes = [dbl]
    L.oracle_thr16.restype = u32
    L.oracle_create.argtypes = [vp, vp, i32, i32, i32, vp]
    L.oracle_destroy.argtypes = [vp]
    L.oracle_randomize.argtypes = [vp, u64]
    L.oracle_set_population.argtypes = [vp, vp, i64]
    L.oracle_get_population.argtypes = [vp, vp, i64]
    L.oracle_evaluate.argtypes = [vp, vp, i64, i32, vp, vp]
    L.oracle_evolve.argtypes = [vp, i32, u64]
    L.oracle_best.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp, vp]
    L.oracle_update_jobs.argtypes = [vp, vp, i32, vp, i32]
    L.oracle_last_parents.argtypes = [vp, vp, vp]
    L.oracle_generation.argtypes = [vp, vp]
    L.oracle_set_generation.argtypes = [vp, u64]
    L.oracle_pairs.argtypes = [vp]
    L.oracle_pairs.restype = i32
    return L


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = _configure(C.CDLL(build()))
    return _lib


class use_library:
    """Context manager: run the wrappers of this module against another build of the oracle
    (the tests use it to show that a planted mistake is caught by the pins)."""

    def __init__(self, path: str):
        self.path = path

    def __enter__(self):
        global _lib
        lib()
        self.saved = _lib
        _lib = _configure(C.CDLL(self.path))
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved
        return False


def _jobs_arr(jobs) -> np.ndarray:
    a = np.ascontiguousarray(jobs)
    if a.dtype.itemsize != 48:
        raise TypeError("job table rows must be 48 bytes")
    return a


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc: int, where: str):
    if rc != 0:
        raise OracleError(rc, where)


# ---- stateless pieces -------------------------------------------------------

def philox(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def word(seed: int, gen: int, row: int, col: int, stream: int) -> int:
    return int(lib().oracle_word(seed, gen, row, col, stream))


def model(jobs, j: int, k: int):
    """(X samples/s, g GPUs) of job j at exponent k."""
    a = _jobs_arr(jobs)
    X = C.c_double()
    g = C.c_int32()
    _check(lib().oracle_model(C.c_void_p(int(a.ctypes.data) + 48 * int(j)), int(k), C.byref(X), C.byref(g)), "model")
    return X.value, g.value


def term(jobs, j: int, k: int, flags: int = 0):
    a = _jobs_arr(jobs)
    X = C.c_double()
    g = C.c_int32()
    _check(lib().oracle_term(C.c_void_p(int(a.ctypes.data) + 48 * int(j)), int(k), flags, C.byref(X), C.byref(g)), "term")
    return X.value, g.value


def fitness(jobs, capacity: int, penalty: float, genome, flags: int = 0):
    a = _jobs_arr(jobs)
    gnm = np.ascontiguousarray(genome, dtype=np.int32)
    assert gnm.shape == (a.shape[0],)
    F = C.c_double()
    G = C.c_int32()
    _check(lib().oracle_fitness(_ptr(a), a.shape[0], capacity, penalty, flags, _ptr(gnm),
                                C.byref(F), C.byref(G)), "fitness")
    return F.value, G.value


def validate_jobs(jobs) -> int:
    a = _jobs_arr(jobs)
    return int(lib().oracle_validate_jobs(_ptr(a), a.shape[0]))


def repair(jobs, capacity: int, genome) -> np.ndarray:
    a = _jobs_arr(jobs)
    gnm = np.array(genome, dtype=np.int32)
    rc = lib().oracle_repair(_ptr(a), a.shape[0], capacity, _ptr(gnm))
    _check(rc, "repair")
    return gnm


def tournament(F, T: int, seed: int, gen: int, q: int, stream: int) -> int:
    f = np.ascontiguousarray(F, dtype=np.float64)
    return int(lib().oracle_tournament(_ptr(f), f.shape[0], T, seed, gen, q, stream))


def top(F, e: int) -> np.ndarray:
    f = np.ascontiguousarray(F, dtype=np.float64)
    idx = np.zeros(max(e, 1), dtype=np.int32)
    _check(lib().oracle_top(_ptr(f), f.shape[0], e, _ptr(idx)), "top")
    return idx[:e]


def fitness_per_gpu(jobs, slots, flags: int = 0):
    """(F, GPUs used, per-job exponents) of one per-GPU genome."""
    a = _jobs_arr(jobs)
    sl = np.ascontiguousarray(slots, dtype=np.int32)
    F = C.c_double()
    G = C.c_int32()
    ks = np.zeros(a.shape[0], dtype=np.int32)
    _check(lib().oracle_fitness_per_gpu(_ptr(a), a.shape[0], sl.shape[0], flags, _ptr(sl), C.byref(F), C.byref(G),
                                        _ptr(ks)), "fitness_per_gpu")
    return F.value, G.value, ks


def reorder(slots, n_jobs: int) -> np.ndarray:
    sl = np.array(slots, dtype=np.int32)
    _check(lib().oracle_reorder(_ptr(sl), sl.shape[0], n_jobs), "reorder")
    return sl


def refresh(jobs, slots, inv, is_new, flags: int = 0) -> np.ndarray:
    """One per-GPU candidate refreshed for a new job table (not packed: see `reorder`)."""
    a = _jobs_arr(jobs)
    sl = np.array(slots, dtype=np.int32)
    iv = np.ascontiguousarray(inv, dtype=np.int32)
    nw = np.ascontiguousarray(is_new, dtype=np.int8)
    assert nw.shape[0] == a.shape[0]
    _check(lib().oracle_refresh(_ptr(a), a.shape[0], flags, _ptr(iv), iv.shape[0], _ptr(nw), _ptr(sl), sl.shape[0]),
           "refresh")
    return sl


def keep_best(F, k: int) -> np.ndarray:
    f = np.ascontiguousarray(F, dtype=np.float64)
    idx = np.zeros(max(k, 1), dtype=np.int32)
    _check(lib().oracle_keep_best(_ptr(f), f.shape[0], k, _ptr(idx)), "keep_best")
    return idx[:k]


def thr16(p: float) -> int:
    return int(lib().oracle_thr16(p))


# ---- the search --------------------------------------------------------------

class Search:
    """CPU oracle search context (mirrors the CUDA library's handle, host memory only)."""

    def __init__(self, jobs, capacity: int, pop: int, *, elitism=2, tournament=4, p_mut=0.1,
                 penalty=1e3, flags=0):
        self._h = C.c_void_p()
        self.jobs = _jobs_arr(jobs).copy()
        self.J = int(self.jobs.shape[0])
        self.N = int(pop)
        self.E = int(elitism)
        self.W = int(capacity) if flags & FLAG_PER_GPU else self.J  # genes per candidate
        self.flags = int(flags)
        prm = _Params(elitism, tournament, p_mut, penalty, flags)
        rc = lib().oracle_create(C.byref(self._h), _ptr(self.jobs), self.J, capacity, pop, C.byref(prm))
        if rc != 0:
            self._h = C.c_void_p()
            raise OracleError(rc, "create")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def randomize(self, seed: int):
        _check(lib().oracle_randomize(self._h, seed), "randomize")

    def set_population(self, genomes: np.ndarray):
        g = np.ascontiguousarray(genomes, dtype=np.int32)
        assert g.shape[0] == self.N and g.shape[1] >= self.W
        _check(lib().oracle_set_population(self._h, _ptr(g), g.shape[1]), "set_population")

    def get_population(self) -> np.ndarray:
        g = np.zeros((self.N, self.W), dtype=np.int32)
        _check(lib().oracle_get_population(self._h, _ptr(g), self.W), "get_population")
        return g

    def evaluate(self, genomes: np.ndarray | None = None):
        if genomes is None:
            F = np.zeros(self.N, dtype=np.float64)
            G = np.zeros(self.N, dtype=np.int32)
            _check(lib().oracle_evaluate(self._h, None, 0, 0, _ptr(F), _ptr(G)), "evaluate")
            return F, G
        g = np.ascontiguousarray(genomes, dtype=np.int32)
        n = g.shape[0]
        F = np.zeros(n, dtype=np.float64)
        G = np.zeros(n, dtype=np.int32)
        _check(lib().oracle_evaluate(self._h, _ptr(g), g.shape[1], n, _ptr(F), _ptr(G)), "evaluate")
        return F, G

    def evolve(self, generations: int, seed: int):
        _check(lib().oracle_evolve(self._h, generations, seed), "evolve")

    def best(self, repair: bool = False) -> dict:
        genome = np.zeros(self.J, dtype=np.int32)
        gpus = np.zeros(self.J, dtype=np.int32)
        rate = np.zeros(self.J, dtype=np.float64)
        F = C.c_double()
        G = C.c_int32()
        idx = C.c_int32()
        rc = lib().oracle_best(self._h, int(repair), _ptr(genome), _ptr(gpus), _ptr(rate),
                               C.byref(F), C.byref(G), C.byref(idx))
        _check(rc, "best")
        return {"genome": genome, "gpus_per_job": gpus, "rate_per_job": rate, "fitness": F.value,
                "total_gpus": G.value, "index": idx.value}

    def update_jobs(self, jobs, remap, capacity: int):
        a = _jobs_arr(jobs).copy()
        r = np.ascontiguousarray(remap, dtype=np.int32)
        assert r.shape[0] == a.shape[0]
        _check(lib().oracle_update_jobs(self._h, _ptr(a), a.shape[0], _ptr(r), capacity), "update_jobs")
        self.jobs = a
        self.J = int(a.shape[0])
        if not self.flags & FLAG_PER_GPU:
            self.W = self.J

    def last_parents(self):
        pairs = int(lib().oracle_pairs(self._h))
        p = np.zeros((max(pairs, 1), 2), dtype=np.int32)
        e = np.zeros(max(self.E, 1), dtype=np.int32)
        _check(lib().oracle_last_parents(self._h, _ptr(p), _ptr(e)), "last_parents")
        return p[:pairs], e[:self.E]

    def set_generation(self, gen: int):
        _check(lib().oracle_set_generation(self._h, gen), "set_generation")

    @property
    def generation(self) -> int:
        g = C.c_uint64()
        _check(lib().oracle_generation(self._h, C.byref(g)), "generation")
        return int(g.value)
