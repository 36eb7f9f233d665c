"""Thin ctypes binding of ``libones.so`` (argument marshalling only).

PyTorch is used for device memory and streams: the workspace, genome tables and
score vectors are torch CUDA tensors whose ``data_ptr()`` crosses the C ABI.
There is no CPU path: if the library cannot be loaded, importing this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build
from .inputs import JOB_DTYPE, SearchParams

FLAG_SRUF = 1
FLAG_UNFUSED = 2
FLAG_TRUNCATION = 4
FLAG_NO_CLUSTER = 8
FLAG_PER_GPU = 16
FLAG_PACKED = 32
MAX_ELITES = 256

ERRORS = {0: "ONES_OK", -1: "ONES_ERR_NULL", -2: "ONES_ERR_BAD_JOB", -3: "ONES_ERR_BAD_PARAM",
          -4: "ONES_ERR_ALIGN", -5: "ONES_ERR_WORKSPACE", -6: "ONES_ERR_CUDA", -7: "ONES_ERR_INFEASIBLE",
          -8: "ONES_ERR_NOMEM"}


class OnesError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        name = ERRORS.get(code, str(code))
        super().__init__(f"{where}: {name} ({lib().ones_strerror(code).decode()}){detail}")
        self.code = code


class ones_params(C.Structure):
    _fields_ = [("elitism", C.c_int32), ("tournament", C.c_int32), ("p_mut", C.c_double),
                ("penalty", C.c_double), ("flags", C.c_uint32)]


_lib = None

_SIGNATURES = {
    "ones_workspace_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "ones_workspace_bytes_flags": (C.c_size_t, [C.c_int32, C.c_int32, C.c_uint32]),
    "ones_workspace_bytes_per_gpu": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32]),
    "ones_create": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                              C.c_size_t, C.c_void_p]),
    "ones_destroy": (C.c_int, [C.c_void_p]),
    "ones_randomize": (C.c_int, [C.c_void_p, C.c_uint64]),
    "ones_set_population": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int]),
    "ones_get_population": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int]),
    "ones_evaluate": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p]),
    "ones_packed_row_bytes": (C.c_size_t, [C.c_int32]),
    "ones_pack_population": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64]),
    "ones_evaluate_packed": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p]),
    "ones_evolve": (C.c_int, [C.c_void_p, C.c_int32, C.c_uint64]),
    "ones_best": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                            C.c_void_p]),
    "ones_update_jobs": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32]),
    "ones_last_parents": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "ones_model_table": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ones_select_top_scratch_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "ones_select_top": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t,
                                  C.c_void_p]),
    "ones_select_top_noalloc": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "ones_generation": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ones_set_generation": (C.c_int, [C.c_void_p, C.c_uint64]),
    "ones_shape": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ones_kernel_launches": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ones_set_profiling": (C.c_int, [C.c_void_p, C.c_int]),
    "ones_stage_times": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "ones_last_cuda_error": (C.c_int, [C.c_void_p]),
    "ones_strerror": (C.c_char_p, [C.c_int]),
}


def lib() -> C.CDLL:
    """The loaded library; raises if it is missing (there is no fallback)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: run paper_2108_03645_b200/build.py (needs nvcc)")
        L = C.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _np_ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _t_ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def workspace_bytes(n_jobs_max: int, pop: int, flags: int = 0) -> int:
    return int(lib().ones_workspace_bytes_flags(n_jobs_max, pop, flags))


def select_top(fitness: torch.Tensor, e: int) -> torch.Tensor:
    """``ones_select_top``: indices of the e best scores (device tensors)."""
    assert fitness.is_cuda and fitness.dtype == torch.float64 and fitness.is_contiguous()
    n = fitness.numel()
    nbytes = int(lib().ones_select_top_scratch_bytes(n, e))
    if nbytes == 0:
        raise OnesError(-3, "ones_select_top_scratch_bytes")
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=fitness.device)
    out = torch.empty(e, dtype=torch.int32, device=fitness.device)
    rc = lib().ones_select_top(_t_ptr(fitness), n, e, _t_ptr(out), _t_ptr(scratch), nbytes, _stream_ptr())
    if rc:
        raise OnesError(rc, "ones_select_top")
    return out


NOALLOC_MAX_TOP = 64


def select_top_noalloc(fitness: torch.Tensor, e: int, out: torch.Tensor) -> torch.Tensor:
    """``ones_select_top_noalloc``: as `select_top`, but the library's built-in scratch is used and
    the caller supplies the output tensor, so nothing is allocated on the way (for callers that
    cannot get device memory at call time).  Calls that may overlap on the GPU must be serialised."""
    assert fitness.is_cuda and fitness.dtype == torch.float64 and fitness.is_contiguous()
    assert out.is_cuda and out.dtype == torch.int32 and out.is_contiguous() and out.numel() >= e
    rc = lib().ones_select_top_noalloc(_t_ptr(fitness), fitness.numel(), e, _t_ptr(out), _stream_ptr())
    if rc:
        raise OnesError(rc, "ones_select_top_noalloc")
    return out


class Search:
    """One ``ones_ctx``: a population of candidate schedules on the current CUDA device."""

    def __init__(self, jobs: np.ndarray, capacity: int, pop: int, params: SearchParams | None = None, *,
                 n_jobs_max: int | None = None, guard_bytes: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self._h = C.c_void_p()
        jobs = np.ascontiguousarray(jobs, dtype=JOB_DTYPE)
        p = params or SearchParams()
        self.params = p
        self.N = int(pop)
        self.J = int(jobs.shape[0])
        self.capacity = int(capacity)
        nmax = max(self.J, int(n_jobs_max or 0))
        self.W = int(capacity) if p.flags & FLAG_PER_GPU else self.J  # genes per candidate
        if p.flags & FLAG_PER_GPU:
            nbytes = int(lib().ones_workspace_bytes_per_gpu(nmax, pop, capacity))
        else:
            nbytes = workspace_bytes(nmax, pop, p.flags)
        if nbytes == 0:
            raise OnesError(-3, "ones_workspace_bytes")
        self.device = torch.device("cuda", torch.cuda.current_device())
        # guard_bytes > 0 (a multiple of 256): the workspace sits between two guard areas filled with a
        # pattern, and guards_intact() tells whether any kernel wrote outside the workspace it was given
        assert guard_bytes % 256 == 0
        self._guard = int(guard_bytes)
        self._arena = torch.empty(nbytes + 2 * self._guard, dtype=torch.uint8, device=self.device)
        if self._guard:
            self._arena[:self._guard].fill_(0xA5)
            self._arena[-self._guard:].fill_(0xA5)
        self.workspace = self._arena[self._guard:self._guard + nbytes]
        prm = ones_params(p.elitism, p.tournament, p.p_mut, p.penalty, p.flags)
        rc = lib().ones_create(C.byref(self._h), _np_ptr(jobs), self.J, capacity, pop, C.byref(prm),
                               _t_ptr(self.workspace), nbytes, _stream_ptr())
        if rc:
            self._h = C.c_void_p()
            raise OnesError(rc, "ones_create")

    def guards_intact(self) -> bool:
        torch.cuda.synchronize()
        g = self._guard
        return g == 0 or bool((self._arena[:g] == 0xA5).all() and (self._arena[-g:] == 0xA5).all())

    # -- lifetime ---------------------------------------------------------------
    def close(self):
        if getattr(self, "_h", None):
            lib().ones_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc:
            detail = ""
            if rc == -6:
                detail = f" cudaError={lib().ones_last_cuda_error(self._h)}"
            raise OnesError(rc, where, detail)

    # -- population ---------------------------------------------------------------
    def randomize(self, seed: int):
        self._check(lib().ones_randomize(self._h, seed), "ones_randomize")

    def set_population(self, genomes):
        if isinstance(genomes, torch.Tensor):
            assert genomes.is_cuda and genomes.dtype == torch.int32 and genomes.is_contiguous()
            assert genomes.shape[0] == self.N
            rc = lib().ones_set_population(self._h, _t_ptr(genomes), genomes.shape[1], 1)
        else:
            g = np.ascontiguousarray(genomes, dtype=np.int32)
            assert g.shape[0] == self.N
            rc = lib().ones_set_population(self._h, _np_ptr(g), g.shape[1], 0)
        self._check(rc, "ones_set_population")

    def get_population(self, on_device: bool = False, ld: int | None = None):
        ld = self.W if ld is None else ld
        if on_device:
            out = torch.zeros((self.N, ld), dtype=torch.int32, device=self.device)
            rc = lib().ones_get_population(self._h, _t_ptr(out), ld, 1)
        else:
            out = np.zeros((self.N, ld), dtype=np.int32)
            rc = lib().ones_get_population(self._h, _np_ptr(out), ld, 0)
        self._check(rc, "ones_get_population")
        return out

    # -- the hot path ---------------------------------------------------------------
    def evaluate(self, genomes: torch.Tensor | None = None, out=None):
        """Scores and GPU demand (device tensors) of `genomes`, or of the current population."""
        if genomes is None:
            n, ld, ptr = self.N, 0, None
        else:
            assert genomes.is_cuda and genomes.dtype == torch.int32 and genomes.is_contiguous()
            n, ld, ptr = genomes.shape[0], genomes.shape[1], _t_ptr(genomes)
        if out is None:
            F = torch.empty(n, dtype=torch.float64, device=self.device)
            G = torch.empty(n, dtype=torch.int32, device=self.device)
        else:
            F, G = out
        if genomes is not None and n == 0:
            return F, G  # an empty tensor has no address to pass
        self._check(lib().ones_evaluate(self._h, ptr, ld, n, _t_ptr(F), _t_ptr(G)), "ones_evaluate")
        return F, G

    def pack(self, genomes: torch.Tensor | None = None) -> torch.Tensor:
        """`genomes` (device int32[n, ld]), or the current population, as packed rows: uint8[n, ld8]."""
        ld8 = int(lib().ones_packed_row_bytes(self.J))
        if genomes is None:
            n, ld, ptr = self.N, 0, None
        else:
            assert genomes.is_cuda and genomes.dtype == torch.int32 and genomes.is_contiguous()
            n, ld, ptr = genomes.shape[0], genomes.shape[1], _t_ptr(genomes)
        packed = torch.empty((n, ld8), dtype=torch.uint8, device=self.device)
        if n:
            self._check(lib().ones_pack_population(self._h, ptr, ld, n, _t_ptr(packed), ld8), "ones_pack_population")
        return packed

    def evaluate_packed(self, packed: torch.Tensor, out=None):
        """Scores and GPU demand of packed rows (see `pack`)."""
        assert packed.is_cuda and packed.dtype == torch.uint8 and packed.is_contiguous()
        n, ld8 = packed.shape
        if out is None:
            F = torch.empty(n, dtype=torch.float64, device=self.device)
            G = torch.empty(n, dtype=torch.int32, device=self.device)
        else:
            F, G = out
        if n:
            self._check(lib().ones_evaluate_packed(self._h, _t_ptr(packed), ld8, n, _t_ptr(F), _t_ptr(G)),
                        "ones_evaluate_packed")
        return F, G

    def evolve(self, generations: int, seed: int):
        self._check(lib().ones_evolve(self._h, generations, seed), "ones_evolve")

    def best(self, repair: bool = False) -> dict:
        genome = np.zeros(self.J, dtype=np.int32)
        gpus = np.zeros(self.J, dtype=np.int32)
        rate = np.zeros(self.J, dtype=np.float64)
        F, G, idx = C.c_double(), C.c_int32(), C.c_int32()
        rc = lib().ones_best(self._h, int(repair), _np_ptr(genome), _np_ptr(gpus), _np_ptr(rate), C.byref(F),
                             C.byref(G), C.byref(idx))
        self._check(rc, "ones_best")
        return {"genome": genome, "gpus_per_job": gpus, "rate_per_job": rate, "fitness": F.value,
                "total_gpus": G.value, "index": idx.value}

    def update_jobs(self, jobs: np.ndarray, remap, capacity: int):
        jobs = np.ascontiguousarray(jobs, dtype=JOB_DTYPE)
        r = np.ascontiguousarray(remap, dtype=np.int32)
        assert r.shape[0] == jobs.shape[0]
        self._check(lib().ones_update_jobs(self._h, _np_ptr(jobs), jobs.shape[0], _np_ptr(r), capacity),
                    "ones_update_jobs")
        self.J = int(jobs.shape[0])
        if not self.params.flags & FLAG_PER_GPU:
            self.W = self.J
        self.capacity = int(capacity)

    # -- inspection ---------------------------------------------------------------
    def last_parents(self):
        pairs = self.N if self.params.flags & FLAG_TRUNCATION else (self.N - self.params.elitism + 1) // 2
        p = np.zeros((max(pairs, 1), 2), dtype=np.int32)
        e = np.zeros(max(self.params.elitism, 1), dtype=np.int32)
        self._check(lib().ones_last_parents(self._h, _np_ptr(p), _np_ptr(e)), "ones_last_parents")
        return p[:pairs], e[:self.params.elitism]

    def model_table(self):
        planes = C.c_int32()
        self._check(lib().ones_model_table(self._h, None, None, C.byref(planes)), "ones_model_table")
        X = np.zeros((planes.value, self.J), dtype=np.float64)
        g = np.zeros((planes.value, self.J), dtype=np.int32)
        self._check(lib().ones_model_table(self._h, _np_ptr(X), _np_ptr(g), C.byref(planes)), "ones_model_table")
        return X, g

    def set_generation(self, gen: int):
        self._check(lib().ones_set_generation(self._h, gen), "ones_set_generation")

    @property
    def generation(self) -> int:
        g = C.c_uint64()
        self._check(lib().ones_generation(self._h, C.byref(g)), "ones_generation")
        return int(g.value)

    @property
    def kernel_launches(self) -> int:
        n = C.c_uint64()
        self._check(lib().ones_kernel_launches(self._h, C.byref(n)), "ones_kernel_launches")
        return int(n.value)

    def set_profiling(self, on):
        """False/0 off, True/1 every generation, n > 1 every n-th generation."""
        self._check(lib().ones_set_profiling(self._h, int(on)), "ones_set_profiling")

    def stage_times(self):
        """({'fitness': ms, 'select': ms, 'evolve': ms}, counts) since the last call."""
        ms = (C.c_double * 3)()
        cnt = (C.c_uint64 * 3)()
        self._check(lib().ones_stage_times(self._h, ms, cnt), "ones_stage_times")
        names = ("fitness", "select", "evolve")
        return {k: ms[i] for i, k in enumerate(names)}, {k: int(cnt[i]) for i, k in enumerate(names)}
