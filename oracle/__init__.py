"""CPU oracle for CoCoA + local SCD: a thin ctypes wrapper around ``cocoa_oracle.c``.

TEST INFRASTRUCTURE ONLY. Nothing in the product package imports this module; it is used by the tests,
by the smoke check and by the benchmark's CPU-baseline leg. It shares no code with the CUDA path.

State is held in fp64 numpy arrays; the data arrays are the caller's fp32 / int32 / int64 arrays, unchanged.
The matrix is passed coordinate-major (one compressed or dense slice per coordinate): CSR or dense rows for
the dual losses (coordinates = examples), CSC for ridge (coordinates = features).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cocoa_oracle.c")
_LIB = os.path.join(_HERE, "libcocoa_oracle.so")

HINGE, LOGISTIC, RIDGE = 0, 1, 2
LOSS_BY_NAME = {"hinge": HINGE, "logistic": LOGISTIC, "ridge": RIDGE}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over partitions) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        lib.orc_mix64.restype = c.c_uint64
        lib.orc_mix64.argtypes = [c.c_uint64]
        lib.orc_partition.restype = c.c_int
        lib.orc_partition.argtypes = [c.c_int64, c.c_int32, c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.orc_partition_sizes.restype = c.c_int
        lib.orc_partition_sizes.argtypes = [c.c_int64, c.c_int32, c.c_uint64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.orc_permutation.restype = c.c_int
        lib.orc_permutation.argtypes = [c.c_void_p, c.c_int64, c.c_uint64, c.c_int64, c.c_int64, c.c_void_p]
        lib.orc_step_hinge.restype = c.c_double
        lib.orc_step_hinge.argtypes = [c.c_double] * 3
        lib.orc_step_logistic.restype = c.c_double
        lib.orc_step_logistic.argtypes = [c.c_double] * 3 + [c.c_void_p]
        lib.orc_round.restype = c.c_int
        lib.orc_round.argtypes = [c.c_int, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64,
                                  c.c_void_p, c.c_double, c.c_void_p, c.c_void_p, c.c_int32, c.c_void_p,
                                  c.c_void_p, c.c_uint64, c.c_int64, c.c_int64, c.c_double, c.c_int, c.c_void_p]
        lib.orc_round_steps.restype = c.c_int
        lib.orc_round_steps.argtypes = [c.c_int, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64,
                                        c.c_void_p, c.c_double, c.c_void_p, c.c_void_p, c.c_int32, c.c_void_p,
                                        c.c_void_p, c.c_uint64, c.c_int64, c.c_void_p, c.c_double, c.c_int, c.c_void_p]
        lib.orc_gap.restype = c.c_int
        lib.orc_gap.argtypes = [c.c_int, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64,
                                c.c_void_p, c.c_double, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
        lib.orc_shared_vector.restype = None
        lib.orc_shared_vector.argtypes = [c.c_int64, c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64,
                                          c.c_void_p, c.c_void_p]
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def mix64(x: int) -> int:
    return int(_load().orc_mix64(ctypes.c_uint64(x & (2**64 - 1))))


def partition(n: int, K: int, seed: int, sizes=None):
    """Returns (owner[n] int32, part_off[K+1] int64, members[n] int32). ``sizes`` (K positive integers summing to n)
    cuts the same random order into blocks of those sizes instead of equal ones."""
    owner = np.empty(n, np.int32)
    off = np.empty(K + 1, np.int64)
    members = np.empty(n, np.int32)
    if sizes is None:
        rc = _load().orc_partition(n, K, ctypes.c_uint64(seed & (2**64 - 1)), _p(owner), _p(off), _p(members))
    else:
        sz = np.ascontiguousarray(sizes, np.int64)
        if sz.size != K:
            raise ValueError("sizes must have K entries")
        rc = _load().orc_partition_sizes(n, K, ctypes.c_uint64(seed & (2**64 - 1)), _p(sz), _p(owner), _p(off), _p(members))
    if rc != 0:
        raise ValueError("orc_partition: bad arguments (need 1 <= K <= n, sizes >= 1 summing to n)")
    return owner, off, members


def permutation(members_k: np.ndarray, seed: int, rnd: int, epoch: int = 0) -> np.ndarray:
    members_k = np.ascontiguousarray(members_k, np.int32)
    out = np.empty_like(members_k)
    rc = _load().orc_permutation(_p(members_k), members_k.size, ctypes.c_uint64(seed & (2**64 - 1)), rnd, epoch, _p(out))
    if rc != 0:
        raise MemoryError("orc_permutation failed")
    return out


def step_hinge(a: float, m: float, q: float) -> float:
    return float(_load().orc_step_hinge(a, m, q))


def step_logistic(a: float, m: float, q: float):
    """Returns (a_new, residual g(z) at the returned point)."""
    r = ctypes.c_double(0.0)
    a_new = float(_load().orc_step_logistic(a, m, q, ctypes.byref(r)))
    return a_new, r.value


class CocoaOracle:
    """Holds the data (by reference), the fp64 state (alpha or w, and v) and the partition map.

    ``fmt`` is "dense" (row-major, rows are the coordinates), "csr" (dual losses) or "csc" (ridge).
    ``labels`` has one entry per example: y in {-1,+1} for hinge/logistic, real targets for ridge.
    """

    def __init__(self, loss: str, fmt: str, n_rows: int, n_cols: int, values, labels, lam: float,
                 indptr=None, indices=None, threads: int = 1):
        self.loss = LOSS_BY_NAME[loss]
        self.fmt = fmt
        self.n_rows, self.n_cols = int(n_rows), int(n_cols)
        self.values = np.ascontiguousarray(values, np.float32).reshape(-1)
        self.labels = np.ascontiguousarray(labels, np.float32)
        self.indptr = None if indptr is None else np.ascontiguousarray(indptr, np.int64)
        self.indices = None if indices is None else np.ascontiguousarray(indices, np.int32)
        self.lam = float(lam)
        self.threads = int(threads)
        if self.loss == RIDGE:
            if fmt == "csc":
                self.n_coord, self.dim, self.ld = self.n_cols, self.n_rows, 0
            elif fmt == "dense_colmajor":          # tiny pins only: values[c*ld + r], ld = n_rows
                self.n_coord, self.dim, self.ld = self.n_cols, self.n_rows, self.n_rows
            else:
                raise ValueError("ridge needs csc (or dense_colmajor for tiny checks)")
        else:
            if fmt == "csr":
                self.n_coord, self.dim, self.ld = self.n_rows, self.n_cols, 0
            elif fmt == "dense":
                self.n_coord, self.dim, self.ld = self.n_rows, self.n_cols, self.n_cols
            else:
                raise ValueError("dual losses need csr or dense rows")
        assert self.labels.size == self.n_rows
        self.state = np.zeros(self.n_coord, np.float64)   # alpha (signed) or w
        self.v = np.zeros(self.dim, np.float64)
        self.round = 0
        self.K = 0
        self.seed = 0
        self.owner = self.part_off = self.members = None
        self.last_newton_resid = 0.0

    # -- a1
    def partition(self, K: int, seed: int, sizes=None):
        self.owner, self.part_off, self.members = partition(self.n_coord, K, seed, sizes)
        self.K, self.seed = int(K), int(seed)

    def partition_chunks(self, K: int, seed: int, chunk_off, chunk_task):
        """The partition that a placement of data chunks on K tasks induces (Sec. 3, Sec. 4.4); ``seed`` keys the
        visiting orders of the rounds that follow."""
        from . import chunks
        self.owner, self.part_off, self.members = chunks.partition_from_chunks(self.n_coord, K, chunk_off, chunk_task)
        self.K, self.seed = int(K), int(seed)

    def permutation(self, rnd: int, k: int, epoch: int = 0) -> np.ndarray:
        return permutation(self.members[self.part_off[k]:self.part_off[k + 1]], self.seed, rnd, epoch)

    # -- a3..a5
    def cocoa_round(self, H: int = 0, sigma_prime: Optional[float] = None, steps=None):
        """One round; ``steps`` (K non-negative integers) gives every partition a step budget of its own instead of H."""
        if self.K == 0:
            raise RuntimeError("partition() first")
        sp = float(self.K if sigma_prime is None else sigma_prime)
        resid = ctypes.c_double(0.0)
        if steps is not None:
            st = np.ascontiguousarray(steps, np.int64)
            if st.size != self.K:
                raise ValueError("steps must have K entries")
            rc = _load().orc_round_steps(self.loss, self.n_coord, self.dim, _p(self.indptr), _p(self.indices),
                                         _p(self.values), self.ld, _p(self.labels), self.lam, _p(self.state), _p(self.v),
                                         self.K, _p(self.part_off), _p(self.members), ctypes.c_uint64(self.seed),
                                         self.round, _p(st), sp, self.threads, ctypes.byref(resid))
            if rc != 0:
                raise RuntimeError("orc_round_steps failed")
            self.last_newton_resid = resid.value
            self.round += 1
            return
        rc = _load().orc_round(self.loss, self.n_coord, self.dim, _p(self.indptr), _p(self.indices),
                               _p(self.values), self.ld, _p(self.labels), self.lam, _p(self.state), _p(self.v),
                               self.K, _p(self.part_off), _p(self.members), ctypes.c_uint64(self.seed),
                               self.round, int(H), sp, self.threads, ctypes.byref(resid))
        if rc != 0:
            raise RuntimeError("orc_round failed")
        self.last_newton_resid = resid.value
        self.round += 1

    # -- a6
    def duality_gap(self, terms: bool = False):
        out = np.zeros(4, np.float64)
        t = np.empty(self.n_coord, np.float64) if terms else None
        rc = _load().orc_gap(self.loss, self.n_coord, self.dim, _p(self.indptr), _p(self.indices), _p(self.values),
                             self.ld, _p(self.labels), self.lam, _p(self.state), _p(self.v), _p(out), _p(t))
        if rc != 0:
            raise RuntimeError("dual variable outside [0,1]")
        res = {"gap": out[0], "primal": out[1], "dual": out[2], "min_term": out[3]}
        if terms:
            res["terms"] = t
        return res

    def recompute_shared_vector(self) -> np.ndarray:
        v = np.empty(self.dim, np.float64)
        _load().orc_shared_vector(self.n_coord, self.dim, _p(self.indptr), _p(self.indices), _p(self.values),
                                  self.ld, _p(self.state), _p(v))
        return v
