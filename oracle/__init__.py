"""CPU oracle for the CD-GraB PairBalance ordering path -- TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper over ``pairbalance_oracle.c`` (plain C, fp64) plus a numpy fp64
statement of the per-example logistic-regression gradient.  Nothing here is part of the
product: only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it, and it imports nothing from the CUDA package.

Paper passages followed (arXiv 2302.00845, algorithms numbered in order of appearance):
Algorithm 7 (server-side PairBalance over a set of vectors) for the loops and the
front/back pointers, Algorithm 6 (balancing without normalization) for the sign rule,
Algorithm 2 (PairBalance) for the pair difference z1 - z2, Algorithm 1 (reorder by
balanced signs) for the permutation, Algorithm 4 (parameter server) for the epoch reset.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pairbalance_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.cdo_create.restype = C.c_void_p
        lib.cdo_create.argtypes = [C.c_int, C.c_int, C.c_longlong]
        lib.cdo_destroy.argtypes = [C.c_void_p]
        lib.cdo_set_perms.argtypes = [C.c_void_p, C.c_void_p]
        lib.cdo_begin_epoch.argtypes = [C.c_void_p]
        lib.cdo_balance_one.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int,
                                        C.c_int, C.c_double]
        lib.cdo_balance_one_randomized.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int,
                                                   C.c_double, C.c_double, C.c_int, C.c_double]
        lib.cdo_out_of_bound.restype = C.c_longlong
        lib.cdo_out_of_bound.argtypes = [C.c_void_p]
        lib.cdo_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_double]
        lib.cdo_end_epoch.argtypes = [C.c_void_p, C.c_void_p]
        for name in ("cdo_get_r", "cdo_get_signs", "cdo_get_own_signs", "cdo_get_perm_cur",
                     "cdo_get_perm_next"):
            getattr(lib, name).argtypes = [C.c_void_p, C.c_void_p]
            getattr(lib, name).restype = None
        lib.cdo_get_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.cdo_get_trace.restype = None
        lib.cdo_near_ties.restype = C.c_longlong
        lib.cdo_near_ties.argtypes = [C.c_void_p]
        lib.cdo_mismatches.restype = C.c_longlong
        lib.cdo_mismatches.argtypes = [C.c_void_p]
        lib.cdo_pairs_done.argtypes = [C.c_void_p]
        lib.cdo_threads.restype = C.c_int
        lib.cdo_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.cdo_philox4x32_10.restype = None
        lib.cdo_uniform.argtypes = [C.c_ulonglong, C.c_uint, C.c_uint, C.c_uint]
        lib.cdo_uniform.restype = C.c_double
        _lib = lib
    return _lib


def _as_rows(a: np.ndarray):
    """Accept float32 arrays, or bfloat16 bit patterns as uint16/int16; return (array, dtype code)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype in (np.uint16, np.int16):
        return a, BF16
    raise TypeError(f"oracle rows must be float32 or bfloat16 bit patterns (uint16), got {a.dtype}")


class PairBalanceOracle:
    """fp64 sequential PairBalance + reorder for m workers with n items each in R^d."""

    def __init__(self, m: int, n: int, d: int):
        lib = _load()
        self._h = lib.cdo_create(m, n, d)
        if not self._h:
            raise ValueError("oracle: need m >= 1, even n >= 2, d >= 1")
        self.m, self.n, self.d = m, n, d

    def close(self):
        if self._h:
            _load().cdo_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_perms(self, perms: np.ndarray):
        p = np.ascontiguousarray(perms, dtype=np.int32)
        assert p.shape == (self.m, self.n)
        if _load().cdo_set_perms(self._h, p.ctypes.data) != 0:
            raise RuntimeError("oracle: set_perms inside an open epoch")

    def begin_epoch(self):
        if _load().cdo_begin_epoch(self._h) != 0:
            raise RuntimeError("oracle: epoch already open")

    def balance_one(self, i: int, g_prev: np.ndarray, g_cur: np.ndarray, replay: int = 0,
                    tau: float = 0.0) -> int:
        """PairBalance for worker i at the current pair index; returns the adopted sign."""
        gp, dt = _as_rows(g_prev)
        gc, dt2 = _as_rows(g_cur)
        assert dt == dt2 and gp.size == self.d and gc.size == self.d
        s = _load().cdo_balance_one(self._h, i, gp.ctypes.data, gc.ctypes.data, dt, int(replay),
                                    float(tau))
        if s == 0:
            raise RuntimeError("oracle: balance_one out of order or outside an epoch")
        return s

    def balance_one_randomized(self, i: int, g_prev: np.ndarray, g_cur: np.ndarray, u: float, w: float,
                               replay: int = 0, tau: float = 0.0) -> int:
        """RandomizedBalance (Algorithm 2's subroutine with Algorithm 5's bound w) for worker i:
        p = 1/2 - <r,c>/(2w), sign +1 iff u < p."""
        gp, dt = _as_rows(g_prev)
        gc, dt2 = _as_rows(g_cur)
        assert dt == dt2 and gp.size == self.d and gc.size == self.d
        s = _load().cdo_balance_one_randomized(self._h, i, gp.ctypes.data, gc.ctypes.data, dt, float(u),
                                               float(w), int(replay), float(tau))
        if s == 0:
            raise RuntimeError("oracle: randomized balance out of order, outside an epoch, or w <= 0")
        return s

    def step_randomized(self, grads: np.ndarray, u: np.ndarray, w: float, replay: np.ndarray | None = None,
                        tau: float = 0.0):
        g, _ = _as_rows(grads)
        assert g.shape == (2, self.m, self.d) and len(u) == self.m
        for i in range(self.m):
            self.balance_one_randomized(i, g[0, i], g[1, i], float(u[i]), w,
                                        0 if replay is None else int(replay[i]), tau)

    @property
    def out_of_bound(self) -> int:
        return int(_load().cdo_out_of_bound(self._h))

    def step(self, grads: np.ndarray, replay: np.ndarray | None = None, tau: float = 0.0):
        """grads: [2][m][d]; slab 0 holds the earlier vector of every worker's pair."""
        g, dt = _as_rows(grads)
        assert g.shape == (2, self.m, self.d), g.shape
        rp = None
        if replay is not None:
            rp = np.ascontiguousarray(replay, dtype=np.int8)
            assert rp.shape == (self.m,)
        if _load().cdo_step(self._h, g.ctypes.data, dt, rp.ctypes.data if rp is not None else None,
                            float(tau)) != 0:
            raise RuntimeError("oracle: step outside an epoch or past n/2 pairs")

    def end_epoch(self) -> np.ndarray:
        out = np.empty((self.m, self.n), dtype=np.int32)
        if _load().cdo_end_epoch(self._h, out.ctypes.data) != 0:
            raise RuntimeError("oracle: end_epoch before all n/2 pairs were balanced")
        return out

    # read-back -----------------------------------------------------------------------
    def r(self) -> np.ndarray:
        out = np.empty(self.d, dtype=np.float64)
        _load().cdo_get_r(self._h, out.ctypes.data)
        return out

    def signs(self) -> np.ndarray:
        out = np.empty((self.m, self.n // 2), dtype=np.int8)
        _load().cdo_get_signs(self._h, out.ctypes.data)
        return out

    def own_signs(self) -> np.ndarray:
        out = np.empty((self.m, self.n // 2), dtype=np.int8)
        _load().cdo_get_own_signs(self._h, out.ctypes.data)
        return out

    def perm_cur(self) -> np.ndarray:
        out = np.empty((self.m, self.n), dtype=np.int32)
        _load().cdo_get_perm_cur(self._h, out.ctypes.data)
        return out

    def perm_next(self) -> np.ndarray:
        out = np.empty((self.m, self.n), dtype=np.int32)
        _load().cdo_get_perm_next(self._h, out.ctypes.data)
        return out

    def trace(self):
        """(t, ||r||, ||c||) recorded before each update, each [m][n/2]."""
        shp = (self.m, self.n // 2)
        t = np.empty(shp); rn = np.empty(shp); cn = np.empty(shp)
        _load().cdo_get_trace(self._h, t.ctypes.data, rn.ctypes.data, cn.ctypes.data)
        return t, rn, cn

    @property
    def near_ties(self) -> int:
        return int(_load().cdo_near_ties(self._h))

    @property
    def mismatches(self) -> int:
        return int(_load().cdo_mismatches(self._h))

    @property
    def pairs_done(self) -> int:
        return int(_load().cdo_pairs_done(self._h))


def threads() -> int:
    """Number of OpenMP threads the C oracle will use."""
    return int(_load().cdo_threads())


def philox4x32_10(ctr, key) -> np.ndarray:
    """Philox4x32-10 block: counter of four and key of two 32-bit words -> four 32-bit words."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    assert c.shape == (4,) and k.shape == (2,)
    _load().cdo_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def uniform(seed: int, epoch: int, k: int, i: int) -> float:
    """The draw RandomizedBalance uses for worker i at pair index k of an epoch, u in [0,1)."""
    return float(_load().cdo_uniform(int(seed), int(epoch), int(k), int(i)))


def logistic_grad(x: np.ndarray, y: float, w: np.ndarray) -> np.ndarray:
    """Per-example gradient of the logistic loss log(1+e^z) - y z at z = <w,x>, in fp64:
    (sigma(z) - y) x with sigma(z) = 1/(1+e^-z) and y in {0,1}.  The paper's workers compute
    the per-example gradient of their loss (Algorithm 3); the logistic-regression task is its
    first experiment (Section 5)."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    z = float(np.dot(w, x))
    sig = 1.0 / (1.0 + np.exp(-z))
    return (sig - float(y)) * x


def herding_objective(z: np.ndarray, perms: np.ndarray) -> float:
    """Parallel herding objective, Eq. (7): max over k of the infinity norm of
    sum_{j<=k} sum_i (z[i, perms[i, j]] - mean), z: [m][n][d], perms: [m][n]."""
    z = np.asarray(z, dtype=np.float64)
    m, n, d = z.shape
    zbar = z.reshape(m * n, d).mean(axis=0)
    acc = np.zeros(d)
    best = 0.0
    for j in range(n):
        for i in range(m):
            acc += z[i, perms[i, j]] - zbar
        best = max(best, float(np.abs(acc).max()))
    return best
