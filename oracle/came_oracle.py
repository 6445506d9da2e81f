"""Loader and thin driver for the CPU float64 CAME oracle (``came_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's
CPU-baseline leg use it; the CUDA product path never imports it, and this
module imports nothing from the product package.

All arithmetic is in the C file.  This module compiles it with gcc, marshals
numpy float64 arrays across ctypes and keeps the per-tensor state lists.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "came_oracle.c")
_LIB = os.path.join(_HERE, "libcame_oracle.so")
_lib = None


class HParams(ctypes.Structure):
    _fields_ = [(k, ctypes.c_double) for k in
                ("lr", "beta1", "beta2", "beta3", "eps1", "eps2", "clip_d", "weight_decay")]


class Diag(ctypes.Structure):
    _fields_ = [(k, ctypes.c_double) for k in ("sum_r", "rms_u", "sum_R")]


def build(force: bool = False) -> str:
    """Compile the oracle into a shared library next to its source (gcc, -O2, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        L.came_oracle_factor_ema.argtypes = [i64, i64, dp, ctypes.c_double, ctypes.c_double, dp, dp]
        L.came_oracle_factor_ema.restype = None
        L.came_oracle_rank1.argtypes = [i64, i64, dp, dp, dp]
        L.came_oracle_rank1.restype = ctypes.c_double
        L.came_oracle_rms.argtypes = [i64, dp]
        L.came_oracle_rms.restype = ctypes.c_double
        L.came_oracle_matrix_step.argtypes = [i64, i64, dp, dp, dp, dp, dp, dp, dp,
                                              ctypes.POINTER(HParams), dp, ctypes.POINTER(Diag)]
        L.came_oracle_matrix_step.restype = ctypes.c_int
        L.came_oracle_vector_step.argtypes = [i64, dp, dp, dp, dp, dp, ctypes.POINTER(HParams),
                                              ctypes.c_int, dp, ctypes.POINTER(Diag)]
        L.came_oracle_vector_step.restype = ctypes.c_int
        L.adafactor_oracle_matrix_step.argtypes = [i64, i64, dp, dp, dp, dp, dp,
                                                   ctypes.POINTER(HParams)]
        L.adafactor_oracle_matrix_step.restype = ctypes.c_int
        L.came_oracle_threads.argtypes = []
        L.came_oracle_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().came_oracle_threads())


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def hparams(**kw) -> HParams:
    return HParams(**{k: float(kw[k]) for k, _ in HParams._fields_})


def factor_ema(X: np.ndarray, eps: float, beta: float, row: np.ndarray, col: np.ndarray) -> None:
    n, m = X.shape
    lib().came_oracle_factor_ema(n, m, _p(X), eps, beta, _p(row), _p(col))


def rank1(row: np.ndarray, col: np.ndarray) -> np.ndarray:
    out = np.empty((row.size, col.size), dtype=np.float64)
    lib().came_oracle_rank1(row.size, col.size, _p(row), _p(col), _p(out))
    return out


def rms(u: np.ndarray) -> float:
    u = np.ascontiguousarray(u, dtype=np.float64)
    return float(lib().came_oracle_rms(u.size, _p(u)))


def matrix_step(theta, g, mom, r, c, R, C, hp: HParams, want_uhat: bool = False):
    """In-place CAME step on one matrix; returns (diag dict, uhat or None)."""
    n, m = theta.shape
    uhat = np.empty((n, m), dtype=np.float64) if want_uhat else None
    d = Diag()
    rc = lib().came_oracle_matrix_step(n, m, _p(theta), _p(g), _p(mom), _p(r), _p(c), _p(R),
                                       _p(C), ctypes.byref(hp), _p(uhat), ctypes.byref(d))
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return dict(sum_r=d.sum_r, rms_u=d.rms_u, sum_R=d.sum_R), uhat


def vector_step(theta, g, mom, v, S, hp: HParams, no_confidence: bool = False,
                want_uhat: bool = False):
    N = theta.size
    uhat = np.empty(N, dtype=np.float64) if want_uhat else None
    d = Diag()
    rc = lib().came_oracle_vector_step(N, _p(theta), _p(g), _p(mom), _p(v), _p(S),
                                       ctypes.byref(hp), int(no_confidence), _p(uhat),
                                       ctypes.byref(d))
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return dict(rms_u=d.rms_u), uhat


def adafactor_matrix_step(theta, g, mom, r, c, hp: HParams) -> None:
    n, m = theta.shape
    rc = lib().adafactor_oracle_matrix_step(n, m, _p(theta), _p(g), _p(mom), _p(r), _p(c),
                                            ctypes.byref(hp))
    if rc != 0:
        raise MemoryError("oracle allocation failed")


class OracleOptimizer:
    """CAME state for a list of tensors, all float64, stepped by the C oracle.

    ``shapes`` are ``(rows,)`` for vectors and ``(rows, cols)`` for matrices.
    State starts at zero (m_0 = r_0 = c_0 = 0 as listed in Algorithm 2, and
    R_0 = C_0 = 0 by the same convention).
    """

    def __init__(self, params: Sequence[np.ndarray], no_weight_decay: Sequence[bool] = (),
                 vec_no_confidence: Sequence[bool] = (), algorithm: str = "came"):
        assert algorithm in ("came", "adafactor")   # Algorithm 2 or Algorithm 1
        self.algorithm = algorithm
        self.p: List[np.ndarray] = [np.ascontiguousarray(x, dtype=np.float64).copy() for x in params]
        self.m = [np.zeros_like(x) for x in self.p]
        self.r, self.c, self.R, self.C = [], [], [], []
        for x in self.p:
            if x.ndim == 2:
                n, m = x.shape
                self.r.append(np.zeros(n)); self.c.append(np.zeros(m))
                self.R.append(np.zeros(n)); self.C.append(np.zeros(m))
            elif x.ndim == 1:
                self.r.append(np.zeros(x.size)); self.c.append(None)   # r holds v
                self.R.append(np.zeros(x.size)); self.C.append(None)   # R holds S
            else:
                raise ValueError("only vectors and matrices are defined")
        k = len(self.p)
        self.no_wd = list(no_weight_decay) or [False] * k
        self.no_conf = list(vec_no_confidence) or [False] * k

    def step(self, grads: Sequence[np.ndarray], **hp_kw) -> None:
        """grads: float64 arrays (already widened from the exact fp32/bf16 inputs)."""
        for i, g in enumerate(grads):
            self.step_tensor(i, g, **hp_kw)

    def step_tensor(self, i: int, g: np.ndarray, **hp_kw) -> None:
        kw = dict(hp_kw)
        if self.no_wd[i]:
            kw["weight_decay"] = 0.0
        hp = hparams(**kw)
        g = np.ascontiguousarray(g, dtype=np.float64)
        if self.p[i].ndim == 2:
            if self.algorithm == "adafactor":
                adafactor_matrix_step(self.p[i], g, self.m[i], self.r[i], self.c[i], hp)
            else:
                matrix_step(self.p[i], g, self.m[i], self.r[i], self.c[i], self.R[i], self.C[i], hp)
        else:
            vector_step(self.p[i], g, self.m[i], self.r[i], self.R[i], hp,
                        no_confidence=self.no_conf[i] or self.algorithm == "adafactor")
