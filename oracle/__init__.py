"""CPU oracle for the APOLLO / APOLLO-Mini optimizer step (test infrastructure only).

A thin ctypes wrapper over ``apollo_oracle.c``: a plain double-precision restatement of
Algorithm 1 of the APOLLO paper (with Eq. 4, the norm-growth limiter, and Eq. 5, the
channel-wise scales).  Nothing here is shared with, imported by, or imports the CUDA
library.  Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
use it; the product path never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "apollo_oracle.c"
_LIB = _HERE / "liboracle.so"

MODE_CHANNEL = 0
MODE_TENSOR = 1
DT_F32 = 0
DT_BF16 = 1


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP on the contraction's outer loop)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Config(ctypes.Structure):
    _fields_ = [
        ("rank", ctypes.c_int32), ("mode", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("bias_correction", ctypes.c_int32), ("state_bf16", ctypes.c_int32), ("pad_", ctypes.c_int32),
        ("alpha", ctypes.c_double), ("gamma", ctypes.c_double),
        ("beta1", ctypes.c_double), ("beta2", ctypes.c_double), ("eps", ctypes.c_double),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.oracle_round_bf16.restype = ctypes.c_double
        _lib.oracle_round_bf16.argtypes = [ctypes.c_double]
    return _lib


def _ptr(a, ctype):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctype))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c, ctypes.c_uint32), _ptr(k, ctypes.c_uint32), _ptr(out, ctypes.c_uint32))
    return out


def philox_draws(seed: int, matrix_id: int, epoch: int, r: int, m: int) -> np.ndarray:
    """The raw words behind P: shape (r, ceil(m/4), 4), uint32."""
    quads = (m + 3) // 4
    out = np.zeros((r, quads, 4), dtype=np.uint32)
    lib().oracle_philox_draws(ctypes.c_uint64(seed), ctypes.c_uint32(matrix_id), ctypes.c_uint32(epoch),
                              ctypes.c_int32(r), ctypes.c_int32(m), _ptr(out, ctypes.c_uint32))
    return out


def standard_normals(seed: int, matrix_id: int, epoch: int, r: int, m: int) -> np.ndarray:
    out = np.zeros((r, m), dtype=np.float64)
    lib().oracle_standard_normals(ctypes.c_uint64(seed), ctypes.c_uint32(matrix_id), ctypes.c_uint32(epoch),
                                  ctypes.c_int32(r), ctypes.c_int32(m), _ptr(out, ctypes.c_double))
    return out


def projection(seed: int, matrix_id: int, epoch: int, r: int, m: int, round_bf16: bool = False) -> np.ndarray:
    """P (r x m), entries N(0, 1/r): standard normals divided by sqrt(r) (optionally bf16-rounded first)."""
    out = np.zeros((r, m), dtype=np.float64)
    lib().oracle_projection(ctypes.c_uint64(seed), ctypes.c_uint32(matrix_id), ctypes.c_uint32(epoch),
                            ctypes.c_int32(r), ctypes.c_int32(m), ctypes.c_int32(int(round_bf16)),
                            _ptr(out, ctypes.c_double))
    return out


def round_bf16(x: float) -> float:
    return float(lib().oracle_round_bf16(ctypes.c_double(x)))


def project(P: np.ndarray, Gv: np.ndarray) -> np.ndarray:
    P = np.ascontiguousarray(P, dtype=np.float64)
    Gv = np.ascontiguousarray(Gv, dtype=np.float64)
    r, m = P.shape
    m2, n = Gv.shape
    assert m == m2
    R = np.zeros((r, n), dtype=np.float64)
    lib().oracle_project(_ptr(P, ctypes.c_double), _ptr(Gv, ctypes.c_double), ctypes.c_int32(r),
                         ctypes.c_int32(m), ctypes.c_int32(n), _ptr(R, ctypes.c_double))
    return R


class StepResult:
    __slots__ = ("W", "dW", "s", "R", "norm", "c")

    def __init__(self, W, dW, s, R, norm, c):
        self.W, self.dW, self.s, self.R, self.norm, self.c = W, dW, s, R, norm, c


class MatrixOracle:
    """Algorithm 1 for one weight matrix; holds M, V, the previous norm and t."""

    def __init__(self, rows: int, cols: int, rank: int, mode: int = MODE_CHANNEL, dtype: int = DT_F32,
                 seed: int = 0, matrix_id: int = 0, T: int = 200, alpha: float = 1.0, gamma: float = 1.01,
                 beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 bias_correction: bool = False, p_round_bf16: bool = False, state_bf16: bool = False):
        self.rows, self.cols = int(rows), int(cols)
        self.m, self.n = min(rows, cols), max(rows, cols)
        self.cfg = _Config(rank, mode, dtype, int(bias_correction), int(state_bf16), 0, alpha, gamma, beta1, beta2, eps)
        self.seed, self.matrix_id, self.T = int(seed), int(matrix_id), int(T)
        self.p_round_bf16 = bool(p_round_bf16)
        self.M = np.zeros((rank, self.n), dtype=np.float64)
        self.V = np.zeros((rank, self.n), dtype=np.float64)
        self.prev_norm = ctypes.c_double(0.0)
        self.t = 0

    def step(self, W: np.ndarray, G: np.ndarray, lr: float, wd: float, P: np.ndarray | None = None,
             want_R: bool = False) -> StepResult:
        W = np.ascontiguousarray(W, dtype=np.float32)
        G = np.ascontiguousarray(G, dtype=np.float32)
        assert W.shape == (self.rows, self.cols) and G.shape == W.shape
        r = self.cfg.rank
        W_out = np.empty_like(W)
        dW = np.empty(W.shape, dtype=np.float64)
        s = np.empty(self.n, dtype=np.float64)
        R = np.empty((r, self.n), dtype=np.float64) if want_R else None
        norm, c = ctypes.c_double(0.0), ctypes.c_double(0.0)
        common = (
            _ptr(W, ctypes.c_float), _ptr(G, ctypes.c_float), ctypes.c_int64(self.rows), ctypes.c_int64(self.cols),
            ctypes.c_int64(self.t), ctypes.c_double(lr), ctypes.c_double(wd),
            _ptr(self.M, ctypes.c_double), _ptr(self.V, ctypes.c_double), ctypes.byref(self.prev_norm),
            _ptr(W_out, ctypes.c_float), _ptr(dW, ctypes.c_double), _ptr(s, ctypes.c_double),
            _ptr(R, ctypes.c_double), ctypes.byref(norm), ctypes.byref(c),
        )
        if P is None:
            rc = lib().oracle_apollo_step(ctypes.byref(self.cfg), ctypes.c_uint64(self.seed),
                                          ctypes.c_uint32(self.matrix_id), ctypes.c_int32(self.T),
                                          ctypes.c_int32(int(self.p_round_bf16)), *common)
        else:
            P = np.ascontiguousarray(P, dtype=np.float64)
            assert P.shape == (r, self.m)
            rc = lib().oracle_apollo_step_with_P(ctypes.byref(self.cfg), _ptr(P, ctypes.c_double), *common)
        if rc != 0:
            raise ValueError(f"oracle step failed with code {rc}")
        self.t += 1
        return StepResult(W_out, dW, s, R, norm.value, c.value)


class ModelOracle:
    """Algorithm 1 over a list of matrices; matrix i draws from Philox stream matrix_id = i."""

    def __init__(self, shapes, **kw):
        self.mats = [MatrixOracle(r_, c_, matrix_id=i, **kw) for i, (r_, c_) in enumerate(shapes)]

    def step(self, Ws, Gs, lr: float, wd: float):
        return [mo.step(W, G, lr, wd) for mo, W, G in zip(self.mats, Ws, Gs)]


def adamw_step(p, g, m, v, t, lr, beta1=0.9, beta2=0.999, eps=1e-8, wd=0.0, dtype=DT_F32, bias_correction=True):
    """One AdamW step (Eq. 1 with decoupled weight decay) on flat arrays; m, v (float64) are updated.

    Returns (p_new as float32 holding values of the stored dtype, update before the final rounding)."""
    p = np.ascontiguousarray(p, dtype=np.float32).reshape(-1)
    g = np.ascontiguousarray(g, dtype=np.float32).reshape(-1)
    assert m.dtype == np.float64 and v.dtype == np.float64 and m.size == p.size and v.size == p.size
    out = np.empty_like(p)
    dp = np.empty(p.size, dtype=np.float64)
    rc = lib().oracle_adamw_step(_ptr(p, ctypes.c_float), _ptr(g, ctypes.c_float), ctypes.c_int64(p.size),
                                 ctypes.c_int32(dtype), ctypes.c_int32(int(bias_correction)), ctypes.c_double(lr),
                                 ctypes.c_double(beta1), ctypes.c_double(beta2), ctypes.c_double(eps),
                                 ctypes.c_double(wd), ctypes.c_int64(t), _ptr(m, ctypes.c_double),
                                 _ptr(v, ctypes.c_double), _ptr(out, ctypes.c_float), _ptr(dp, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle adamw step failed with code {rc}")
    return out, dp
