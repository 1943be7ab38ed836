"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, see ada_oracle.c).

Argument marshalling only; every number is computed by the C file next to it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ada_oracle.c")
_LIB = os.path.join(_HERE, "libada_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB,
               _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = C.CDLL(_LIB)
        dp, ip, bp = C.POINTER(C.c_double), C.POINTER(C.c_int32), C.POINTER(C.c_uint8)
        i64 = C.c_int64
        lib.ada_oracle_num_threads.restype = C.c_int
        lib.ada_oracle_set_threads.argtypes = [C.c_int]
        lib.ada_oracle_normalize.argtypes = [dp, i64, i64, dp, dp]
        lib.ada_oracle_normalize.restype = None
        lib.ada_oracle_full.argtypes = [dp, i64, i64, C.c_double, dp, ip]
        lib.ada_oracle_full.restype = i64
        lib.ada_oracle_full_rows.argtypes = [dp, i64, i64, ip, i64, dp]
        lib.ada_oracle_full_rows.restype = C.c_int
        lib.ada_oracle_cascade.argtypes = [dp, i64, i64, C.c_double, ip, i64, C.c_int, bp,
                                           ip, i64, dp, dp, ip, ip, ip, C.POINTER(i64)]
        lib.ada_oracle_cascade.restype = C.c_int
        lib.ada_oracle_nearest.argtypes = [dp, i64, i64, ip, i64, ip, dp]
        lib.ada_oracle_nearest.restype = C.c_int
        lib.ada_oracle_op_count.argtypes = [C.c_int, i64, i64, i64]
        lib.ada_oracle_op_count.restype = C.c_uint64
        lib.ada_oracle_jaccard.argtypes = [ip, i64, ip, i64]
        lib.ada_oracle_jaccard.restype = C.c_double
        lib.ada_oracle_turnover.argtypes = [i64, i64, i64]
        lib.ada_oracle_turnover.restype = C.c_double
        lib.ada_oracle_attention_reps.argtypes = [dp, dp, dp, i64, i64, i64, ip, i64, ip, C.c_int, dp]
        lib.ada_oracle_attention_reps.restype = C.c_int
        lib.ada_oracle_tau_update.argtypes = [C.c_double] * 6
        lib.ada_oracle_tau_update.restype = C.c_double
        _lib = lib
    return _lib


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _x(X) -> np.ndarray:
    X = np.ascontiguousarray(X, dtype=np.float64)
    if X.ndim != 2:
        raise ValueError("X must be T x d")
    return X


def num_threads() -> int:
    return int(_load().ada_oracle_num_threads())


def set_threads(n: int) -> None:
    _load().ada_oracle_set_threads(int(n))


def normalize(X):
    X = _x(X)
    T, d = X.shape
    Xhat = np.empty_like(X)
    norm = np.empty(T, dtype=np.float64)
    _load().ada_oracle_normalize(_dp(X), T, d, _dp(Xhat), _dp(norm))
    return Xhat, norm


def select_full(X, tau: float):
    """Definition 1.  Returns (rep ascending int32, gamma float64[T])."""
    X = _x(X)
    T, d = X.shape
    gamma = np.empty(T, dtype=np.float64)
    rep = np.empty(T, dtype=np.int32)
    r = _load().ada_oracle_full(_dp(X), T, d, float(tau), _dp(gamma), _ip(rep))
    if r < 0:
        raise MemoryError
    return rep[:r].copy(), gamma


def full_rows(X, rows: Sequence[int]):
    """gamma_t of Definition 1 for the given token indices only."""
    X = _x(X)
    T, d = X.shape
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    gamma = np.empty(rows.size, dtype=np.float64)
    if _load().ada_oracle_full_rows(_dp(X), T, d, _ip(rows), rows.size, _dp(gamma)) != 0:
        raise MemoryError
    return gamma


@dataclass
class CascadeResult:
    rep: np.ndarray          # R^(l+1), ascending
    add: np.ndarray          # R_new, ascending
    rem: np.ndarray          # R^(l) \ R_valid, ascending
    gamma_rep: np.ndarray    # by position in the inherited list
    gamma_cross: np.ndarray  # by token index (0 for inherited reps)


def cascade_step(X, tau: float, rep_in, causal: bool = False,
                 force_valid: Optional[np.ndarray] = None,
                 only_rows: Optional[Sequence[int]] = None) -> CascadeResult:
    """Algorithm 1."""
    X = _x(X)
    T, d = X.shape
    rep_in = np.ascontiguousarray(rep_in, dtype=np.int32)
    r = rep_in.size
    if r and (np.any(np.diff(rep_in) <= 0) or rep_in[0] < 0 or rep_in[-1] >= T):
        raise ValueError("inherited set must be strictly ascending and inside [0, T)")
    gr = np.zeros(max(r, 1), dtype=np.float64)
    gc = np.zeros(T, dtype=np.float64)
    rep = np.empty(T, dtype=np.int32)
    add = np.empty(T, dtype=np.int32)
    rem = np.empty(max(r, 1), dtype=np.int32)
    n = (C.c_int64 * 3)()
    fv = None
    if force_valid is not None:
        fv_arr = np.ascontiguousarray(force_valid, dtype=np.uint8)
        assert fv_arr.size == r
        fv = fv_arr.ctypes.data_as(C.POINTER(C.c_uint8))
    rows_p, n_rows = None, 0
    if only_rows is not None:
        rows_arr = np.ascontiguousarray(only_rows, dtype=np.int32)
        rows_p, n_rows = _ip(rows_arr), rows_arr.size
    rc = _load().ada_oracle_cascade(_dp(X), T, d, float(tau), _ip(rep_in), r, int(bool(causal)),
                                    fv, rows_p, n_rows, _dp(gr), _dp(gc), _ip(rep), _ip(add),
                                    _ip(rem), n)
    if rc != 0:
        raise MemoryError
    return CascadeResult(rep[:n[0]].copy(), add[:n[1]].copy(), rem[:n[2]].copy(), gr[:r].copy(), gc)


def nearest(X, rep):
    """Section 2.3: nearest representative of every token.  Returns (nearest int32[T], gamma[T])."""
    X = _x(X)
    T, d = X.shape
    rep = np.ascontiguousarray(rep, dtype=np.int32)
    out = np.empty(T, dtype=np.int32)
    g = np.empty(T, dtype=np.float64)
    if _load().ada_oracle_nearest(_dp(X), T, d, _ip(rep), rep.size, _ip(out), _dp(g)) != 0:
        raise MemoryError
    return out, g


def attention_reps(Q, K, V, rep, nearest_idx=None, causal: bool = False) -> np.ndarray:
    """Eq. 2 on the representative rows of Q, K, V (each T x h x d_h), expanded to all tokens
    through `nearest_idx` when given (Section 2.3).  Returns out float64 [T, h, d_h]."""
    Q, K, V = (np.ascontiguousarray(a, dtype=np.float64) for a in (Q, K, V))
    T, h, d_h = Q.shape
    assert K.shape == Q.shape and V.shape == Q.shape
    rep = np.ascontiguousarray(rep, dtype=np.int32)
    if rep.size and (np.any(np.diff(rep) <= 0) or rep[0] < 0 or rep[-1] >= T):
        raise ValueError("representative set must be strictly ascending and inside [0, T)")
    out = np.empty((T, h, d_h), dtype=np.float64)
    near_p = None
    if nearest_idx is not None:
        near = np.ascontiguousarray(nearest_idx, dtype=np.int32)
        assert near.size == T
        near_p = _ip(near)
    _load().ada_oracle_attention_reps(_dp(Q), _dp(K), _dp(V), T, h, d_h, _ip(rep), rep.size, near_p,
                                      int(bool(causal)), _dp(out))
    return out


def op_count(cascade: bool, T: int, d: int, r: int = 0) -> int:
    return int(_load().ada_oracle_op_count(int(bool(cascade)), T, d, r))


def jaccard(a, b) -> float:
    a = np.ascontiguousarray(a, dtype=np.int32)
    b = np.ascontiguousarray(b, dtype=np.int32)
    return float(_load().ada_oracle_jaccard(_ip(a), a.size, _ip(b), b.size))


def tau_update(tau: float, rho: float, target: float, gain: float, tau_min: float,
               tau_max: float) -> float:
    """Section 8.1, reading: clipped proportional step of tau toward a target turnover."""
    return float(_load().ada_oracle_tau_update(float(tau), float(rho), float(target), float(gain),
                                               float(tau_min), float(tau_max)))


def turnover(n_add: int, n_rem: int, r: int) -> float:
    return float(_load().ada_oracle_turnover(n_add, n_rem, r))
