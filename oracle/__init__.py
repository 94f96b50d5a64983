"""ctypes front end of the CPU fp64 oracle (``more_oracle.c``).

TEST INFRASTRUCTURE: only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It neither imports nor is imported by the CUDA library's package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "more_oracle.c")
_LIB = os.path.join(_HERE, "libmore_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``more_oracle.c`` with gcc (+OpenMP) into ``libmore_oracle.so`` next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        i64p = ctypes.POINTER(ctypes.c_int64)
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.more_oracle_route.argtypes = [u16p, u16p, u16p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_int, i32p, f64p, f64p, f64p, f64p, i64p, ctypes.c_int]
        lib.more_oracle_route.restype = ctypes.c_int
        lib.more_oracle_logits.argtypes = [u16p, u16p, u16p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, f64p]
        lib.more_oracle_logits.restype = ctypes.c_int
        lib.more_oracle_logits_at.argtypes = [u16p, u16p, u16p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, i32p, f64p]
        lib.more_oracle_logits_at.restype = ctypes.c_int
        lib.more_oracle_threads.restype = ctypes.c_int
        lib.more_oracle_psum.argtypes = [u16p, u16p, u16p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, f64p, f64p]
        lib.more_oracle_psum.restype = ctypes.c_int
        lib.more_oracle_dispatch.argtypes = [i32p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, i64p, i64p]
        lib.more_oracle_dispatch.restype = ctypes.c_int
        lib.more_oracle_merge.argtypes = [i32p, f64p, f64p, ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, i32p, f64p, f64p, f64p, i64p]
        lib.more_oracle_merge.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _check(X, R1, R2):
    X = np.ascontiguousarray(X, dtype=np.uint16)
    R1 = np.ascontiguousarray(R1, dtype=np.uint16)
    R2 = np.ascontiguousarray(R2, dtype=np.uint16)
    T, h = X.shape
    h2, r = R1.shape
    r2, M = R2.shape
    if h2 != h or r2 != r:
        raise ValueError("shape mismatch between X, R1, R2")
    return X, R1, R2, T, h, r, M


@dataclass
class OracleResult:
    idx: np.ndarray     # [T][k] int32, descending logit, ties by ascending id
    gate: np.ndarray    # [T][k] float64
    topval: np.ndarray  # [T][k] float64, the selected logits
    lse: np.ndarray     # [T] float64, log-sum-exp over all M logits
    gap: np.ndarray     # [T] float64, k-th minus (k+1)-th largest logit (+inf when k == M)
    counts: np.ndarray  # [M] int64


def threads() -> int:
    return int(_load().more_oracle_threads())


def route(X, R1, R2, k: int, gate_mode: int, nthreads: int = 0) -> OracleResult:
    """Run the oracle on bf16 bit patterns ``X [T][h]``, ``R1 [h][r]``, ``R2 [r][M]``."""
    lib = _load()
    X, R1, R2, T, h, r, M = _check(X, R1, R2)
    idx = np.zeros((T, k), dtype=np.int32)
    gate = np.zeros((T, k), dtype=np.float64)
    topval = np.zeros((T, k), dtype=np.float64)
    lse = np.zeros((T,), dtype=np.float64)
    gap = np.zeros((T,), dtype=np.float64)
    counts = np.zeros((M,), dtype=np.int64)
    rc = lib.more_oracle_route(_p(X, ctypes.c_uint16), _p(R1, ctypes.c_uint16), _p(R2, ctypes.c_uint16),
                               T, h, r, M, k, gate_mode, _p(idx, ctypes.c_int32), _p(gate, ctypes.c_double),
                               _p(topval, ctypes.c_double), _p(lse, ctypes.c_double), _p(gap, ctypes.c_double),
                               _p(counts, ctypes.c_int64), nthreads)
    if rc != 0:
        raise ValueError("more_oracle_route rejected its arguments")
    return OracleResult(idx, gate, topval, lse, gap, counts)


def logits(X, R1, R2) -> np.ndarray:
    """The full ``[T][M]`` fp64 logit matrix (small inputs only)."""
    lib = _load()
    X, R1, R2, T, h, r, M = _check(X, R1, R2)
    out = np.zeros((T, M), dtype=np.float64)
    rc = lib.more_oracle_logits(_p(X, ctypes.c_uint16), _p(R1, ctypes.c_uint16), _p(R2, ctypes.c_uint16),
                                T, h, r, M, _p(out, ctypes.c_double))
    if rc != 0:
        raise MemoryError("more_oracle_logits failed")
    return out


def logits_at(X, R1, R2, ids) -> np.ndarray:
    """fp64 logits of the experts ``ids [T][q]`` of each token (NaN for ids outside ``[0, M)``)."""
    lib = _load()
    X, R1, R2, T, h, r, M = _check(X, R1, R2)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    q = ids.shape[1]
    out = np.zeros((T, q), dtype=np.float64)
    rc = lib.more_oracle_logits_at(_p(X, ctypes.c_uint16), _p(R1, ctypes.c_uint16), _p(R2, ctypes.c_uint16),
                                   T, h, r, M, q, _p(ids, ctypes.c_int32), _p(out, ctypes.c_double))
    if rc != 0:
        raise MemoryError("more_oracle_logits_at failed")
    return out


def dispatch(idx, M: int):
    """Sort + Count of the selected ids ``idx [T][k]``: ``(offsets [M+1], sorted_pairs [number of valid pairs])`` with
    pairs named by their flat position ``n*k + j``, grouped by expert, ascending within an expert."""
    lib = _load()
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, k = idx.shape
    offsets = np.zeros((M + 1,), dtype=np.int64)
    pairs = np.zeros((T * k,), dtype=np.int64)
    rc = lib.more_oracle_dispatch(_p(idx, ctypes.c_int32), T, k, M, _p(offsets, ctypes.c_int64), _p(pairs, ctypes.c_int64))
    if rc != 0:
        raise ValueError("more_oracle_dispatch rejected its arguments")
    return offsets, pairs[:offsets[M]]


def psum(X, R1, R2):
    """Column sums of the softmax over all experts, ``psum[i] = sum_n P[n, i]`` (Algorithm 2's statistic), and the
    per-token log-sum-exp: ``(psum [M], lse [T])``."""
    lib = _load()
    X, R1, R2, T, h, r, M = _check(X, R1, R2)
    out = np.zeros((M,), dtype=np.float64)
    lse = np.zeros((T,), dtype=np.float64)
    rc = lib.more_oracle_psum(_p(X, ctypes.c_uint16), _p(R1, ctypes.c_uint16), _p(R2, ctypes.c_uint16),
                              T, h, r, M, _p(out, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError("more_oracle_psum rejected its arguments")
    return out, lse


def merge(idx, val, lse, M: int, gate_mode: int):
    """Global top-k from per-shard top-k lists: ``idx [S][T][k]`` (global expert ids, < 0 = unused), ``val [S][T][k]``,
    ``lse [S][T]`` or None.  Returns ``(idx [T][k], gate [T][k], val [T][k], lse [T] or None, counts [M])``."""
    lib = _load()
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    val = np.ascontiguousarray(val, dtype=np.float64)
    S, T, k = idx.shape
    if val.shape != idx.shape:
        raise ValueError("idx and val must have the same shape")
    lse_c = None if lse is None else np.ascontiguousarray(lse, dtype=np.float64)
    if lse_c is not None and lse_c.shape != (S, T):
        raise ValueError("lse must be [S][T]")
    out_idx = np.zeros((T, k), dtype=np.int32)
    out_gate = np.zeros((T, k), dtype=np.float64)
    out_val = np.zeros((T, k), dtype=np.float64)
    out_lse = np.zeros((T,), dtype=np.float64) if lse_c is not None else None
    counts = np.zeros((M,), dtype=np.int64)
    rc = lib.more_oracle_merge(_p(idx, ctypes.c_int32), _p(val, ctypes.c_double),
                               None if lse_c is None else _p(lse_c, ctypes.c_double), S, T, k, M, gate_mode,
                               _p(out_idx, ctypes.c_int32), _p(out_gate, ctypes.c_double), _p(out_val, ctypes.c_double),
                               None if out_lse is None else _p(out_lse, ctypes.c_double), _p(counts, ctypes.c_int64))
    if rc != 0:
        raise ValueError("more_oracle_merge rejected its arguments")
    return out_idx, out_gate, out_val, out_lse, counts
