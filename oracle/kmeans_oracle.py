"""ctypes front end of the fp64 CPU oracle (``kmeans_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the benchmark's
CPU-baseline / reference arm.  The CUDA library and its Python binding never import this module,
and this module imports nothing from them.

All point / centroid inputs are raw bf16 bit patterns held in ``numpy.uint16`` arrays; the oracle
widens them exactly to fp64.  See the C file's header for the passage of the paper each function
follows (Section 5, "Flash-KMeans clean-start workload") and for the list of pins.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kmeans_oracle.c")
_SO = os.path.join(_HERE, "libkmeans_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no BLAS, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, vp = ctypes.c_longlong, ctypes.c_int, ctypes.c_void_p
        lib.oracle_bf16_to_f64.argtypes = [vp, i64, vp]
        lib.oracle_bf16_to_f64.restype = None
        lib.oracle_f64_to_bf16.argtypes = [vp, i64, vp]
        lib.oracle_f64_to_bf16.restype = None
        lib.oracle_assign_f64c.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp]
        lib.oracle_assign.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp]
        lib.oracle_pair_sqdist.argtypes = [vp, vp, i64, i32, i32, vp, vp]
        lib.oracle_update.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp]
        lib.oracle_lloyd.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_knn.argtypes = [vp, vp, i64, i64, i32, i32, vp, vp]
        lib.oracle_num_threads.restype = i32
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bits(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or a.ndim != 2:
        raise TypeError(f"{name} must be a 2-D uint16 array of bf16 bit patterns")
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().oracle_bf16_to_f64(_p(bits), bits.size, _p(out))
    return out


def f64_to_bf16(vals: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16, round-to-nearest-even at both steps."""
    vals = np.ascontiguousarray(vals, dtype=np.float64)
    out = np.empty(vals.shape, dtype=np.uint16)
    _load().oracle_f64_to_bf16(_p(vals), vals.size, _p(out))
    return out


def assign(X: np.ndarray, C: np.ndarray):
    """Nearest centroid of every point.

    X [N,D] bf16 bits; C [K,D] bf16 bits (uint16) or fp64 values (float64).
    Returns (idx int32 [N], dist f64 [N], second f64 [N]).
    """
    X = _bits(X, "X")
    N, D = X.shape
    C = np.ascontiguousarray(C)
    if C.ndim != 2 or C.shape[1] != D:
        raise ValueError("C must be [K,D]")
    K = C.shape[0]
    idx = np.empty(N, dtype=np.int32)
    dist = np.empty(N, dtype=np.float64)
    second = np.empty(N, dtype=np.float64)
    lib = _load()
    if C.dtype == np.uint16:
        rc = lib.oracle_assign(_p(X), _p(C), N, D, K, _p(idx), _p(dist), _p(second))
    elif C.dtype == np.float64:
        rc = lib.oracle_assign_f64c(_p(X), _p(C), N, D, K, _p(idx), _p(dist), _p(second))
    else:
        raise TypeError("C must be uint16 (bf16 bits) or float64")
    if rc != 0:
        raise RuntimeError(f"oracle_assign failed: {rc}")
    return idx, dist, second


def pair_sqdist(X: np.ndarray, C: np.ndarray, g: np.ndarray) -> np.ndarray:
    """d(x_i, c_{g[i]}) in fp64 for a given pairing (C as bf16 bits or fp64)."""
    X = _bits(X, "X")
    N, D = X.shape
    Cd = bf16_to_f64(C) if np.asarray(C).dtype == np.uint16 else np.ascontiguousarray(C, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.int32)
    out = np.empty(N, dtype=np.float64)
    rc = _load().oracle_pair_sqdist(_p(X), _p(Cd), N, D, Cd.shape[0], _p(g), _p(out))
    if rc != 0:
        raise RuntimeError(f"oracle_pair_sqdist failed: {rc}")
    return out


def update(X: np.ndarray, idx: np.ndarray, K: int, C_prev: np.ndarray | None = None,
           return_sums: bool = False):
    """Per-cluster sums / counts / means; empty clusters keep C_prev (zeros if None).

    C_prev may be bf16 bits or fp64.  Returns (C_new f64 [K,D], counts int64 [K][, sums f64]).
    """
    X = _bits(X, "X")
    N, D = X.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    if idx.shape != (N,):
        raise ValueError("idx must be [N]")
    if C_prev is not None:
        C_prev = bf16_to_f64(C_prev) if np.asarray(C_prev).dtype == np.uint16 else \
            np.ascontiguousarray(C_prev, dtype=np.float64)
        if C_prev.shape != (K, D):
            raise ValueError("C_prev must be [K,D]")
    C_new = np.empty((K, D), dtype=np.float64)
    counts = np.empty(K, dtype=np.int64)
    sums = np.empty((K, D), dtype=np.float64) if return_sums else None
    rc = _load().oracle_update(_p(X), _p(idx), N, D, K, _p(C_prev), _p(C_new), _p(counts), _p(sums))
    if rc != 0:
        raise RuntimeError(f"oracle_update failed: {rc}")
    return (C_new, counts, sums) if return_sums else (C_new, counts)


def knn(Q: np.ndarray, X: np.ndarray, k: int):
    """The k database rows nearest to every query: Q [N,D], X [M,D] bf16 bits -> (idx int32 [N,k], dist f64 [N,k]),
    ascending by (distance, row number); idx -1 / dist +inf where M < k."""
    Q, X = _bits(Q, "Q"), _bits(X, "X")
    if Q.shape[1] != X.shape[1] or k < 1:
        raise ValueError("Q and X need the same D, k >= 1")
    N, D = Q.shape
    idx = np.empty((N, k), dtype=np.int32)
    dist = np.empty((N, k), dtype=np.float64)
    rc = _load().oracle_knn(_p(Q), _p(X), N, X.shape[0], D, k, _p(idx), _p(dist))
    if rc != 0:
        raise RuntimeError(f"oracle_knn failed: {rc}")
    return idx, dist


def kmeanspp_step(mind: np.ndarray, u_k: float):
    """One draw of the seeding below: the first row whose running sum of `mind` exceeds u_k * sum(mind)
    (a uniform row if every entry is zero).  Returns (row, running sums)."""
    N = mind.shape[0]
    cum = np.cumsum(mind)
    total = cum[-1]
    if not total > 0.0:
        return min(int(u_k * N), N - 1), cum
    return min(int(np.searchsorted(cum, u_k * total, side="right")), N - 1), cum


def kmeanspp(X: np.ndarray, K: int, u: np.ndarray) -> np.ndarray:
    """k-means++ seeding (D^2 sampling) with the random numbers passed in: u [K] uniforms in [0, 1).

    Row 0 of the result is floor(u[0] * N); for k >= 1, with mind[i] the squared distance (direct differences,
    fp64) from x_i to the nearest of the k rows chosen so far, row k is the first i whose running sum
    mind[0] + ... + mind[i] exceeds u[k] * sum(mind).  The paper's K-means workload starts from sampled rows and
    names no seeding; this is the textbook procedure, offered as an initialiser.  Returns the K row numbers.
    """
    X = _bits(X, "X")
    N = X.shape[0]
    u = np.asarray(u, dtype=np.float64)
    if K < 1 or u.shape != (K,) or N < 1:
        raise ValueError("need K >= 1 uniforms and N >= 1 rows")
    Xf = bf16_to_f64(X)
    rows = [min(int(u[0] * N), N - 1)]
    mind = np.full(N, np.inf)
    for k in range(1, K):
        diff = Xf - Xf[rows[-1]]
        mind = np.minimum(mind, (diff * diff).sum(1))
        r, _ = kmeanspp_step(mind, float(u[k]))
        rows.append(r)
    return np.asarray(rows, dtype=np.int64)


@dataclass
class LloydResult:
    C: np.ndarray          # [K,D] f64, means of the last update (unrounded)
    C_bits: np.ndarray     # [K,D] bf16 bits of C
    idx: np.ndarray        # [N] int32, last assign
    dist: np.ndarray       # [N] f64, last assign
    second: np.ndarray     # [N] f64, last assign
    counts: np.ndarray     # [K] int64, last update
    inertia: np.ndarray    # [iters] f64, inertia[t] = sum_i d(x_i, C_t[idx_t(i)])


def lloyd(X: np.ndarray, C0: np.ndarray, iters: int, round_centroids: bool = True) -> LloydResult:
    X = _bits(X, "X")
    C0 = _bits(C0, "C0")
    N, D = X.shape
    K = C0.shape[0]
    C = np.empty((K, D), dtype=np.float64)
    Cb = np.empty((K, D), dtype=np.uint16)
    idx = np.zeros(N, dtype=np.int32)
    dist = np.zeros(N, dtype=np.float64)
    second = np.zeros(N, dtype=np.float64)
    counts = np.zeros(K, dtype=np.int64)
    inertia = np.zeros(iters, dtype=np.float64)
    rc = _load().oracle_lloyd(_p(X), _p(C0), N, D, K, iters, int(bool(round_centroids)), _p(C), _p(Cb),
                              _p(idx), _p(dist), _p(second), _p(counts), _p(inertia))
    if rc != 0:
        raise RuntimeError(f"oracle_lloyd failed: {rc}")
    return LloydResult(C, Cb, idx, dist, second, counts, inertia)
