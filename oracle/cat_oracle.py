"""CAT oracle, Python face -- TEST INFRASTRUCTURE, not part of the product.

Thin ctypes wrapper over ``cat_oracle.c`` (plain C, fp64 arithmetic, written
from Section 3.1 and Algorithms 1-2 of the CAT paper).  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import this module.  It shares
no code with the CUDA library and never imports it.

Functions take and return numpy arrays (fp32 data, int32 labels).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cat_oracle.c")
_LIB = os.path.join(_HERE, "libcat_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile cat_oracle.c with gcc (-O2, no fast-math, OpenMP) if stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
           "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    f32p = ctypes.POINTER(ctypes.c_float)
    f64p = ctypes.POINTER(ctypes.c_double)
    i32p = ctypes.POINTER(ctypes.c_int32)
    i64p = ctypes.POINTER(ctypes.c_int64)
    i64, i32, f64 = ctypes.c_int64, ctypes.c_int32, ctypes.c_double
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
    lib.oracle_assign.argtypes = [f32p, i64, i32, i32, f32p, i32p, f64p, f64p]
    lib.oracle_assign.restype = None
    lib.oracle_update_centroids.argtypes = [f32p, i32p, i64, i32, i32, f32p, i64p]
    lib.oracle_update_centroids.restype = None
    lib.oracle_solve_gamma_beta.argtypes = [f32p, f32p, i32p, i64, i32, i32, f32p, f32p]
    lib.oracle_solve_gamma_beta.restype = None
    lib.oracle_fit.argtypes = [f32p, f32p, i64, i32, i32, i32, f32p, f64,
                               f32p, f32p, f32p, i32p, f64p, i64p, i64p]
    lib.oracle_fit.restype = ctypes.c_int
    lib.oracle_apply.argtypes = [f32p, i64, i32, i32, f32p, f32p, f32p, f64,
                                 f32p, i32p, f64p, f64p]
    lib.oracle_apply.restype = None
    lib.oracle_affine_with_labels.argtypes = [f32p, i32p, i64, i32, f32p, f32p, f64, f32p]
    lib.oracle_affine_with_labels.restype = None
    _lib = lib
    return lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def assign(Yq, C):
    """Nearest centroid per row (lowest index on ties).

    Returns (labels int32[N], best float64[N], second float64[N])."""
    Yq, C = _f32(Yq), _f32(C)
    N, D = Yq.shape
    K = C.shape[0]
    assert C.shape[1] == D
    labels = np.empty(N, np.int32)
    best = np.empty(N, np.float64)
    second = np.empty(N, np.float64)
    _load().oracle_assign(_p(Yq, ctypes.c_float), N, D, K, _p(C, ctypes.c_float),
                          _p(labels, ctypes.c_int32), _p(best, ctypes.c_double),
                          _p(second, ctypes.c_double))
    return labels, best, second


def near_tie_mask(best, second, rel=1e-6):
    """Rows whose best-vs-second gap is at most `rel` relative to second."""
    return (second - best) <= rel * second


def update_centroids(Yq, labels, C_prev):
    """One Lloyd update: cluster means (fp64 sums, fp32 result); an empty
    cluster keeps C_prev's row.  Returns (C float32[K,D], counts int64[K])."""
    Yq = _f32(Yq)
    C = _f32(C_prev).copy()
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, D = Yq.shape
    K = C.shape[0]
    assert labels.shape == (N,) and labels.min(initial=0) >= 0 and labels.max(initial=0) < K
    counts = np.empty(K, np.int64)
    _load().oracle_update_centroids(_p(Yq, ctypes.c_float), _p(labels, ctypes.c_int32),
                                    N, D, K, _p(C, ctypes.c_float), _p(counts, ctypes.c_int64))
    return C, counts


def solve_gamma_beta(Yq, Yfp, labels, K):
    """Closed-form per-cluster gamma/beta for the given labels."""
    Yq, Yfp = _f32(Yq), _f32(Yfp)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, D = Yq.shape
    assert Yfp.shape == (N, D) and labels.shape == (N,)
    assert labels.min(initial=0) >= 0 and labels.max(initial=0) < K
    gamma = np.empty((K, D), np.float32)
    beta = np.empty((K, D), np.float32)
    _load().oracle_solve_gamma_beta(_p(Yq, ctypes.c_float), _p(Yfp, ctypes.c_float),
                                    _p(labels, ctypes.c_int32), N, D, K,
                                    _p(gamma, ctypes.c_float), _p(beta, ctypes.c_float))
    return gamma, beta


@dataclass
class FitResult:
    centroids: np.ndarray   # float32 [K, D]
    gamma: np.ndarray       # float32 [K, D]
    beta: np.ndarray        # float32 [K, D]
    labels: np.ndarray      # int32 [N], final assignment
    J: np.ndarray           # float64 [iters+1], objective of each assignment
    near: np.ndarray        # int64 [iters+1], near-tie rows of each assignment
    counts: np.ndarray      # int64 [K], final cluster sizes


def fit(Yq, Yfp, K, iters, init=None, near_rel=1e-6) -> FitResult:
    """CAT fitting (Algorithm 1 without PCA): `iters` Lloyd rounds from
    `init` (default: first K rows), a final assignment, then gamma/beta."""
    Yq, Yfp = _f32(Yq), _f32(Yfp)
    N, D = Yq.shape
    assert Yfp.shape == (N, D)
    C = np.empty((K, D), np.float32)
    gamma = np.empty((K, D), np.float32)
    beta = np.empty((K, D), np.float32)
    labels = np.empty(N, np.int32)
    J = np.empty(iters + 1, np.float64)
    near = np.empty(iters + 1, np.int64)
    counts = np.empty(K, np.int64)
    if init is not None:
        init = _f32(init)
        assert init.shape == (K, D)
        initp = _p(init, ctypes.c_float)
    else:
        initp = None
    rc = _load().oracle_fit(_p(Yq, ctypes.c_float), _p(Yfp, ctypes.c_float), N, D, K, iters,
                            initp, float(near_rel), _p(C, ctypes.c_float),
                            _p(gamma, ctypes.c_float), _p(beta, ctypes.c_float),
                            _p(labels, ctypes.c_int32), _p(J, ctypes.c_double),
                            _p(near, ctypes.c_int64), _p(counts, ctypes.c_int64))
    if rc != 0:
        raise ValueError("oracle_fit: bad arguments (need N >= K >= 1, D >= 1, iters >= 0)")
    return FitResult(C, gamma, beta, labels, J, near, counts)


def apply(Yq, C, gamma, beta, alpha=1.0):
    """CAT inference (Algorithm 2 without PCA).

    Returns (out float32[N,D], labels int32[N], best float64[N], second float64[N])."""
    Yq, C, gamma, beta = _f32(Yq), _f32(C), _f32(gamma), _f32(beta)
    N, D = Yq.shape
    K = C.shape[0]
    assert C.shape == (K, D) and gamma.shape == (K, D) and beta.shape == (K, D)
    out = np.empty((N, D), np.float32)
    labels = np.empty(N, np.int32)
    best = np.empty(N, np.float64)
    second = np.empty(N, np.float64)
    _load().oracle_apply(_p(Yq, ctypes.c_float), N, D, K, _p(C, ctypes.c_float),
                         _p(gamma, ctypes.c_float), _p(beta, ctypes.c_float), float(alpha),
                         _p(out, ctypes.c_float), _p(labels, ctypes.c_int32),
                         _p(best, ctypes.c_double), _p(second, ctypes.c_double))
    return out, labels, best, second


def affine_with_labels(Yq, labels, gamma, beta, alpha=1.0):
    """out_i = blend(q_i, gamma[labels_i]*q_i + beta[labels_i]) for given labels."""
    Yq, gamma, beta = _f32(Yq), _f32(gamma), _f32(beta)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, D = Yq.shape
    out = np.empty((N, D), np.float32)
    _load().oracle_affine_with_labels(_p(Yq, ctypes.c_float), _p(labels, ctypes.c_int32), N, D,
                                      _p(gamma, ctypes.c_float), _p(beta, ctypes.c_float),
                                      float(alpha), _p(out, ctypes.c_float))
    return out


def to_bf16(x):
    """Round fp32 values to bfloat16 (8 significant bits, round to nearest, ties to even) and return
    them as fp32.  Written out on the bit pattern: add half of the dropped 16 bits' range (plus the
    parity of the kept part for ties), then clear the low 16 bits.  NaN and infinities pass through."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    keep_odd = (u >> 16) & 1
    r = ((u + 0x7FFF + keep_odd) >> 16) << 16
    out = (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32).reshape(a.shape)
    special = ~np.isfinite(a)
    return np.where(special, a, out)


def apply_bf16(Yq, C, gamma, beta):
    """CAT inference with a bfloat16 result: the fp32 corrected outputs of `apply` (one rounding of
    gamma*q + beta), rounded once more to bfloat16.  Returns (out as fp32 holding bf16 values, labels,
    best, second)."""
    out, labels, best, second = apply(Yq, C, gamma, beta)
    return to_bf16(out), labels, best, second
