"""Python face of libcat.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/cat.h)
and takes torch CUDA tensors (or, for the *_host calls, CPU tensors); torch
supplies device memory and the current stream, nothing else.  All arithmetic
happens in the CUDA library; if it cannot be loaded these functions raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

_lib = None

CAT_OK = 0
STATUS_NAMES = {0: "CAT_OK", 1: "CAT_ERR_NULL", 2: "CAT_ERR_SHAPE", 3: "CAT_ERR_ALIGN",
                4: "CAT_ERR_WORKSPACE", 5: "CAT_ERR_CUDA", 6: "CAT_ERR_DEVICE_TIMEOUT",
                7: "CAT_ERR_UNSUPPORTED"}
MAX_K = 512
MAX_D = 16384
DIAG_MAX_ROUNDS = 64                       # CAT_DIAG_MAX_ROUNDS
_DIAG_WORDS = 5 + 3 * DIAG_MAX_ROUNDS      # cat_fit_diag_t in 8-byte words
ASSIGN_FP16_OPERANDS = 1                   # CAT_ASSIGN_FP16_OPERANDS


class _FastScores(ctypes.Structure):       # cat_fast_scores_t
    _fields_ = [("best", ctypes.c_void_p), ("second", ctypes.c_void_p), ("bound", ctypes.c_void_p),
                ("label", ctypes.c_void_p)]

EXPORTS = [
    "cat_fit_workspace_bytes", "cat_fit", "cat_fit_from", "cat_apply_workspace_bytes",
    "cat_apply", "cat_apply_blend", "cat_apply_bf16", "cat_assign", "cat_assign_scores", "cat_assign_noalloc", "cat_cluster_sums",
    "cat_fit_shard_begin", "cat_fit_shard_round", "cat_fit_shard_update",
    "cat_pca_workspace_bytes", "cat_pca_fit", "cat_pca_project", "cat_affine_with_labels",
    "cat_fit_pca_workspace_bytes", "cat_fit_pca", "cat_apply_pca_workspace_bytes", "cat_apply_pca",
    "cat_centroids_from_sums",
    "cat_centred_moments", "cat_solve_gamma_beta", "cat_apply_host_workspace_bytes",
    "cat_apply_host", "cat_fit_host_workspace_bytes", "cat_fit_host", "cat_workspace_report",
    "cat_selftest_wait_timeout",
    "cat_set_tensor_core_min_k", "cat_get_tensor_core_min_k", "cat_tensor_path_available",
    "cat_set_small_problem_kernels", "cat_get_small_problem_kernels",
    "cat_set_apply_column_split", "cat_get_apply_column_split", "cat_status_string",
    "cat_last_cuda_error", "cat_version", "cat_kernel_launches",
]


class CatError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().cat_status_string(status).decode()
        extra = ""
        if status == 5:
            extra = f" (cudaError {lib().cat_last_cuda_error()})"
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}: {msg}{extra}")


def library_path() -> str:
    return _build.LIB


def lib():
    """Load libcat.so (building it first if the sources are newer).  Raises if
    it is missing and cannot be built: there is no other implementation."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if os.environ.get("CAT_NO_BUILD") != "1":
        try:
            path = _build.build()
        except Exception as e:  # pragma: no cover
            if not os.path.exists(path):
                raise RuntimeError(f"libcat.so is missing and could not be built: {e}") from e
    if not os.path.exists(path):
        raise RuntimeError("libcat.so is missing; run python -m paper_2509_26277_b200.build")
    L = ctypes.CDLL(path)
    vp, i64, i32, sz, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t, ctypes.c_float
    L.cat_fit_workspace_bytes.argtypes = [i64, i32, i32]
    L.cat_fit_workspace_bytes.restype = sz
    L.cat_apply_workspace_bytes.argtypes = [i64, i32, i32]
    L.cat_apply_workspace_bytes.restype = sz
    L.cat_apply_host_workspace_bytes.argtypes = [i64, i32, i32]
    L.cat_apply_host_workspace_bytes.restype = sz
    L.cat_fit_host_workspace_bytes.argtypes = [i64, i32, i32]
    L.cat_fit_host_workspace_bytes.restype = sz
    L.cat_fit.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    L.cat_fit_from.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_apply.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_apply_blend.argtypes = [vp, i64, i32, i32, vp, vp, vp, f32, vp, vp, vp, sz, vp]
    L.cat_assign.argtypes = [vp, i64, i32, i32, vp, vp, vp, sz, vp]
    L.cat_apply_bf16.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_apply_bf16.restype = ctypes.c_int
    L.cat_assign_scores.argtypes = [vp, i64, i32, i32, vp, vp, ctypes.POINTER(_FastScores), i32, vp, sz, vp]
    L.cat_assign_scores.restype = ctypes.c_int
    L.cat_assign_noalloc.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    L.cat_assign_noalloc.restype = ctypes.c_int
    L.cat_fit_shard_begin.argtypes = [vp, i64, i32, i32, vp, vp, sz, vp]
    L.cat_fit_shard_round.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_fit_shard_update.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    for name in ("cat_fit_shard_begin", "cat_fit_shard_round", "cat_fit_shard_update"):
        getattr(L, name).restype = ctypes.c_int
    L.cat_pca_workspace_bytes.argtypes = [i64, i32, i32]
    L.cat_pca_workspace_bytes.restype = sz
    L.cat_fit_pca_workspace_bytes.argtypes = [i64, i32, i32, i32]
    L.cat_fit_pca_workspace_bytes.restype = sz
    L.cat_apply_pca_workspace_bytes.argtypes = [i64, i32, i32, i32]
    L.cat_apply_pca_workspace_bytes.restype = sz
    L.cat_pca_fit.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, sz, vp]
    L.cat_pca_project.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp]
    L.cat_affine_with_labels.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp]
    L.cat_fit_pca.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_apply_pca.argtypes = [vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    for name in ("cat_pca_fit", "cat_pca_project", "cat_affine_with_labels", "cat_fit_pca", "cat_apply_pca"):
        getattr(L, name).restype = ctypes.c_int
    L.cat_cluster_sums.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, sz, vp]
    L.cat_centroids_from_sums.argtypes = [vp, vp, i32, i32, vp, vp]
    L.cat_centred_moments.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    L.cat_solve_gamma_beta.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    L.cat_apply_host.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    L.cat_fit_host.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    for name in ("cat_fit", "cat_fit_from", "cat_apply", "cat_apply_blend", "cat_assign",
                 "cat_cluster_sums", "cat_centroids_from_sums", "cat_centred_moments",
                 "cat_solve_gamma_beta", "cat_apply_host", "cat_fit_host"):
        getattr(L, name).restype = ctypes.c_int
    L.cat_selftest_wait_timeout.argtypes = [vp, sz, i32, vp]
    L.cat_selftest_wait_timeout.restype = ctypes.c_int
    L.cat_workspace_report.argtypes = [vp, vp, vp, vp, vp]
    L.cat_workspace_report.restype = ctypes.c_int
    L.cat_set_tensor_core_min_k.argtypes = [i32]
    L.cat_set_tensor_core_min_k.restype = None
    L.cat_get_tensor_core_min_k.restype = i32
    L.cat_set_small_problem_kernels.argtypes = [i32]
    L.cat_set_small_problem_kernels.restype = None
    L.cat_get_small_problem_kernels.restype = i32
    L.cat_tensor_path_available.restype = i32
    L.cat_set_apply_column_split.argtypes = [i32]
    L.cat_set_apply_column_split.restype = None
    L.cat_get_apply_column_split.restype = i32
    L.cat_status_string.argtypes = [ctypes.c_int]
    L.cat_status_string.restype = ctypes.c_char_p
    L.cat_last_cuda_error.restype = ctypes.c_int
    L.cat_version.restype = ctypes.c_char_p
    L.cat_kernel_launches.restype = ctypes.c_int64
    _lib = L
    return L


# ---------------------------------------------------------------- marshalling helpers

def _dev(t: Optional[torch.Tensor], dtype, shape=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _cpu(t: Optional[torch.Tensor], dtype, shape=None, name="tensor"):
    if t is None:
        return None
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CPU tensor of {dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


_ws_cache = {}


def workspace(kind: str, N: int, D: int, K: int, device) -> torch.Tensor:
    """Caller-side device scratch for one (entry-point family, N, D, K), cached."""
    device = torch.device(device)
    key = (kind, N, D, K, device.index if device.index is not None else torch.cuda.current_device())
    ws = _ws_cache.get(key)
    if ws is None:
        fn = {"fit": lib().cat_fit_workspace_bytes, "apply": lib().cat_apply_workspace_bytes,
              "apply_host": lib().cat_apply_host_workspace_bytes,
              "fit_host": lib().cat_fit_host_workspace_bytes}[kind]
        n = int(fn(N, D, K))
        if n == 0:
            raise CatError(7 if (K > MAX_K or D > MAX_D or N >= 2 ** 31) else 2, f"{kind} workspace query")
        ws = torch.empty(n, dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


def clear_workspaces():
    _ws_cache.clear()


def _check(status: int, where: str):
    if status != CAT_OK:
        raise CatError(status, where)


# ---------------------------------------------------------------- entry points

def cat_fit(Yq, Yfp, K: int, iters: int, init_centroids=None, want_labels=True, want_diag=False,
            ws=None):
    """cat_fit / cat_fit_from.  Returns (centroids, gamma, beta, labels or None[, diag dict])."""
    N, D = Yq.shape
    dev = Yq.device
    C = torch.empty((K, D), dtype=torch.float32, device=dev)
    G = torch.empty((K, D), dtype=torch.float32, device=dev)
    B = torch.empty((K, D), dtype=torch.float32, device=dev)
    labels = torch.empty((N,), dtype=torch.int32, device=dev) if want_labels else None
    diag = torch.zeros((_DIAG_WORDS,), dtype=torch.int64, device=dev) if want_diag else None
    ws = workspace("fit", N, D, K, dev) if ws is None else ws
    st = lib().cat_fit_from(_dev(Yq, torch.float32, None, "Yq"), _dev(Yfp, torch.float32, (N, D), "Yfp"),
                            N, D, K, iters, _dev(init_centroids, torch.float32, (K, D), "init_centroids"),
                            _dev(C, torch.float32), _dev(G, torch.float32), _dev(B, torch.float32),
                            _dev(labels, torch.int32), _dev(diag, torch.int64),
                            ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_fit")
    if want_diag:
        d = diag.cpu()
        n, R = int(d[4]), DIAG_MAX_ROUNDS
        return C, G, B, labels, dict(refined_rows_total=int(d[0]), refined_rows_final=int(d[1]),
                                     empty_clusters_final=int(d[2]), device_status=int(d[3]),
                                     assignments_recorded=n,
                                     undecided_rows=d[5:5 + n].tolist(),
                                     near_tie_rows=d[5 + R:5 + R + n].tolist(),
                                     objective=d[5 + 2 * R:5 + 2 * R + n].view(torch.float64).tolist())
    return C, G, B, labels


def cat_fit_into(Yq, Yfp, K: int, iters: int, C, G, B, labels, ws):
    """cat_fit with caller-provided outputs and workspace (no allocation: for timing loops)."""
    N, D = Yq.shape
    st = lib().cat_fit(_dev(Yq, torch.float32), _dev(Yfp, torch.float32, (N, D)), N, D, K, iters,
                       _dev(C, torch.float32, (K, D)), _dev(G, torch.float32, (K, D)),
                       _dev(B, torch.float32, (K, D)), _dev(labels, torch.int32),
                       ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_fit")


def cat_apply(Yq, centroids, gamma, beta, out=None, want_labels=False, alpha: float = 1.0, ws=None):
    """cat_apply (alpha == 1) or cat_apply_blend.  Returns out or (out, labels)."""
    N, D = Yq.shape
    K = centroids.shape[0]
    dev = Yq.device
    if out is None:
        out = torch.empty((N, D), dtype=torch.float32, device=dev)
    labels = torch.empty((N,), dtype=torch.int32, device=dev) if want_labels else None
    ws = workspace("apply", N, D, K, dev) if ws is None else ws
    args = (_dev(Yq, torch.float32, None, "Yq"), N, D, K, _dev(centroids, torch.float32, (K, D), "centroids"),
            _dev(gamma, torch.float32, (K, D), "gamma"), _dev(beta, torch.float32, (K, D), "beta"))
    tail = (_dev(out, torch.float32, (N, D), "out"), _dev(labels, torch.int32),
            ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    if alpha == 1.0:
        st = lib().cat_apply(*args, *tail)
    else:
        st = lib().cat_apply_blend(*args, ctypes.c_float(alpha), *tail)
    _check(st, "cat_apply")
    return (out, labels) if want_labels else out


def cat_apply_bf16(Yq, centroids, gamma, beta, out=None, want_labels=False, ws=None):
    """cat_apply_bf16: the corrected rows as a bf16 tensor."""
    N, D = Yq.shape
    K = centroids.shape[0]
    dev = Yq.device
    if out is None:
        out = torch.empty((N, D), dtype=torch.bfloat16, device=dev)
    labels = torch.empty((N,), dtype=torch.int32, device=dev) if want_labels else None
    ws = workspace("apply", N, D, K, dev) if ws is None else ws
    st = lib().cat_apply_bf16(_dev(Yq, torch.float32, None, "Yq"), N, D, K, _dev(centroids, torch.float32, (K, D)),
                              _dev(gamma, torch.float32, (K, D)), _dev(beta, torch.float32, (K, D)),
                              _dev(out, torch.bfloat16, (N, D), "out"), _dev(labels, torch.int32),
                              ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_apply_bf16")
    return (out, labels) if want_labels else out


def cat_apply_blend(Yq, centroids, gamma, beta, alpha: float, out=None, want_labels=False, ws=None):
    N, D = Yq.shape
    K = centroids.shape[0]
    dev = Yq.device
    if out is None:
        out = torch.empty((N, D), dtype=torch.float32, device=dev)
    labels = torch.empty((N,), dtype=torch.int32, device=dev) if want_labels else None
    ws = workspace("apply", N, D, K, dev) if ws is None else ws
    st = lib().cat_apply_blend(_dev(Yq, torch.float32, None, "Yq"), N, D, K,
                               _dev(centroids, torch.float32, (K, D)), _dev(gamma, torch.float32, (K, D)),
                               _dev(beta, torch.float32, (K, D)), ctypes.c_float(alpha),
                               _dev(out, torch.float32, (N, D)), _dev(labels, torch.int32),
                               ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_apply_blend")
    return (out, labels) if want_labels else out


def cat_assign(Yq, centroids, ws=None):
    N, D = Yq.shape
    K = centroids.shape[0]
    labels = torch.empty((N,), dtype=torch.int32, device=Yq.device)
    ws = workspace("apply", N, D, K, Yq.device) if ws is None else ws
    st = lib().cat_assign(_dev(Yq, torch.float32, None, "Yq"), N, D, K,
                          _dev(centroids, torch.float32, (K, D), "centroids"), _dev(labels, torch.int32),
                          ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_assign")
    return labels


def cat_assign_scores(Yq, centroids, fp16_operands: bool = False, ws=None):
    """cat_assign_scores: returns (labels, dict(best, second, bound, label)) -- the final labels and what
    the fast pass saw for every row (see cat.h)."""
    N, D = Yq.shape
    K = centroids.shape[0]
    dev = Yq.device
    labels = torch.empty((N,), dtype=torch.int32, device=dev)
    rec = dict(best=torch.empty((N,), dtype=torch.float32, device=dev),
               second=torch.empty((N,), dtype=torch.float32, device=dev),
               bound=torch.empty((N,), dtype=torch.float32, device=dev),
               label=torch.empty((N,), dtype=torch.int32, device=dev))
    fs = _FastScores(rec["best"].data_ptr(), rec["second"].data_ptr(), rec["bound"].data_ptr(),
                     rec["label"].data_ptr())
    if ws is None:
        ws = workspace("fit" if fp16_operands else "apply", N, D, K, dev)
    st = lib().cat_assign_scores(_dev(Yq, torch.float32, None, "Yq"), N, D, K,
                                 _dev(centroids, torch.float32, (K, D), "centroids"), _dev(labels, torch.int32),
                                 ctypes.byref(fs), ASSIGN_FP16_OPERANDS if fp16_operands else 0,
                                 ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_assign_scores")
    return labels, rec


NOALLOC_MAX_ROWS = 262144


def cat_assign_noalloc(Yq, centroids, labels_out):
    """cat_assign_noalloc: labels into the caller's `labels_out`; the library uses its own
    fixed scratch (no workspace, no allocation).  At most NOALLOC_MAX_ROWS rows; calls that
    could overlap on the GPU must be ordered by the caller."""
    N, D = Yq.shape
    K = centroids.shape[0]
    st = lib().cat_assign_noalloc(_dev(Yq, torch.float32, None, "Yq"), N, D, K,
                                  _dev(centroids, torch.float32, (K, D), "centroids"),
                                  _dev(labels_out, torch.int32, (N,), "labels_out"), _stream())
    _check(st, "cat_assign_noalloc")
    return labels_out


def cat_fit_shard_begin(Yq, K: int, amax_out, ws):
    N, D = Yq.shape
    _check(lib().cat_fit_shard_begin(_dev(Yq, torch.float32, None, "Yq"), N, D, K, _dev(amax_out, torch.float32, (1,)),
                                     ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream()), "cat_fit_shard_begin")


def cat_fit_shard_round(Yq, K: int, rnd: int, centroids, amax, delta_sums, delta_counts, labels_out, ws):
    N, D = Yq.shape
    _check(lib().cat_fit_shard_round(_dev(Yq, torch.float32, None, "Yq"), N, D, K, int(rnd),
                                     _dev(centroids, torch.float32, (K, D), "centroids"), _dev(amax, torch.float32, (1,)),
                                     _dev(delta_sums, torch.float64, (K, D)), _dev(delta_counts, torch.int64, (K,)),
                                     _dev(labels_out, torch.int32, (N,)),
                                     ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream()), "cat_fit_shard_round")


def cat_fit_shard_update(delta_sums, delta_counts, sums, counts, centroids):
    K, D = centroids.shape
    _check(lib().cat_fit_shard_update(_dev(delta_sums, torch.float64, (K, D)), _dev(delta_counts, torch.int64, (K,)),
                                      D, K, _dev(sums, torch.float64, (K, D)), _dev(counts, torch.int64, (K,)),
                                      _dev(centroids, torch.float32, (K, D)), _stream()), "cat_fit_shard_update")


def _scratch(nbytes: int, device, where: str):
    if nbytes == 0:
        raise CatError(7, where + " workspace query")
    return torch.empty(int(nbytes), dtype=torch.uint8, device=device)


def cat_pca_fit(Yq, p: int, want_eigenvalues=False):
    """Returns (mean [D], components [p, D][, eigenvalues float64 [p]])."""
    N, D = Yq.shape
    dev = Yq.device
    mean = torch.empty((D,), dtype=torch.float32, device=dev)
    comps = torch.empty((p, D), dtype=torch.float32, device=dev)
    eig = torch.empty((p,), dtype=torch.float64, device=dev) if want_eigenvalues else None
    ws = _scratch(lib().cat_pca_workspace_bytes(N, D, p), dev, "cat_pca_fit")
    _check(lib().cat_pca_fit(_dev(Yq, torch.float32, None, "Yq"), N, D, p, _dev(mean, torch.float32),
                             _dev(comps, torch.float32), _dev(eig, torch.float64),
                             ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream()), "cat_pca_fit")
    return (mean, comps, eig) if want_eigenvalues else (mean, comps)


def cat_pca_project(Y, mean, comps):
    N, D = Y.shape
    p = comps.shape[0]
    Z = torch.empty((N, p), dtype=torch.float32, device=Y.device)
    _check(lib().cat_pca_project(_dev(Y, torch.float32, None, "Y"), N, D, p, _dev(mean, torch.float32, (D,), "mean"),
                                 _dev(comps, torch.float32, (p, D), "components"), _dev(Z, torch.float32), _stream()),
           "cat_pca_project")
    return Z


def cat_affine_with_labels(Yq, labels, gamma, beta, out=None):
    N, D = Yq.shape
    K = gamma.shape[0]
    if out is None:
        out = torch.empty_like(Yq)
    _check(lib().cat_affine_with_labels(_dev(Yq, torch.float32, None, "Yq"), N, D, K, _dev(labels, torch.int32, (N,), "labels"),
                                        _dev(gamma, torch.float32, (K, D), "gamma"), _dev(beta, torch.float32, (K, D), "beta"),
                                        _dev(out, torch.float32, (N, D), "out"), _stream()), "cat_affine_with_labels")
    return out


def cat_fit_pca(Yq, Yfp, K: int, iters: int, p: int):
    """Returns dict(mean, comps, centroids [K, p], gamma, beta [K, D], labels)."""
    N, D = Yq.shape
    dev = Yq.device
    r = dict(mean=torch.empty((D,), dtype=torch.float32, device=dev),
             comps=torch.empty((p, D), dtype=torch.float32, device=dev),
             centroids=torch.empty((K, p), dtype=torch.float32, device=dev),
             gamma=torch.empty((K, D), dtype=torch.float32, device=dev),
             beta=torch.empty((K, D), dtype=torch.float32, device=dev),
             labels=torch.empty((N,), dtype=torch.int32, device=dev))
    ws = _scratch(lib().cat_fit_pca_workspace_bytes(N, D, K, p), dev, "cat_fit_pca")
    _check(lib().cat_fit_pca(_dev(Yq, torch.float32, None, "Yq"), _dev(Yfp, torch.float32, (N, D), "Yfp"), N, D, K, iters, p,
                             _dev(r["mean"], torch.float32), _dev(r["comps"], torch.float32),
                             _dev(r["centroids"], torch.float32), _dev(r["gamma"], torch.float32),
                             _dev(r["beta"], torch.float32), _dev(r["labels"], torch.int32),
                             ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream()), "cat_fit_pca")
    return r


def cat_apply_pca(Yq, mean, comps, centroids, gamma, beta, out=None, want_labels=False):
    N, D = Yq.shape
    K, p = centroids.shape
    dev = Yq.device
    if out is None:
        out = torch.empty_like(Yq)
    labels = torch.empty((N,), dtype=torch.int32, device=dev) if want_labels else None
    ws = _scratch(lib().cat_apply_pca_workspace_bytes(N, D, K, p), dev, "cat_apply_pca")
    _check(lib().cat_apply_pca(_dev(Yq, torch.float32, None, "Yq"), N, D, K, p, _dev(mean, torch.float32, (D,)),
                               _dev(comps, torch.float32, (p, D)), _dev(centroids, torch.float32, (K, p)),
                               _dev(gamma, torch.float32, (K, D)), _dev(beta, torch.float32, (K, D)),
                               _dev(out, torch.float32, (N, D)), _dev(labels, torch.int32),
                               ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream()), "cat_apply_pca")
    return (out, labels) if want_labels else out


def cat_cluster_sums(Y, labels, K: int, ws=None):
    """Returns (sums float64 [K, D], counts int64 [K])."""
    N, D = Y.shape
    sums = torch.empty((K, D), dtype=torch.float64, device=Y.device)
    counts = torch.empty((K,), dtype=torch.int64, device=Y.device)
    ws = workspace("fit", N, D, K, Y.device) if ws is None else ws
    st = lib().cat_cluster_sums(_dev(Y, torch.float32, None, "Y"), _dev(labels, torch.int32, (N,), "labels"),
                                N, D, K, _dev(sums, torch.float64), _dev(counts, torch.int64),
                                ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_cluster_sums")
    return sums, counts


def cat_centroids_from_sums(sums, counts, centroids):
    K, D = centroids.shape
    st = lib().cat_centroids_from_sums(_dev(sums, torch.float64, (K, D), "sums"),
                                       _dev(counts, torch.int64, (K,), "counts"), D, K,
                                       _dev(centroids, torch.float32), _stream())
    _check(st, "cat_centroids_from_sums")
    return centroids


def cat_centred_moments(Yq, Yfp, labels, meanQ, meanF, ws=None):
    """Returns (var_sum, cov_sum) float64 [K, D]."""
    N, D = Yq.shape
    K = meanQ.shape[0]
    var = torch.empty((K, D), dtype=torch.float64, device=Yq.device)
    cov = torch.empty((K, D), dtype=torch.float64, device=Yq.device)
    ws = workspace("fit", N, D, K, Yq.device) if ws is None else ws
    st = lib().cat_centred_moments(_dev(Yq, torch.float32, None, "Yq"), _dev(Yfp, torch.float32, (N, D), "Yfp"),
                                   _dev(labels, torch.int32, (N,), "labels"), N, D, K,
                                   _dev(meanQ, torch.float64, (K, D), "meanQ"),
                                   _dev(meanF, torch.float64, (K, D), "meanF"),
                                   _dev(var, torch.float64), _dev(cov, torch.float64),
                                   ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_centred_moments")
    return var, cov


def cat_solve_gamma_beta(sumQ, sumF, var_sum, cov_sum, counts):
    K, D = sumQ.shape
    gamma = torch.empty((K, D), dtype=torch.float32, device=sumQ.device)
    beta = torch.empty((K, D), dtype=torch.float32, device=sumQ.device)
    st = lib().cat_solve_gamma_beta(_dev(sumQ, torch.float64), _dev(sumF, torch.float64, (K, D)),
                                    _dev(var_sum, torch.float64, (K, D)), _dev(cov_sum, torch.float64, (K, D)),
                                    _dev(counts, torch.int64, (K,)), D, K,
                                    _dev(gamma, torch.float32), _dev(beta, torch.float32), _stream())
    _check(st, "cat_solve_gamma_beta")
    return gamma, beta


def cat_apply_host(Yq_host, centroids_host, gamma_host, beta_host, out_host, labels_host=None,
                   device="cuda", ws=None):
    """cat_apply_host: CPU tensors in and out (page-locked for overlap); blocks until done."""
    N, D = Yq_host.shape
    K = centroids_host.shape[0]
    ws = workspace("apply_host", N, D, K, device) if ws is None else ws
    st = lib().cat_apply_host(_cpu(Yq_host, torch.float32, None, "Yq_host"), N, D, K,
                              _cpu(centroids_host, torch.float32, (K, D)), _cpu(gamma_host, torch.float32, (K, D)),
                              _cpu(beta_host, torch.float32, (K, D)), _cpu(out_host, torch.float32, (N, D)),
                              _cpu(labels_host, torch.int32, (N,)),
                              ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_apply_host")
    return out_host


def cat_fit_host(Yq_host, Yfp_host, K: int, iters: int, C_host, G_host, B_host, labels_host=None,
                 device="cuda", ws=None):
    """cat_fit_host: CPU tensors in and out; blocks until done."""
    N, D = Yq_host.shape
    ws = workspace("fit_host", N, D, K, device) if ws is None else ws
    st = lib().cat_fit_host(_cpu(Yq_host, torch.float32, None, "Yq_host"), _cpu(Yfp_host, torch.float32, (N, D)),
                            N, D, K, iters, _cpu(C_host, torch.float32, (K, D)),
                            _cpu(G_host, torch.float32, (K, D)), _cpu(B_host, torch.float32, (K, D)),
                            _cpu(labels_host, torch.int32, (N,)),
                            ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream())
    _check(st, "cat_fit_host")
    return C_host, G_host, B_host


def cat_selftest_wait_timeout(ws, limit_ms: int = 20) -> None:
    """Enqueue the bounded-wait self-test on workspace `ws` (see cat.h); read the outcome with
    cat_workspace_report."""
    _check(lib().cat_selftest_wait_timeout(ctypes.c_void_p(ws.data_ptr()), ws.numel() * ws.element_size(),
                                           int(limit_ms), _stream()), "cat_selftest_wait_timeout")


def cat_workspace_report(ws) -> dict:
    """Counters of the calls that last used workspace `ws` (synchronises the current stream)."""
    last, total, status = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int32(0)
    st = lib().cat_workspace_report(ctypes.c_void_p(ws.data_ptr()), _stream(), ctypes.byref(last),
                                    ctypes.byref(total), ctypes.byref(status))
    _check(st, "cat_workspace_report")
    return dict(refined_rows_last=last.value, refined_rows_total=total.value, device_status=status.value)


def cat_set_tensor_core_min_k(min_k: int) -> None:
    lib().cat_set_tensor_core_min_k(int(min_k))


def cat_get_tensor_core_min_k() -> int:
    return int(lib().cat_get_tensor_core_min_k())


def cat_set_small_problem_kernels(mask: int) -> None:
    """Process-wide switch of the persistent single-launch kernels for small shapes:
    bit 0 = inference, bit 1 = the K-Means rounds of a fit (default 3: both on)."""
    lib().cat_set_small_problem_kernels(int(mask))


def cat_get_small_problem_kernels() -> int:
    return int(lib().cat_get_small_problem_kernels())


def cat_tensor_path_available() -> bool:
    return bool(lib().cat_tensor_path_available())


def cat_set_apply_column_split(cs: int) -> None:
    lib().cat_set_apply_column_split(int(cs))


def cat_get_apply_column_split() -> int:
    return int(lib().cat_get_apply_column_split())


def cat_version() -> str:
    return lib().cat_version().decode()


def cat_kernel_launches() -> int:
    return int(lib().cat_kernel_launches())
