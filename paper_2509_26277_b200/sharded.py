"""Row-sharded CAT fitting and inference over several GPUs (one process per GPU).

Rows are independent in every step of CAT except the per-cluster sums, so each
rank keeps a contiguous shard of the rows and the only exchange is an
all-reduce (sum) of the K x D partial sums and K counts once per Lloyd round,
and of the four statistics of the closed form once per fit.  Inference needs no
collective: centroids, gamma and beta are replicated.

`backend` supplies the per-rank compute steps.  The default is the CUDA library
(binding); tests inject a CPU stand-in to exercise the collective logic with the
gloo backend.  With group=None or world size 1 no collective is issued.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


class CudaBackend:
    """Per-rank steps on the CUDA library (step-level entry points of cat.h)."""

    def __init__(self):
        from . import binding
        self.b = binding

    def assign(self, Yq, C):
        return self.b.cat_assign(Yq, C)

    def cluster_sums(self, Y, labels, K):
        return self.b.cat_cluster_sums(Y, labels, K)

    def centroids_from_sums(self, sums, counts, C):
        return self.b.cat_centroids_from_sums(sums, counts, C)

    def centred_moments(self, Yq, Yfp, labels, meanQ, meanF):
        return self.b.cat_centred_moments(Yq, Yfp, labels, meanQ, meanF)

    def solve(self, sumQ, sumF, var, cov, counts):
        return self.b.cat_solve_gamma_beta(sumQ, sumF, var, cov, counts)

    def apply(self, Yq, C, gamma, beta, out=None):
        return self.b.cat_apply(Yq, C, gamma, beta, out=out)


def _world(group) -> int:
    if group is None and not (dist.is_available() and dist.is_initialized()):
        return 1
    return dist.get_world_size(group)


def _allreduce(t: torch.Tensor, group):
    if _world(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


def shard_bounds(n_rows: int, world: int, rank: int):
    """Contiguous, balanced row range [lo, hi) of `rank`."""
    base, rem = divmod(n_rows, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def fit_sharded(Yq_local, Yfp_local, K: int, iters: int, group=None, backend=None,
                init_centroids: Optional[torch.Tensor] = None):
    """CAT fitting over row shards.  Every rank returns identical
    (centroids, gamma, beta) and its own shard's labels.

    Without init_centroids the first K rows of rank 0's shard start the
    clustering (rank 0 must hold at least K rows) and are broadcast."""
    backend = backend or CudaBackend()
    world = _world(group)
    D = Yq_local.shape[1]
    if init_centroids is not None:
        C = init_centroids.clone()
    else:
        rank = dist.get_rank(group) if world > 1 else 0
        if rank == 0:
            if Yq_local.shape[0] < K:
                raise ValueError("rank 0 needs at least K rows to seed the centroids")
            C = Yq_local[:K].clone()
        else:
            C = torch.empty((K, D), dtype=Yq_local.dtype, device=Yq_local.device)
        if world > 1:
            dist.broadcast(C, src=dist.get_global_rank(group, 0) if group is not None else 0, group=group)
    for _ in range(iters):
        labels = backend.assign(Yq_local, C)
        sums, counts = backend.cluster_sums(Yq_local, labels, K)
        _allreduce(sums, group)
        _allreduce(counts, group)
        backend.centroids_from_sums(sums, counts, C)
    labels = backend.assign(Yq_local, C)
    sumQ, counts = backend.cluster_sums(Yq_local, labels, K)
    sumF, _ = backend.cluster_sums(Yfp_local, labels, K)
    _allreduce(sumQ, group)
    _allreduce(sumF, group)
    _allreduce(counts, group)
    n = counts.clamp(min=1).to(torch.float64)[:, None]
    var, cov = backend.centred_moments(Yq_local, Yfp_local, labels, sumQ / n, sumF / n)
    _allreduce(var, group)
    _allreduce(cov, group)
    gamma, beta = backend.solve(sumQ, sumF, var, cov, counts)
    return C, gamma, beta, labels


def apply_sharded(Yq_local, C, gamma, beta, backend=None, out=None):
    """CAT inference on this rank's rows (no communication)."""
    backend = backend or CudaBackend()
    return backend.apply(Yq_local, C, gamma, beta, out=out)
