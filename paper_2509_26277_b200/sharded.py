"""Row-sharded CAT fitting and inference over several GPUs (one process per GPU).

Rows are independent in every step of CAT except the per-cluster sums, so each
rank keeps a contiguous shard of the rows and the only exchange is an
all-reduce once per Lloyd round -- of what the round changed in the K x D
per-cluster sums and the K cluster sizes -- and of the statistics of the closed
form once per fit.  Inference needs no collective: centroids, gamma and beta
are replicated.

`backend` supplies the per-rank compute steps.  The default is the CUDA library
(the cat_fit_shard_* entry points: the same fp16-copy / changed-rows kernels a
single-GPU cat_fit runs); tests inject a CPU stand-in to exercise the collective
logic with the gloo backend.  With world size 1 no collective is issued.  A rank
may hold no rows at all: it skips its local steps and contributes zeros.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


class CudaBackend:
    """Per-rank steps on the CUDA library.  All buffers of a fit are made once in begin()."""

    def __init__(self, private_workspace: bool = False):
        """private_workspace: allocate this backend's own scratch instead of the per-shape cached one
        (needed when several shards of one shape live in one process)."""
        from . import binding
        self.b = binding
        self.private = private_workspace

    def begin(self, Yq, K):
        """Prepares this shard for the rounds; returns its largest magnitude (1 float, device)."""
        N, D = Yq.shape
        dev = Yq.device
        self.K = K
        self.ws = self.b.workspace("fit", N, D, K, dev)
        if self.private:
            self.ws = torch.empty_like(self.ws)
        self.dsums = torch.empty((K, D), dtype=torch.float64, device=dev)
        self.dcounts = torch.empty((K,), dtype=torch.int64, device=dev)
        self.labels = torch.empty((N,), dtype=torch.int32, device=dev)
        amax = torch.zeros((1,), dtype=torch.float32, device=dev)
        self.b.cat_fit_shard_begin(Yq, K, amax, self.ws)
        return amax

    def round(self, Yq, rnd, C, amax):
        """Local half of round `rnd`: (delta_sums, delta_counts, labels) of this shard."""
        self.b.cat_fit_shard_round(Yq, self.K, rnd, C, amax, self.dsums, self.dcounts, self.labels, self.ws)
        return self.dsums, self.dcounts, self.labels

    def update(self, dsums, dcounts, sums, counts, C):
        self.b.cat_fit_shard_update(dsums, dcounts, sums, counts, C)

    def cluster_sums(self, Y, labels, K):
        return self.b.cat_cluster_sums(Y, labels, K, ws=self.ws)

    def centred_moments(self, Yq, Yfp, labels, meanQ, meanF):
        return self.b.cat_centred_moments(Yq, Yfp, labels, meanQ, meanF, ws=self.ws)

    def solve(self, sumQ, sumF, var, cov, counts):
        return self.b.cat_solve_gamma_beta(sumQ, sumF, var, cov, counts)

    def apply(self, Yq, C, gamma, beta, out=None):
        return self.b.cat_apply(Yq, C, gamma, beta, out=out)


def _world(group) -> int:
    if group is None and not (dist.is_available() and dist.is_initialized()):
        return 1
    return dist.get_world_size(group)


def _allreduce(t: torch.Tensor, group, op=dist.ReduceOp.SUM):
    if _world(group) > 1:
        dist.all_reduce(t, op=op, group=group)
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
    n_local, D = Yq_local.shape
    dev = Yq_local.device
    if init_centroids is not None:
        C = init_centroids.clone()
    else:
        rank = dist.get_rank(group) if world > 1 else 0
        if rank == 0:
            if n_local < K:
                raise ValueError("rank 0 needs at least K rows to seed the centroids")
            C = Yq_local[:K].clone()
        else:
            C = torch.empty((K, D), dtype=Yq_local.dtype, device=dev)
        if world > 1:
            dist.broadcast(C, src=dist.get_global_rank(group, 0) if group is not None else 0, group=group)

    def zeros():
        return (torch.zeros((K, D), dtype=torch.float64, device=dev), torch.zeros((K,), dtype=torch.int64, device=dev))

    # a rank without rows takes part in every collective with zeros
    amax = backend.begin(Yq_local, K) if n_local else torch.zeros((1,), dtype=torch.float32, device=dev)
    _allreduce(amax, group, dist.ReduceOp.MAX)
    sums, counts = zeros()
    labels = torch.empty((0,), dtype=torch.int32, device=dev)
    C_final = None
    for rnd in range(iters + 1):
        if n_local:
            dsums, dcounts, labels = backend.round(Yq_local, rnd, C, amax)
        else:
            dsums, dcounts = zeros()
        _allreduce(dsums, group)
        _allreduce(dcounts, group)
        if rnd < iters:
            backend.update(dsums, dcounts, sums, counts, C)
        else:
            # the final assignment moves the running sums and sizes, not the centroids
            C_final = C.clone()
            backend.update(dsums, dcounts, sums, counts, C_final)
    sumQ = sums
    if n_local:
        sumF, _ = backend.cluster_sums(Yfp_local, labels, K)
    else:
        sumF, _ = zeros()
    _allreduce(sumF, group)
    n = counts.clamp(min=1).to(torch.float64)[:, None]
    if n_local:
        var, cov = backend.centred_moments(Yq_local, Yfp_local, labels, sumQ / n, sumF / n)
    else:
        var, cov = zeros()[0], zeros()[0]
    _allreduce(var, group)
    _allreduce(cov, group)
    gamma, beta = backend.solve(sumQ, sumF, var, cov, counts)
    return C, gamma, beta, labels


def apply_sharded(Yq_local, C, gamma, beta, backend=None, out=None):
    """CAT inference on this rank's rows (no communication)."""
    backend = backend or CudaBackend()
    if Yq_local.shape[0] == 0:
        return out if out is not None else torch.empty_like(Yq_local)
    return backend.apply(Yq_local, C, gamma, beta, out=out)
