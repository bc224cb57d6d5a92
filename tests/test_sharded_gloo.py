"""Row-sharded fitting over 2 processes (gloo, CPU): the collective logic of
paper_2509_26277_b200.sharded with a CPU stand-in for the per-rank CUDA steps.
The sharded result must equal the single-process oracle on the whole matrix."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import cat_oracle as O
from paper_2509_26277_b200 import sharded


class CpuStandIn:
    """Per-rank steps for the test: the oracle's assignment, numpy fp64 sums."""

    def begin(self, Yq, K):
        self.K = K
        self.prev = None
        return Yq.abs().max().reshape(1).float()

    def round(self, Yq, rnd, C, amax):
        """Labels from the oracle; what changed in the per-cluster sums since the previous round."""
        labels = O.assign(Yq.numpy(), C.numpy())[0]
        y = Yq.numpy().astype(np.float64)
        dsums = np.zeros((self.K, y.shape[1]), np.float64)
        dcounts = np.zeros(self.K, np.int64)
        moved = np.ones(len(y), bool) if self.prev is None else labels != self.prev
        np.add.at(dsums, labels[moved], y[moved])
        np.add.at(dcounts, labels[moved], 1)
        if self.prev is not None:
            np.add.at(dsums, self.prev[moved], -y[moved])
            np.add.at(dcounts, self.prev[moved], -1)
        self.prev = labels
        return torch.from_numpy(dsums), torch.from_numpy(dcounts), torch.from_numpy(labels)

    def update(self, dsums, dcounts, sums, counts, C):
        sums += dsums
        counts += dcounts
        m = counts > 0
        C[m] = (sums[m] / counts[m].double()[:, None]).float()

    def cluster_sums(self, Y, labels, K):
        sums = np.zeros((K, Y.shape[1]), np.float64)
        np.add.at(sums, labels.numpy(), Y.numpy().astype(np.float64))
        counts = np.bincount(labels.numpy(), minlength=K).astype(np.int64)
        return torch.from_numpy(sums), torch.from_numpy(counts)

    def centred_moments(self, Yq, Yfp, labels, meanQ, meanF):
        l = labels.numpy()
        dq = Yq.numpy().astype(np.float64) - meanQ.numpy()[l]
        df = Yfp.numpy().astype(np.float64) - meanF.numpy()[l]
        var = np.zeros(meanQ.shape)
        cov = np.zeros(meanQ.shape)
        np.add.at(var, l, dq * dq)
        np.add.at(cov, l, dq * df)
        return torch.from_numpy(var), torch.from_numpy(cov)

    def solve(self, sumQ, sumF, var, cov, counts):
        n = counts.double()[:, None]
        empty = (counts == 0)[:, None]
        nn = n.clamp(min=1)
        g = (cov / nn) / torch.clamp(var / nn, min=1e-8)
        b = sumF / nn - g * (sumQ / nn)
        g = torch.where(empty, torch.ones_like(g), g)
        b = torch.where(empty, torch.zeros_like(b), b)
        return g.float(), b.float()

    def apply(self, Yq, C, gamma, beta, out=None):
        return torch.from_numpy(O.apply(Yq.numpy(), C.numpy(), gamma.numpy(), beta.numpy())[0])


def _data():
    r = np.random.default_rng(123)
    centers = r.normal(size=(5, 12)) * 3
    comp = r.integers(0, 5, size=601)
    Yq = (centers[comp] + r.normal(size=(601, 12))).astype(np.float32)
    Yfp = (Yq * 1.2 + 0.3 + 0.2 * r.normal(size=(601, 12))).astype(np.float32)
    return Yq, Yfp


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Yq, Yfp = _data()
        lo, hi = sharded.shard_bounds(len(Yq), world, rank)
        C, g, b, labels = sharded.fit_sharded(torch.from_numpy(Yq[lo:hi]), torch.from_numpy(Yfp[lo:hi]),
                                              5, 6, backend=CpuStandIn())
        out = sharded.apply_sharded(torch.from_numpy(Yq[lo:hi]), C, g, b, backend=CpuStandIn())
        q.put((rank, lo, hi, C.numpy(), g.numpy(), b.numpy(), labels.numpy(), out.numpy()))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def _worker_uneven(rank, world, port, q):
    """Rank 1 holds no rows at all: it must pass through every collective with zeros."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Yq, Yfp = _data()
        lo, hi = (0, len(Yq)) if rank == 0 else (len(Yq), len(Yq))
        C, g, b, labels = sharded.fit_sharded(torch.from_numpy(Yq[lo:hi]), torch.from_numpy(Yfp[lo:hi]),
                                              5, 4, backend=CpuStandIn())
        q.put((rank, C.numpy(), g.numpy(), b.numpy(), labels.numpy()))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_shard_bounds_cover_all_rows():
    for n, w in [(10, 3), (601, 2), (7, 8), (4_194_304, 8)]:
        spans = [sharded.shard_bounds(n, w, r) for r in range(w)]
        assert spans[0][0] == 0 and spans[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        sizes = [hi - lo for lo, hi in spans]
        assert max(sizes) - min(sizes) <= 1


def test_single_process_sharded_equals_oracle():
    Yq, Yfp = _data()
    C, g, b, labels = sharded.fit_sharded(torch.from_numpy(Yq), torch.from_numpy(Yfp), 5, 6,
                                          backend=CpuStandIn())
    ora = O.fit(Yq, Yfp, 5, 6)
    assert np.array_equal(labels.numpy(), ora.labels)
    np.testing.assert_allclose(C.numpy(), ora.centroids, rtol=1e-6, atol=1e-6)
    np.testing.assert_allclose(g.numpy(), ora.gamma, rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(b.numpy(), ora.beta, rtol=1e-5, atol=1e-6)


@pytest.mark.timeout(300)
def test_two_rank_gloo_fit_equals_single_process_oracle():
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted([q.get(timeout=240) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    Yq, Yfp = _data()
    ora = O.fit(Yq, Yfp, 5, 6)
    want_out = O.apply(Yq, ora.centroids, ora.gamma, ora.beta)[0]
    for rank, lo, hi, C, g, b, labels, out in results:
        np.testing.assert_allclose(C, ora.centroids, rtol=1e-6, atol=1e-6)
        np.testing.assert_allclose(g, ora.gamma, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(b, ora.beta, rtol=1e-5, atol=1e-6)
        assert np.array_equal(labels, ora.labels[lo:hi])
        np.testing.assert_allclose(out, want_out[lo:hi], rtol=1e-5, atol=1e-6)
    # both ranks hold bit-identical models
    for a, b_ in zip(results[0][3:6], results[1][3:6]):
        assert np.array_equal(a, b_)


@pytest.mark.timeout(300)
def test_a_rank_without_rows_takes_part_with_zeros():
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker_uneven, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted([q.get(timeout=240) for _ in range(world)], key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    Yq, Yfp = _data()
    ora = O.fit(Yq, Yfp, 5, 4)
    for rank, C, g, b, labels in results:
        np.testing.assert_allclose(C, ora.centroids, rtol=1e-6, atol=1e-6)
        np.testing.assert_allclose(g, ora.gamma, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(b, ora.beta, rtol=1e-5, atol=1e-6)
    assert np.array_equal(results[0][4], ora.labels) and len(results[1][4]) == 0
