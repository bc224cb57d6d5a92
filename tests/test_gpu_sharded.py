"""The CUDA backend of the row-sharded fit on one GPU.

With one shard the cat_fit_shard_* calls run cat_fit's own kernels in cat_fit's order, so the
model must come out bit for bit; two shards on one device (the all-reduce done by hand between
the calls) must agree with the CPU oracle on the whole matrix."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2509_26277_b200 import binding as B
from paper_2509_26277_b200 import sharded
from paper_2509_26277_b200 import workloads as W
from tests.parity import NEAR_REL, close, labels_match

pytestmark = pytest.mark.gpu


def host(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("config,scale", [(1, 1.0), (3, 0.125), (4, 1.0 / 256)])
def test_one_shard_equals_cat_fit(config, scale):
    w = W.make(config, device="cuda", rows_scale=scale)
    C, G, Bt, labels = sharded.fit_sharded(w.Yq_fit, w.Yfp_fit, w.K, w.iters, group=None,
                                           backend=sharded.CudaBackend())
    # (the general path of cat_fit: small shapes would otherwise take the persistent kernel, whose sums
    # are added in another order)
    old = B.cat_get_small_problem_kernels()
    B.cat_set_small_problem_kernels(old & 1)
    try:
        C0, G0, B0, l0 = B.cat_fit(w.Yq_fit, w.Yfp_fit, w.K, w.iters)
    finally:
        B.cat_set_small_problem_kernels(old)
    assert torch.equal(labels, l0)
    assert torch.equal(C, C0)
    close(host(G), host(G0), "gamma, one shard vs cat_fit")
    close(host(Bt), host(B0), "beta, one shard vs cat_fit")
    out = sharded.apply_sharded(w.Yq_apply[:4096], C, G, Bt)
    assert torch.equal(out, B.cat_apply(w.Yq_apply[:4096].contiguous(), C, G, Bt))


@pytest.mark.parametrize("shape", [(3001, 1000, 16), (5000, 64, 64), (2500, 256, 40), (130, 12, 7)])
def test_two_shards_on_one_device_equal_the_oracle(shape):
    """Ranks emulated in one process: each shard has its own backend (workspace, label history);
    the sums of the deltas stand in for the all-reduce."""
    n, d, k = shape
    iters = 5
    rng = np.random.default_rng(n + d + k)
    cen = rng.normal(size=(k, d)) * 2
    Yq = (cen[rng.integers(0, k, size=n)] + rng.normal(size=(n, d))).astype(np.float32)
    Yfp = (Yq * 0.8 + 0.1 * rng.normal(size=(n, d))).astype(np.float32)
    cut = n // 3 + 1
    shards = [(torch.from_numpy(Yq[:cut]).cuda(), torch.from_numpy(Yfp[:cut]).cuda()),
              (torch.from_numpy(Yq[cut:]).cuda(), torch.from_numpy(Yfp[cut:]).cuda())]
    backs = [sharded.CudaBackend(private_workspace=True), sharded.CudaBackend(private_workspace=True)]
    amaxes = [bk.begin(q, k) for bk, (q, _) in zip(backs, shards)]
    amax = torch.maximum(amaxes[0], amaxes[1])
    C = shards[0][0][:k].clone()
    sums = torch.zeros((k, d), dtype=torch.float64, device="cuda")
    counts = torch.zeros((k,), dtype=torch.int64, device="cuda")
    labels = [None, None]
    for rnd in range(iters + 1):
        ds = torch.zeros_like(sums)
        dc = torch.zeros_like(counts)
        for i, (bk, (q, _)) in enumerate(zip(backs, shards)):
            a, b, l = bk.round(q, rnd, C, amax)
            ds += a
            dc += b
            labels[i] = l.clone()
        backs[0].update(ds, dc, sums, counts, C if rnd < iters else C.clone())
    lab = torch.cat(labels)
    ora = O.fit(Yq, Yfp, k, iters, near_rel=NEAR_REL)
    olab, best, second = O.assign(Yq, host(C))
    labels_match(host(lab), olab, best, second, "two-shard labels")
    assert host(counts).tolist() == np.bincount(host(lab), minlength=k).tolist()
    if int(ora.near.sum()) == 0:
        assert np.array_equal(host(lab), ora.labels)
        close(host(C), ora.centroids, "two-shard centroids")
    # the running sums after the final assignment are the per-cluster sums of Yq
    want = np.zeros((k, d))
    np.add.at(want, host(lab), Yq.astype(np.float64))
    np.testing.assert_allclose(host(sums), want, rtol=1e-12, atol=1e-9)
