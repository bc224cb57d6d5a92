"""Full-size workloads in the launch configuration bench.py times, checked on sampled
outputs and on properties the oracle can verify at any size.

Configs 0-2 (D = 1000; 1024, 50 000 and 50 000 apply rows) and config 3 (200 704 x 64, K = 64)
are small enough for the whole protocol on every row.  Config 4
(4 194 304 x 1024 apply, 262 144 x 1024 fit, K = 256) is checked by
  * apply: labels in range on every row; labels and outputs of a seeded row sample
    equal to the oracle's for the same parameters;
  * fit: labels_out is the argmin against centroids_out on a row sample; the centroid
    update between round T and T + 1 equals the oracle's update from the GPU's labels
    (all rows, label-conditioned); gamma/beta equal the oracle's closed form from the
    GPU's labels (all rows).
"""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2509_26277_b200 import binding as B
from paper_2509_26277_b200 import workloads as W
from tests.parity import close, labels_match

pytestmark = pytest.mark.gpu


def host(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("config", [0, 1, 2])
@pytest.mark.parametrize("path", ["fp32", "tensor"])
def test_linear_head_configs_full_size(config, path):
    """The whole fit and the whole apply set (a row pitch of 4000 bytes, several tiles per CTA of the
    persistent kernels), every row against the oracle, on both contraction paths."""
    old = B.cat_get_tensor_core_min_k()
    B.cat_set_tensor_core_min_k(1 << 30 if path == "fp32" else 1)
    try:
        w = W.make(config, device="cpu")
        Yq, Yfp, Ya = w.Yq_fit.numpy(), w.Yfp_fit.numpy(), w.Yq_apply.numpy()
        C, G, Bt, labels = B.cat_fit(w.Yq_fit.cuda(), w.Yfp_fit.cuda(), w.K, w.iters)
        lab, best, second = O.assign(Yq, host(C))
        labels_match(host(labels), lab, best, second, f"config {config} fit labels")
        g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(labels), w.K)
        close(host(G), g_want, f"config {config} gamma")
        close(host(Bt), b_want, f"config {config} beta")
        want, alab_want, best, second = O.apply(Ya, host(C), host(G), host(Bt))
        out, alab = B.cat_apply(w.Yq_apply.cuda(), C, G, Bt, want_labels=True)
        n_near, n_diff = labels_match(host(alab), alab_want, best, second, f"config {config} apply labels")
        want2 = want if n_diff == 0 else O.affine_with_labels(Ya, host(alab), host(G), host(Bt))
        err = close(host(out), want2, f"config {config} apply outputs")
        print(f"config {config} ({path}): apply rows {len(Ya)}, near-tie rows {n_near} (label differs on {n_diff}), "
              f"max |err| {err:.2e}")
    finally:
        B.cat_set_tensor_core_min_k(old)


def test_config3_full_size():
    w = W.make(3, device="cuda")
    Yq, Yfp = host(w.Yq_fit), host(w.Yfp_fit)
    C, G, Bt, labels, diag = B.cat_fit(w.Yq_fit, w.Yfp_fit, w.K, w.iters, want_diag=True)
    C1 = B.cat_fit(w.Yq_fit, w.Yfp_fit, w.K, w.iters + 1, want_labels=False)[0]
    lab, best, second = O.assign(Yq, host(C))
    n_near, n_diff = labels_match(host(labels), lab, best, second, "config 3 fit labels")
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(labels), w.K)
    close(host(G), g_want, "config 3 gamma")
    close(host(Bt), b_want, "config 3 beta")
    C_want, _ = O.update_centroids(Yq, host(labels), host(C))
    close(host(C1), C_want, "config 3 centroid update T -> T+1")
    out, alab = B.cat_apply(w.Yq_apply, C, G, Bt, want_labels=True)
    want = O.affine_with_labels(Yq, host(alab), host(G), host(Bt))
    labels_match(host(alab), lab, best, second, "config 3 apply labels")
    close(host(out), want, "config 3 apply outputs")
    print(f"config 3: near-tie rows {n_near} (differs on {n_diff}), exact-pass rows {diag['refined_rows_total']}")


def test_config4_full_size():
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs about 50 GiB of device memory")
    B.clear_workspaces()
    w = W.make(4, device="cuda")
    K, D = w.K, w.D
    T = 2
    C, G, Bt, labels = B.cat_fit(w.Yq_fit, w.Yfp_fit, K, T)
    C1 = B.cat_fit(w.Yq_fit, w.Yfp_fit, K, T + 1, want_labels=False)[0]
    torch.cuda.synchronize()
    Yq_fit, Yfp_fit = host(w.Yq_fit), host(w.Yfp_fit)
    hl = host(labels)
    assert hl.min() >= 0 and hl.max() < K
    rng = np.random.default_rng(4)
    idx = np.sort(rng.choice(w.N_fit, size=4096, replace=False))
    lab, best, second = O.assign(Yq_fit[idx], host(C))
    labels_match(hl[idx], lab, best, second, "config 4 fit labels (sample)")
    C_want, _ = O.update_centroids(Yq_fit, hl, host(C))
    close(host(C1), C_want, "config 4 centroid update T -> T+1")
    g_want, b_want = O.solve_gamma_beta(Yq_fit, Yfp_fit, hl, K)
    close(host(G), g_want, "config 4 gamma")
    close(host(Bt), b_want, "config 4 beta")
    del Yq_fit, Yfp_fit

    out, alab = B.cat_apply(w.Yq_apply, C, G, Bt, want_labels=True)
    torch.cuda.synchronize()
    assert int(alab.min()) >= 0 and int(alab.max()) < K
    idx = np.sort(rng.choice(w.N_apply, size=8192, replace=False))
    tidx = torch.from_numpy(idx).cuda()
    want, lab, best, second = O.apply(host(w.Yq_apply[tidx]), host(C), host(G), host(Bt))
    labels_match(host(alab[tidx]), lab, best, second, "config 4 apply labels (sample)")
    close(host(out[tidx]), want, "config 4 apply outputs (sample)")
    # every row: the output equals the affine map of its own label (checked on device in fp64,
    # the same single-rounding definition) on a strided subset of columns
    cols = torch.arange(0, D, 37, device="cuda")
    for r0 in range(0, w.N_apply, 1 << 19):
        sl = slice(r0, r0 + (1 << 19))
        l = alab[sl].long()
        y = w.Yq_apply[sl][:, cols].double()
        ref = (G[l][:, cols].double() * y + Bt[l][:, cols].double()).float()
        assert torch.equal(ref, out[sl][:, cols])
    # every form of the fused kernel gives the same labels and the same bits
    del y, ref, l
    for form in (1, 2, 64):
        try:
            B.cat_set_apply_column_split(form)
            out2, alab2 = B.cat_apply(w.Yq_apply, C, G, Bt, want_labels=True)
            torch.cuda.synchronize()
        finally:
            B.cat_set_apply_column_split(0)
        assert torch.equal(alab2, alab), form
        assert torch.equal(out2, out), form
        del out2, alab2
    B.clear_workspaces()
