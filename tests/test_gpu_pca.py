"""PCA front-end on the GPU against the CPU oracle (Section 3.1, Algorithm 1 step 1, Algorithm 2
step 1).  Eigenvectors are compared as subspaces and, where the spectrum separates them, one by one
(same sign convention on both sides); everything downstream of the projection is compared given the
GPU's own components, so that a rotation inside a near-degenerate eigenspace cannot hide an error."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from oracle import cat_pca_oracle as P
from paper_2509_26277_b200 import binding as B
from paper_2509_26277_b200 import workloads as W
from tests.parity import close, labels_match

pytestmark = pytest.mark.gpu


def host(t):
    return t.detach().cpu().numpy()


def dev(a):
    return torch.as_tensor(np.ascontiguousarray(a)).cuda()


def _lowrank(seed, n, d, r, noise):
    rng = np.random.default_rng(seed)
    basis = np.linalg.qr(rng.normal(size=(d, r)))[0].T
    Y = (rng.normal(size=(n, r)) * np.linspace(6.0, 1.5, r)) @ basis + 2.0 + noise * rng.normal(size=(n, d))
    return Y.astype(np.float32)


@pytest.mark.parametrize("n,d,p", [(500, 30, 1), (700, 64, 8), (1500, 1000, 50), (900, 257, 20), (300, 12, 12)])
def test_pca_fit_matches_the_oracle(n, d, p):
    Y = _lowrank(n + d + p, n, d, min(d, max(p + 3, 10)), noise=0.2)
    mean, comps, eig = B.cat_pca_fit(dev(Y), p, want_eigenvalues=True)
    o_mean, o_comps, o_eig = P.pca_fit(Y, p)
    close(host(mean), o_mean, "column means")
    np.testing.assert_allclose(host(eig), o_eig, rtol=1e-9, atol=1e-12 * o_eig[0])
    C = host(comps).astype(np.float64)
    np.testing.assert_allclose(C @ C.T, np.eye(p), atol=1e-6)          # unit length, mutually orthogonal (fp32 storage)
    if p < d:
        assert P.projector_distance(C, o_comps) < 1e-5
    gaps = np.minimum(np.abs(np.diff(o_eig, prepend=np.inf)), np.abs(np.diff(o_eig, append=P.pca_fit(Y, min(d, p + 1))[2][-1] if p < d else -np.inf)))
    for r in range(p):
        if gaps[r] > 1e-3 * o_eig[0]:                                  # a direction the spectrum pins down
            np.testing.assert_allclose(C[r], o_comps[r], atol=2e-6)


@pytest.mark.parametrize("n,d,p", [(1000, 1000, 50), (777, 130, 7), (64, 40, 40)])
def test_projection_matches_the_oracle_for_given_components(n, d, p):
    Y = _lowrank(n + p, n, d, min(d, p + 5), noise=0.3)
    mean, comps = B.cat_pca_fit(dev(Y), p)
    Z = B.cat_pca_project(dev(Y), mean, comps)
    want = P.pca_transform(Y, host(mean), host(comps))
    err = np.abs(host(Z).astype(np.float64) - want)
    assert (err <= 1e-6 + 1e-6 * np.abs(want)).all(), float(err.max())   # both round one fp64 sum to fp32


def test_affine_with_labels_is_bit_exact():
    rng = np.random.default_rng(3)
    Yq = rng.normal(size=(3001, 1000)).astype(np.float32)
    g, b = rng.normal(size=(7, 1000)).astype(np.float32), rng.normal(size=(7, 1000)).astype(np.float32)
    labels = rng.integers(0, 7, size=3001).astype(np.int32)
    out = B.cat_affine_with_labels(dev(Yq), dev(labels), dev(g), dev(b))
    np.testing.assert_array_equal(host(out), O.affine_with_labels(Yq, labels, g, b))
    Yo = rng.normal(size=(50, 7)).astype(np.float32)              # D % 4 != 0
    lo = rng.integers(0, 3, size=50).astype(np.int32)
    go, bo = rng.normal(size=(3, 7)).astype(np.float32), rng.normal(size=(3, 7)).astype(np.float32)
    np.testing.assert_array_equal(host(B.cat_affine_with_labels(dev(Yo), dev(lo), dev(go), dev(bo))),
                                  O.affine_with_labels(Yo, lo, go, bo))


@pytest.mark.parametrize("config,p", [(0, 1), (1, 50), (2, 220)])
def test_fit_and_apply_with_pca_on_the_linear_head_configs(config, p):
    """Algorithm 1 and Algorithm 2 as printed, on the D = 1000 workloads with the paper's range of PCA
    dimensions.  Given the library's own components: reduced rows, clustering, gamma/beta and corrected
    outputs must equal the oracle's."""
    w = W.make(config, device="cpu")
    Yq, Yfp, Ya = w.Yq_fit.numpy(), w.Yfp_fit.numpy(), w.Yq_apply.numpy()[:8192]
    r = B.cat_fit_pca(dev(Yq), dev(Yfp), w.K, w.iters, p)
    o_mean, o_comps, _ = P.pca_fit(Yq, p)
    close(host(r["mean"]), o_mean, "means")
    assert P.projector_distance(host(r["comps"]), o_comps) < 1e-4
    # downstream of the projection, with the library's components
    Z = P.pca_transform(Yq, host(r["mean"]), host(r["comps"]))
    km = O.fit(Z, Z, w.K, w.iters)
    lab, best, second = O.assign(Z, host(r["centroids"]))
    labels_match(host(r["labels"]), lab, best, second, "labels in the reduced space")
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(r["labels"]), w.K)
    close(host(r["gamma"]), g_want, "gamma")
    close(host(r["beta"]), b_want, "beta")
    if int(km.near.sum()) == 0:
        assert np.array_equal(host(r["labels"]), km.labels)
        close(host(r["centroids"]), km.centroids, "centroids in the reduced space", abs_tol=2e-6)
    out, alab = B.cat_apply_pca(dev(Ya), r["mean"], r["comps"], r["centroids"], r["gamma"], r["beta"], want_labels=True)
    want, olab, best, second = P.apply_pca(Ya, host(r["mean"]), host(r["comps"]), host(r["centroids"]),
                                           host(r["gamma"]), host(r["beta"]))
    n_near, n_diff = labels_match(host(alab), olab, best, second, "apply labels")
    want2 = want if n_diff == 0 else O.affine_with_labels(Ya, host(alab), host(r["gamma"]), host(r["beta"]))
    np.testing.assert_array_equal(host(out), want2)
    print(f"config {config} p={p}: near-tie rows {n_near} (label differs on {n_diff})")
