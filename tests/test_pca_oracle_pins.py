"""Pins for the PCA front-end of the CPU oracle (Section 3.1, Algorithm 1 step 1, Algorithm 2
step 1): against scikit-learn's PCA, against planted low-rank data, and against identities that a
dropped mean, a transposed operand or a wrong ordering would break."""
import numpy as np
import pytest

from oracle import cat_oracle as O
from oracle import cat_pca_oracle as P


def _lowrank(seed, n, d, r, noise=0.01):
    rng = np.random.default_rng(seed)
    basis = np.linalg.qr(rng.normal(size=(d, r)))[0].T            # [r, d], orthonormal rows
    scales = np.linspace(5.0, 1.0, r)
    Y = (rng.normal(size=(n, r)) * scales) @ basis + 3.0 + noise * rng.normal(size=(n, d))
    return Y.astype(np.float32), basis


def test_matches_scikit_learn_pca():
    sk = pytest.importorskip("sklearn.decomposition")
    Y, _ = _lowrank(1, 400, 30, 6, noise=0.3)
    mean, comps, eig = P.pca_fit(Y, 6)
    ref = sk.PCA(n_components=6, svd_solver="full").fit(Y.astype(np.float64))
    np.testing.assert_allclose(mean, ref.mean_, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(eig, ref.explained_variance_, rtol=1e-9)
    for a, b in zip(comps, ref.components_):                       # same directions up to sign
        assert min(np.abs(a - b).max(), np.abs(a + b).max()) < 1e-8
    Z = P.pca_transform(Y, mean, comps)
    Zr = ref.transform(Y.astype(np.float64))
    for j in range(6):
        s = np.sign(comps[j] @ ref.components_[j])
        np.testing.assert_allclose(Z[:, j], s * Zr[:, j], rtol=1e-5, atol=1e-5)


def test_planted_subspace_is_recovered_and_ordered():
    Y, basis = _lowrank(2, 2000, 40, 5, noise=1e-3)
    mean, comps, eig = P.pca_fit(Y, 5)
    assert P.projector_distance(comps, basis) < 1e-2
    assert np.all(np.diff(eig) <= 0)                               # decreasing variances
    np.testing.assert_allclose(comps @ comps.T, np.eye(5), atol=1e-12)   # orthonormal
    # with the scales 5 ... 1 the first direction is the first planted one
    assert abs(abs(comps[0] @ basis[0]) - 1) < 1e-2


def test_sign_convention_and_centering():
    Y, _ = _lowrank(3, 300, 12, 4, noise=0.2)
    mean, comps, _ = P.pca_fit(Y, 4)
    for c in comps:
        assert c[np.argmax(np.abs(c))] > 0
    Z = P.pca_transform(Y, mean, comps).astype(np.float64)
    assert np.abs(Z.mean(axis=0)).max() < 1e-5                    # centred rows project to mean zero
    # a dropped mean would show here: shifting every row moves nothing but the mean
    mean2, comps2, eig2 = P.pca_fit(Y.astype(np.float64) + 100.0, 4)
    np.testing.assert_allclose(mean2, mean + 100.0, rtol=1e-9)
    np.testing.assert_allclose(eig2, P.pca_fit(Y, 4)[2], rtol=1e-9)
    assert P.projector_distance(comps2, comps) < 1e-9


def test_variance_of_projection_and_reconstruction_error():
    Y, _ = _lowrank(4, 500, 20, 20, noise=0.0)
    Yd = Y.astype(np.float64)
    mean, comps, eig = P.pca_fit(Y, 7)
    Z = (Yd - mean) @ comps.T
    np.testing.assert_allclose(Z.var(axis=0, ddof=1), eig, rtol=1e-9)       # eigenvalue = variance along its direction
    all_eig = P.pca_fit(Y, 20)[2]
    rec = Z @ comps + mean
    err = ((Yd - rec) ** 2).sum() / (len(Y) - 1)
    np.testing.assert_allclose(err, all_eig[7:].sum(), rtol=1e-8)           # what is cut off is the discarded variance


def test_full_rank_projection_keeps_the_clustering():
    """p = D is a rotation of the centred rows: distances, hence the whole K-Means run, are the ones
    of the unprojected rows (up to the fp32 storage of Z, so compared on well separated data)."""
    rng = np.random.default_rng(5)
    cen = rng.normal(size=(4, 10)) * 6
    Yq = (cen[rng.integers(0, 4, size=300)] + 0.3 * rng.normal(size=(300, 10))).astype(np.float32)
    Yfp = (Yq * 1.1 + 0.05 * rng.normal(size=Yq.shape)).astype(np.float32)
    full = P.fit_pca(Yq, Yfp, 4, 6, p=10)
    plain = O.fit(Yq, Yfp, 4, 6)
    assert np.array_equal(full["labels"], plain.labels)
    np.testing.assert_allclose(full["gamma"], plain.gamma, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(full["beta"], plain.beta, rtol=1e-6, atol=1e-7)
    out, labels, _, _ = P.apply_pca(Yq, full["mean"], full["comps"], full["centroids"], full["gamma"], full["beta"])
    assert np.array_equal(labels, plain.labels)
    np.testing.assert_array_equal(out, O.affine_with_labels(Yq, plain.labels, plain.gamma, plain.beta))


def test_affine_stays_in_the_original_space():
    """gamma and beta have D columns whatever p is, and with Yfp = a Yq + b they recover (a, b)."""
    rng = np.random.default_rng(6)
    Yq = rng.normal(size=(500, 16)).astype(np.float32)
    a, b = rng.uniform(0.5, 2, size=16), rng.normal(size=16)
    Yfp = (Yq * a + b).astype(np.float32)
    r = P.fit_pca(Yq, Yfp, 3, 5, p=2)
    assert r["gamma"].shape == (3, 16) and r["centroids"].shape == (3, 2)
    np.testing.assert_allclose(r["gamma"], np.tile(a, (3, 1)), rtol=1e-4)
    np.testing.assert_allclose(r["beta"], np.tile(b, (3, 1)), rtol=1e-3, atol=1e-4)
