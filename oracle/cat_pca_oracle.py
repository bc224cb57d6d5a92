"""CPU oracle for CAT with the PCA front-end (test infrastructure: only tests, the smoke check
and bench.py's CPU baseline may import it; the product never does).

Section 3.1 reduces the LQ outputs with PCA before clustering ("PCA is only used to obtain
clusters": the affine correction stays in the original D-dimensional space); Algorithm 1 step 1
fits the projection on all_q, Algorithm 2 step 1 applies it to the new outputs.

Plain numpy, fp64 throughout.  The eigen-decomposition is numpy.linalg.eigh on the D x D
covariance of the centred rows (a library routine serving as one step); everything else is
written out.  Readings where the paper is silent: the rows are centred with the column means of
the fit set; components are ordered by decreasing eigenvalue; each component's sign is fixed so
that its entry of largest magnitude is positive (lowest index on equal magnitudes); the
projected rows are stored in fp32, like every matrix that crosses the library's boundary.
"""
from __future__ import annotations

import numpy as np

from . import cat_oracle as O


def pca_fit(Yq, p: int):
    """Column means, top-p principal directions (rows of the returned [p, D] matrix) and their
    eigenvalues (variances with the 1 / (N - 1) normalisation), from the rows of Yq."""
    Y = np.asarray(Yq, dtype=np.float64)
    N, D = Y.shape
    assert 1 <= p <= D and N >= 2
    mean = Y.sum(axis=0) / N
    Yc = Y - mean
    cov = (Yc.T @ Yc) / (N - 1)
    w, V = np.linalg.eigh(cov)                 # ascending eigenvalues, eigenvectors in columns
    order = np.argsort(-w, kind="stable")[:p]
    comps = V[:, order].T.copy()               # [p, D]
    for r in range(p):
        j = int(np.argmax(np.abs(comps[r])))   # first index of the largest magnitude
        if comps[r, j] < 0:
            comps[r] = -comps[r]
    return mean, comps, w[order]


def pca_transform(Y, mean, comps):
    """Z = (Y - mean) comps^T, computed in fp64 and stored in fp32."""
    Y = np.asarray(Y, dtype=np.float64)
    return ((Y - np.asarray(mean, np.float64)) @ np.asarray(comps, np.float64).T).astype(np.float32)


def fit_pca(Yq, Yfp, K: int, iters: int, p: int):
    """Algorithm 1 as printed: PCA on all_q, K-Means on the reduced rows (first K reduced rows
    as the start, `iters` Lloyd rounds, one final assignment), then per cluster the closed-form
    gamma/beta from the ORIGINAL D-dimensional Yq, Yfp.
    Returns dict(mean, comps, eig, Z, centroids [K, p], labels, gamma, beta, J, near)."""
    mean, comps, eig = pca_fit(Yq, p)
    Z = pca_transform(Yq, mean.astype(np.float32), comps.astype(np.float32))
    km = O.fit(Z, Z, K, iters)                 # cluster model in the reduced space (its gamma/beta are not used)
    gamma, beta = O.solve_gamma_beta(Yq, Yfp, km.labels, K)
    return dict(mean=mean.astype(np.float32), comps=comps.astype(np.float32), eig=eig, Z=Z,
                centroids=km.centroids, labels=km.labels, gamma=gamma, beta=beta, J=km.J, near=km.near)


def apply_pca(Yq, mean, comps, centroids, gamma, beta, alpha: float = 1.0):
    """Algorithm 2 as printed: project, predict the cluster in the reduced space, correct in the
    original space.  Returns (out, labels, best, second)."""
    Z = pca_transform(Yq, mean, comps)
    labels, best, second = O.assign(Z, centroids)
    out = O.affine_with_labels(Yq, labels, gamma, beta, alpha)
    return out, labels, best, second


def projector_distance(A, B):
    """Largest singular value of P_A - P_B for the row spaces of A and B (0 for equal subspaces,
    1 for subspaces that share no direction): the sine of the largest principal angle."""
    Qa = np.linalg.qr(np.asarray(A, np.float64).T)[0]
    Qb = np.linalg.qr(np.asarray(B, np.float64).T)[0]
    return float(np.linalg.norm(Qa @ Qa.T - Qb @ Qb.T, 2))
