"""Pins for the CPU oracle: each test checks it against something other than
itself -- a closed form, an invariant, brute force on tiny inputs, or a library
routine in a special case -- chosen so that a dropped term, a wrong sign or
index, or a wrong normalisation in the oracle fails at least one of them."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import cat_oracle as O

HERE = os.path.dirname(os.path.abspath(__file__))


def rng(seed):
    return np.random.default_rng(seed)


# --------------------------------------------------------------------------
# assignment
# --------------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(6))
def test_assign_minimises_total_distance_by_enumeration(seed):
    """For N <= 8, K = 2 the argmin labels are the one labelling (out of all
    K**N) with the smallest total squared distance to fixed centroids.
    Small-integer data keeps every distance exact."""
    r = rng(seed)
    N, D, K = 8, 3, 2
    Y = r.integers(-6, 7, size=(N, D)).astype(np.float32)
    C = r.integers(-6, 7, size=(K, D)).astype(np.float32) + 0.5  # half-integers: no exact ties
    labels, best, second = O.assign(Y, C)
    best_total, best_lab = None, None
    for lab in itertools.product(range(K), repeat=N):
        tot = sum(int(round(4 * np.sum((Y[i].astype(np.float64) - C[l]) ** 2)))
                  for i, l in enumerate(lab))
        if best_total is None or tot < best_total:
            best_total, best_lab = tot, lab
    assert tuple(labels) == best_lab
    assert int(round(4 * best.sum())) == best_total
    assert np.all(second >= best)


def test_assign_matches_cdist_argmin():
    """Special case of a library routine: scipy's squared-Euclidean distance matrix."""
    from scipy.spatial.distance import cdist
    r = rng(10)
    Y = r.normal(size=(300, 37)).astype(np.float32)
    C = r.normal(size=(11, 37)).astype(np.float32)
    labels, best, second = O.assign(Y, C)
    Dm = cdist(Y.astype(np.float64), C.astype(np.float64), "sqeuclidean")
    assert np.array_equal(labels, Dm.argmin(1))
    srt = np.sort(Dm, axis=1)
    np.testing.assert_allclose(best, srt[:, 0], rtol=1e-12)
    np.testing.assert_allclose(second, srt[:, 1], rtol=1e-12)


def test_assign_ties_go_to_lowest_index():
    Y = np.array([[0.0, 0.0], [1.0, 0.0], [5.0, 5.0]], np.float32)
    # centroids 1 and 3 coincide; row 0 is equidistant from centroids 0 and 2
    C = np.array([[-1.0, 0.0], [5.0, 5.0], [1.0, 0.0], [5.0, 5.0]], np.float32)
    labels, best, second = O.assign(Y, C)
    assert labels.tolist() == [0, 2, 1]
    assert best[0] == 1.0 and second[0] == 1.0      # exact tie is reported as gap 0
    assert best[2] == 0.0 and second[2] == 0.0
    assert O.near_tie_mask(best, second).tolist() == [True, False, True]


def test_assign_permuting_centroids_permutes_labels():
    r = rng(11)
    Y = r.normal(size=(200, 16)).astype(np.float32)
    C = r.normal(size=(7, 16)).astype(np.float32)
    perm = r.permutation(7)
    l0, b0, s0 = O.assign(Y, C)
    l1, b1, s1 = O.assign(Y, C[perm])
    assert np.array_equal(perm[l1], l0)
    np.testing.assert_array_equal(b0, b1)
    np.testing.assert_array_equal(s0, s1)


def test_assign_single_cluster():
    Y = rng(12).normal(size=(5, 4)).astype(np.float32)
    labels, best, second = O.assign(Y, Y[:1])
    assert labels.tolist() == [0] * 5 and best[0] == 0.0 and np.all(np.isinf(second))


# --------------------------------------------------------------------------
# Lloyd iterations
# --------------------------------------------------------------------------

def _blobs(seed, n, d, k, spread=0.3):
    r = rng(seed)
    centers = r.normal(size=(k, d)) * 4
    comp = r.integers(0, k, size=n)
    return (centers[comp] + spread * r.normal(size=(n, d))).astype(np.float32), comp, centers


@pytest.mark.parametrize("seed,n,d,k", [(0, 500, 8, 5), (1, 300, 20, 9), (2, 64, 3, 16)])
def test_lloyd_objective_non_increasing(seed, n, d, k):
    Y = rng(seed).normal(size=(n, d)).astype(np.float32)
    res = O.fit(Y, Y, k, 15)
    J = res.J
    assert np.all(J[1:] <= J[:-1] * (1 + 1e-12) + 1e-12)
    assert J[0] > J[-1]


def test_lloyd_reaches_fixed_point():
    Y, _, _ = _blobs(3, 400, 6, 4)
    a = O.fit(Y, Y, 4, 40)
    b = O.fit(Y, Y, 4, 41)
    assert a.J[-1] == a.J[-2]
    assert np.array_equal(a.labels, b.labels)
    np.testing.assert_array_equal(a.centroids, b.centroids)
    # at a fixed point every centroid is the mean of its own rows
    for k in range(4):
        np.testing.assert_allclose(a.centroids[k], Y[a.labels == k].astype(np.float64).mean(0),
                                   rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("seed", range(4))
def test_lloyd_never_beats_global_optimum(seed):
    """N = 8, K = 2: enumerate all 2**8 partitions; the best partition's
    within-cluster sum of squares bounds Lloyd's final objective from below,
    and Lloyd's objective equals the within-cluster sum of squares of its own
    partition once converged."""
    r = rng(100 + seed)
    Y = r.normal(size=(8, 2)).astype(np.float32)
    Yd = Y.astype(np.float64)

    def wcss(lab):
        tot = 0.0
        for k in (0, 1):
            pts = Yd[np.array(lab) == k]
            if len(pts):
                tot += ((pts - pts.mean(0)) ** 2).sum()
        return tot

    opt = min(wcss(lab) for lab in itertools.product((0, 1), repeat=8))
    res = O.fit(Y, Y, 2, 30)
    assert res.J[-1] >= opt * (1 - 1e-6)
    np.testing.assert_allclose(res.J[-1], wcss(res.labels), rtol=1e-6)


def test_lloyd_k_equals_n_distinct_rows():
    Y = rng(5).normal(size=(12, 5)).astype(np.float32)
    res = O.fit(Y, Y, 12, 3)
    assert np.all(res.J == 0.0)
    np.testing.assert_array_equal(res.centroids, Y)
    assert res.labels.tolist() == list(range(12))


def test_lloyd_recovers_planted_partition_in_one_round():
    k, d = 6, 10
    Y, comp, centers = _blobs(6, 600, d, k, spread=0.05)
    # put one row of each component first so that the first-K-rows init has one seed per component
    first = [int(np.flatnonzero(comp == c)[0]) for c in range(k)]
    rest = [i for i in range(len(Y)) if i not in first]
    order = np.array(first + rest)
    Y, comp = Y[order], comp[order]
    res = O.fit(Y, Y, k, 1)
    assert np.array_equal(res.labels, comp)          # seeds were placed in component order
    for c in range(k):
        np.testing.assert_allclose(res.centroids[c], Y[comp == c].astype(np.float64).mean(0),
                                   rtol=1e-6, atol=1e-6)


def test_lloyd_explicit_init_equals_first_rows_default():
    Y = rng(7).normal(size=(100, 4)).astype(np.float32)
    a = O.fit(Y, Y, 5, 7)
    b = O.fit(Y, Y, 5, 7, init=Y[:5].copy())
    np.testing.assert_array_equal(a.centroids, b.centroids)
    assert np.array_equal(a.labels, b.labels)


def test_lloyd_zero_iterations_is_init_plus_final_assignment():
    Y = rng(8).normal(size=(50, 3)).astype(np.float32)
    res = O.fit(Y, Y, 4, 0)
    np.testing.assert_array_equal(res.centroids, Y[:4])
    lab, _, _ = O.assign(Y, Y[:4])
    assert np.array_equal(res.labels, lab)
    assert res.J.shape == (1,)


@pytest.mark.parametrize("seed,iters", [(0, 1), (1, 5), (2, 25)])
def test_lloyd_matches_sklearn_from_same_init(seed, iters):
    """Library cross-check in a special case: scikit-learn's Lloyd k-means run
    from the same explicit init for the same number of rounds (tol = 0),
    on data where no cluster empties and no near-tie occurs."""
    from sklearn.cluster import KMeans
    Y, _, _ = _blobs(20 + seed, 800, 12, 6, spread=1.5)
    res = O.fit(Y, Y, 6, iters, near_rel=1e-4)
    assert res.near.sum() == 0 and res.counts.min() > 0
    import warnings
    with warnings.catch_warnings():
        warnings.simplefilter("ignore")
        km = KMeans(n_clusters=6, init=Y[:6].astype(np.float64), n_init=1, max_iter=iters,
                    tol=0.0, algorithm="lloyd").fit(Y.astype(np.float64))
    np.testing.assert_allclose(res.centroids, km.cluster_centers_, rtol=1e-5, atol=1e-6)
    assert np.array_equal(res.labels, km.labels_)
    np.testing.assert_allclose(res.J[-1], km.inertia_, rtol=1e-7)  # fp32-rounded centroids


def test_update_centroids_empty_cluster_keeps_previous():
    Y = rng(9).normal(size=(10, 3)).astype(np.float32)
    labels = np.array([0, 0, 2, 2, 2, 0, 0, 2, 2, 0], np.int32)
    prev = rng(10).normal(size=(3, 3)).astype(np.float32)
    C, counts = O.update_centroids(Y, labels, prev)
    assert counts.tolist() == [5, 0, 5]
    np.testing.assert_array_equal(C[1], prev[1])
    np.testing.assert_allclose(C[0], Y[labels == 0].astype(np.float64).mean(0), rtol=1e-6)
    np.testing.assert_allclose(C[2], Y[labels == 2].astype(np.float64).mean(0), rtol=1e-6)


def test_empty_cluster_during_fit():
    """Duplicate init rows: the higher-index duplicate never wins a tie, so it is
    empty in the first assignment.  With iters = 0 it stays empty and gets
    gamma = 1, beta = 0 (Algorithm 1); after one round it has kept its centroid."""
    Y = rng(11).normal(size=(40, 4)).astype(np.float32)
    Y[1] = Y[0]
    F = rng(12).normal(size=(40, 4)).astype(np.float32)
    res = O.fit(Y, F, 3, 0)
    assert res.counts[1] == 0 and res.counts.sum() == 40
    assert np.all(res.gamma[1] == 1.0) and np.all(res.beta[1] == 0.0)
    assert not np.all(res.gamma[0] == 1.0)
    res1 = O.fit(Y, F, 3, 1)
    np.testing.assert_array_equal(res1.centroids[1], Y[1])
    assert not np.array_equal(res1.centroids[0], Y[0])
    res5 = O.fit(Y, F, 3, 5)
    assert np.all(res5.J[1:] <= res5.J[:-1] * (1 + 1e-12))


# --------------------------------------------------------------------------
# gamma / beta
# --------------------------------------------------------------------------

def test_gamma_beta_are_the_least_squares_solution():
    """Per cluster and column, (gamma, beta) solve min sum (f - gamma q - beta)^2:
    compared with numpy's least-squares solver on the design matrix [q, 1]."""
    r = rng(30)
    N, D, K = 60, 5, 3
    Q = r.normal(size=(N, D)).astype(np.float32)
    F = (0.7 * Q + r.normal(size=(N, D)) * 0.3 + 1.0).astype(np.float32)
    labels = r.integers(0, K, size=N).astype(np.int32)
    gamma, beta = O.solve_gamma_beta(Q, F, labels, K)
    for k in range(K):
        m = labels == k
        for j in range(D):
            A = np.stack([Q[m, j].astype(np.float64), np.ones(m.sum())], 1)
            sol, *_ = np.linalg.lstsq(A, F[m, j].astype(np.float64), rcond=None)
            np.testing.assert_allclose([gamma[k, j], beta[k, j]], sol, rtol=2e-6, atol=1e-7)


def test_k1_reduces_to_plain_affine():
    """One cluster = one parameter set for all outputs: labels all 0, centroid =
    column means, gamma/beta = a global per-column line fit."""
    r = rng(31)
    Q = r.normal(size=(200, 6)).astype(np.float32) * 2 + 1
    F = (Q * r.normal(size=6) + r.normal(size=(200, 6))).astype(np.float32)
    res = O.fit(Q, F, 1, 4)
    assert not res.labels.any()
    np.testing.assert_allclose(res.centroids[0], Q.astype(np.float64).mean(0), rtol=1e-6)
    for j in range(6):
        slope, icpt = np.polyfit(Q[:, j].astype(np.float64), F[:, j].astype(np.float64), 1)
        np.testing.assert_allclose([res.gamma[0, j], res.beta[0, j]], [slope, icpt],
                                   rtol=2e-6, atol=1e-7)
    out, lab, _, _ = O.apply(Q, res.centroids, res.gamma, res.beta)
    np.testing.assert_allclose(out, Q * res.gamma[0] + res.beta[0], rtol=1e-6, atol=1e-6)


def test_identical_inputs_give_identity_parameters():
    Q = rng(32).normal(size=(300, 7)).astype(np.float32)
    res = O.fit(Q, Q, 4, 6)
    assert res.counts.min() > 1
    np.testing.assert_allclose(res.gamma, 1.0, rtol=0, atol=1e-6)
    np.testing.assert_allclose(res.beta, 0.0, rtol=0, atol=1e-6)
    out, *_ = O.apply(Q, res.centroids, res.gamma, res.beta)
    np.testing.assert_allclose(out, Q, rtol=1e-6, atol=1e-6)


def test_affine_recovery_any_k():
    """Yfp = a*Yq + b column-wise  =>  gamma_k = a, beta_k = b in every cluster."""
    r = rng(33)
    Q = r.normal(size=(400, 5)).astype(np.float64)
    a = np.array([2.0, -0.5, 0.25, 1.0, -3.0])
    b = np.array([0.5, 1.0, -2.0, 0.0, 4.0])
    Q32 = Q.astype(np.float32)
    F32 = (Q32.astype(np.float64) * a + b).astype(np.float32)
    res = O.fit(Q32, F32, 5, 8)
    assert res.counts.min() > 2
    np.testing.assert_allclose(res.gamma, np.broadcast_to(a, (5, 5)), rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(res.beta, np.broadcast_to(b, (5, 5)), rtol=1e-5, atol=2e-6)


def test_constant_column_and_singleton_hit_the_variance_floor():
    """Var = 0 is floored to 1e-8 and cov is exactly 0, so gamma = 0 and
    beta = mean(F) (Algorithm 1's max(Var, 1e-8))."""
    Q = np.array([[1.0, 3.0], [2.0, 3.0], [4.0, 3.0], [9.0, 9.0]], np.float32)
    F = np.array([[1.5, 7.0], [2.5, 8.0], [4.5, 9.0], [5.0, 6.0]], np.float32)
    labels = np.array([0, 0, 0, 1], np.int32)
    gamma, beta = O.solve_gamma_beta(Q, F, labels, 2)
    assert gamma[0, 1] == 0.0 and beta[0, 1] == 8.0          # constant column
    np.testing.assert_allclose([gamma[0, 0], beta[0, 0]], [1.0, 0.5], rtol=1e-6)
    assert gamma[1].tolist() == [0.0, 0.0] and beta[1].tolist() == [5.0, 6.0]  # singleton


def test_variance_floor_value():
    """A column whose variance is below 1e-8 divides by exactly 1e-8."""
    q = np.array([1.0, 1.0 + 2.0 ** -20], np.float32)       # var = 2^-42 ~ 2.3e-13
    f = np.array([0.0, 1.0], np.float32)
    gamma, beta = O.solve_gamma_beta(q[:, None], f[:, None], np.zeros(2, np.int32), 1)
    dq = 2.0 ** -21
    cov = dq * 0.5                                          # mean of (+-dq)(+-0.5)
    np.testing.assert_allclose(gamma[0, 0], cov / 1e-8, rtol=1e-6)
    np.testing.assert_allclose(beta[0, 0], 0.5 - (cov / 1e-8) * (1.0 + dq), rtol=1e-6)


def test_population_normalisation_not_sample():
    """cov and var use the same 1/n, so two points give the exact line through them."""
    q = np.array([[1.0], [3.0]], np.float32)
    f = np.array([[2.0], [8.0]], np.float32)
    gamma, beta = O.solve_gamma_beta(q, f, np.zeros(2, np.int32), 1)
    assert gamma[0, 0] == 3.0 and beta[0, 0] == -1.0


def test_gamma_beta_residual_is_a_minimum():
    r = rng(34)
    Q = r.normal(size=(50, 3)).astype(np.float32)
    F = r.normal(size=(50, 3)).astype(np.float32)
    labels = (np.arange(50) % 2).astype(np.int32)
    gamma, beta = O.solve_gamma_beta(Q, F, labels, 2)

    def resid(g, b):
        return ((F - (g[labels] * Q + b[labels])) ** 2).astype(np.float64).sum()

    base = resid(gamma, beta)
    for dg, db in [(1e-2, 0), (-1e-2, 0), (0, 1e-2), (0, -1e-2)]:
        assert resid(gamma + dg, beta + db) > base


# --------------------------------------------------------------------------
# inference
# --------------------------------------------------------------------------

def test_apply_identity_parameters_are_bit_exact():
    Y = rng(40).normal(size=(100, 9)).astype(np.float32)
    C = Y[:4].copy()
    out, *_ = O.apply(Y, C, np.ones((4, 9), np.float32), np.zeros((4, 9), np.float32))
    assert np.array_equal(out, Y)


def test_apply_is_a_single_rounding_of_the_exact_value():
    r = rng(41)
    Y = r.normal(size=(6, 4)).astype(np.float32)
    C = Y[:2].copy()
    g = r.normal(size=(2, 4)).astype(np.float32)
    b = r.normal(size=(2, 4)).astype(np.float32)
    out, labels, _, _ = O.apply(Y, C, g, b)
    for i in range(6):
        for j in range(4):
            exact = Fraction(float(Y[i, j])) * Fraction(float(g[labels[i], j])) \
                + Fraction(float(b[labels[i], j]))
            # nearest float32 to the exact rational value
            cand = np.float32(float(exact))
            assert out[i, j] == cand


def test_apply_uses_the_assigned_cluster_parameters():
    Y = np.array([[0.0, 0.0], [10.0, 10.0]], np.float32)
    C = np.array([[0.0, 1.0], [9.0, 9.0]], np.float32)
    g = np.array([[2.0, 2.0], [3.0, 3.0]], np.float32)
    b = np.array([[1.0, 1.0], [-1.0, -1.0]], np.float32)
    out, labels, _, _ = O.apply(Y, C, g, b)
    assert labels.tolist() == [0, 1]
    assert out.tolist() == [[1.0, 1.0], [29.0, 29.0]]


def test_alpha_blend_endpoints_and_both_algebraic_forms():
    """alpha = 0 leaves the LQ outputs, alpha = 1 is the pure affine correction,
    and q + alpha(affine - q) equals (1 - alpha) q + alpha * affine."""
    r = rng(42)
    Y = r.normal(size=(50, 5)).astype(np.float32)
    C = Y[:3].copy()
    g = r.normal(size=(3, 5)).astype(np.float32)
    b = r.normal(size=(3, 5)).astype(np.float32)
    out0, lab, _, _ = O.apply(Y, C, g, b, alpha=0.0)
    out1, _, _, _ = O.apply(Y, C, g, b, alpha=1.0)
    outh, _, _, _ = O.apply(Y, C, g, b, alpha=0.4)
    assert np.array_equal(out0, Y)
    aff = Y.astype(np.float64) * g[lab] + b[lab]
    np.testing.assert_allclose(out1, aff, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(outh, 0.6 * Y.astype(np.float64) + 0.4 * aff, rtol=1e-6, atol=1e-6)
    np.testing.assert_array_equal(O.affine_with_labels(Y, lab, g, b, 0.4), outh)


def test_fit_labels_equal_apply_labels_on_the_fit_rows():
    Y = rng(43).normal(size=(300, 6)).astype(np.float32)
    F = rng(44).normal(size=(300, 6)).astype(np.float32)
    res = O.fit(Y, F, 7, 3)
    _, lab, _, _ = O.apply(Y, res.centroids, res.gamma, res.beta)
    assert np.array_equal(lab, res.labels)
    g2, b2 = O.solve_gamma_beta(Y, F, res.labels, 7)
    np.testing.assert_array_equal(g2, res.gamma)
    np.testing.assert_array_equal(b2, res.beta)


def test_cat_reduces_fit_error_versus_plain_affine():
    """With cluster-dependent distortion, per-cluster parameters fit the FP
    outputs better than one global parameter set (the paper's motivation)."""
    r = rng(45)
    k, d = 4, 6
    Q, comp, _ = _blobs(46, 800, d, k, spread=0.5)
    a = r.normal(size=(k, d)) + 1.0
    b = r.normal(size=(k, d))
    F = (Q * a[comp] + b[comp]).astype(np.float32)
    cat = O.fit(Q, F, k, 10)
    plain = O.fit(Q, F, 1, 1)
    e_cat = ((O.apply(Q, cat.centroids, cat.gamma, cat.beta)[0] - F) ** 2).mean()
    e_plain = ((O.apply(Q, plain.centroids, plain.gamma, plain.beta)[0] - F) ** 2).mean()
    assert e_cat < 0.05 * e_plain


def test_parameter_count_matches_the_papers_worked_example():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "param_overhead.txt"))
            if l.strip() and not l.startswith("#")]
    k, d, base, added, total = map(int, rows[0])
    Y = rng(47).normal(size=(k, d)).astype(np.float32)
    res = O.fit(Y, Y, k, 0)
    # k x d centroids and k x d values per affine coefficient array
    assert res.centroids.size == k * d and res.gamma.size == k * d and res.beta.size == k * d
    assert res.centroids.size + res.gamma.size == added and base + added == total


def test_fit_rejects_bad_shapes():
    Y = np.zeros((3, 2), np.float32)
    with pytest.raises(ValueError):
        O.fit(Y, Y, 4, 1)
    with pytest.raises(ValueError):
        O.fit(Y, Y, 0, 1)


def test_bf16_rounding_ties_to_even_and_matches_torch():
    import torch
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: the tie goes to the even mantissa (1); 1 + 3 * 2^-8 goes up
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, -1.0 - 2.0 ** -8, 0.0,
                  3.0e38, 1e-40, np.inf], np.float32)
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, -1.0, 0.0, 3.0e38, 1e-40, np.inf], np.float32)
    got = O.to_bf16(x)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.0 + 2.0 ** -7)
    assert got[3] == np.float32(1.0 + 2.0 ** -6) and got[4] == -1.0 and got[5] == 0.0 and np.isinf(got[8])
    r = np.random.default_rng(0).normal(size=100000).astype(np.float32) * np.float32(1e3)
    ref = torch.from_numpy(r).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(O.to_bf16(r), ref)
    assert (np.abs(O.to_bf16(r) - r) <= np.abs(r) * 2.0 ** -8).all()      # within half a bf16 ulp
