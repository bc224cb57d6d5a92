"""The persistent single-launch kernels for small shapes (D in {32, 64, 128}, K <= 128), through
the C ABI, against the CPU oracle: inference and the K-Means rounds of a fit, including rows that need the exact pass over two, four and
all K centroids, a ragged last tile, exact ties and run-to-run repeatability."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2509_26277_b200 import binding as B
from tests.parity import close, labels_match

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


@pytest.fixture
def small_mask():
    """Restores the process-wide switch after the test."""
    old = B.cat_get_small_problem_kernels()
    yield
    B.cat_set_small_problem_kernels(old)


def _data(seed, n, d, spread=3.0):
    rng = np.random.default_rng(seed)
    Yfp = rng.normal(size=(n, d)).astype(np.float32)
    Yq = (np.round(Yfp * spread) / spread + 0.01 * rng.normal(size=(n, d))).astype(np.float32)
    return Yq, Yfp


SHAPES = [(1000, 32, 40), (5000, 128, 32), (333, 64, 33), (128, 64, 64), (20001, 64, 64), (3000, 32, 128)]


@pytest.mark.parametrize("n,d,k", SHAPES + [(2000, 128, 128), (4097, 64, 128), (129, 32, 32)])
def test_inference_matches_the_oracle(n, d, k, small_mask):
    Yq, _ = _data(n + d + k, n, d)
    rng = np.random.default_rng(7)
    C = Yq[rng.choice(n, size=k, replace=False)].copy()
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    B.cat_set_small_problem_kernels(1)
    ws = B.workspace("apply", n, d, k, "cuda")
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True, ws=ws)
    _, n_diff = labels_match(host(glab), lab, best, second, "small-kernel inference labels")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), G, Bt)
    close(host(out), want2, "small-kernel inference outputs")
    # the general path gives the same bits
    B.cat_set_small_problem_kernels(0)
    out0, glab0 = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True)
    assert torch.equal(glab0, glab) and torch.equal(out0, out)
    assert B.cat_workspace_report(ws)["device_status"] == 0


@pytest.mark.parametrize("n,d,k", SHAPES)
def test_fit_matches_the_oracle_and_repeats(n, d, k, small_mask):
    Yq, Yfp = _data(2 * n + d + k, n, d)
    iters = 4
    B.cat_set_small_problem_kernels(3)
    C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), k, iters)
    C2, G2, Bt2, labels2 = B.cat_fit(dev(Yq), dev(Yfp), k, iters)
    assert torch.equal(C, C2) and torch.equal(G, G2) and torch.equal(Bt, Bt2) and torch.equal(labels, labels2)
    # final assignment against the oracle, with the library's own centroids
    lab, best, second = O.assign(Yq, host(C))
    labels_match(host(labels), lab, best, second, "small-kernel fit labels")
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(labels), k)
    close(host(G), g_want, "gamma")
    close(host(Bt), b_want, "beta")
    # one more round moves the centroids like the oracle's update
    C1 = B.cat_fit(dev(Yq), dev(Yfp), k, iters + 1, want_labels=False)[0]
    C_want, _ = O.update_centroids(Yq, host(labels), host(C))
    close(host(C1), C_want, "centroid update T -> T+1")
    # the general path agrees: its sums differ by fp64 rounding at most, which can move a centroid by
    # one fp32 step and with it a row that sits on a bisector
    B.cat_set_small_problem_kernels(0)
    C0, G0, Bt0, labels0 = B.cat_fit(dev(Yq), dev(Yfp), k, iters)
    if torch.equal(labels0, labels):
        close(host(C0), host(C), "centroids, general path against the persistent kernel")
    else:
        assert (labels0 != labels).float().mean().item() < 1e-3


def test_whole_fit_against_the_oracle(small_mask):
    """Well separated data: the whole trajectory is the oracle's."""
    rng = np.random.default_rng(5)
    k, d, n = 24, 64, 6000
    means = 6.0 * rng.normal(size=(k, d))
    which = rng.integers(0, k, size=n)
    Yfp = (means[which] + rng.normal(size=(n, d))).astype(np.float32)
    Yq = (Yfp + 0.05 * rng.normal(size=(n, d))).astype(np.float32)
    B.cat_set_small_problem_kernels(3)
    old = B.cat_get_tensor_core_min_k()
    B.cat_set_tensor_core_min_k(1)
    try:
        C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), k, 6)
    finally:
        B.cat_set_tensor_core_min_k(old)
    ora = O.fit(Yq, Yfp, k, 6)
    assert np.array_equal(host(labels), ora.labels)
    close(host(C), ora.centroids, "centroids")
    close(host(G), ora.gamma, "gamma")
    close(host(Bt), ora.beta, "beta")


@pytest.mark.parametrize("d,k", [(64, 40), (32, 96), (128, 32)])
def test_rows_next_to_a_bisector(d, k, small_mask):
    """Every row undecidable for the TF32 scores: the in-kernel exact pass decides like the oracle."""
    rng = np.random.default_rng(d + k)
    C = rng.normal(size=(k, d)).astype(np.float32)
    n = 5000
    a = rng.integers(0, k, size=n)
    b = (a + 1 + rng.integers(0, k - 1, size=n)) % k
    s = (10.0 ** rng.uniform(-6.9, -4.9, size=n)) * rng.choice([-1.0, 1.0], size=n)
    Yq = ((C[a].astype(np.float64) + C[b]) / 2 + s[:, None] * (C[b].astype(np.float64) - C[a])).astype(np.float32)
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    B.cat_set_small_problem_kernels(1)
    ws = B.workspace("apply", n, d, k, "cuda")
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True, ws=ws)
    assert B.cat_workspace_report(ws)["refined_rows_last"] > n // 2
    _, n_diff = labels_match(host(glab), lab, best, second, "labels next to a bisector")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), G, Bt)
    close(host(out), want2, "outputs next to a bisector")


def test_many_candidates_and_exact_ties(small_mask):
    """Centroids in tight bunches (more than four within the error bound of the best: the scan over
    every candidate) and duplicated centroids (exact ties go to the lowest index)."""
    rng = np.random.default_rng(11)
    d, k, n = 64, 64, 4000
    base = rng.normal(size=(8, d)).astype(np.float32)
    C = np.repeat(base, 8, axis=0) + (1e-4 * rng.normal(size=(k, d))).astype(np.float32)
    C[8:16] = C[8]            # eight identical centroids
    C[40] = C[3]              # a duplicate far away in index
    Yq = (base[rng.integers(0, 8, size=n)] + 0.3 * rng.normal(size=(n, d))).astype(np.float32)
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    B.cat_set_small_problem_kernels(1)
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True)
    g = host(glab)
    _, n_diff = labels_match(g, lab, best, second, "bunched centroids")
    assert not np.isin(g, np.arange(9, 16)).any() and not (g == 40).any()   # duplicates: lowest index only
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, g, G, Bt)
    close(host(out), want2, "outputs, bunched centroids")
    # the same through a fit round: sums follow the exact labels
    B.cat_set_small_problem_kernels(3)
    Cf, _, _, labels = B.cat_fit(dev(Yq), dev(Yq), k, 1, init_centroids=dev(C))
    lab1, best1, second1 = O.assign(Yq, host(Cf))
    labels_match(host(labels), lab1, best1, second1, "fit labels, bunched centroids")


def test_fit_without_rounds_is_the_assignment_to_the_first_rows(small_mask):
    """iters = 0: one pass of the persistent kernel that leaves the centroids alone; its sums and
    sizes still feed the closed form."""
    n, d, k = 3000, 64, 48
    Yq, Yfp = _data(99, n, d)
    B.cat_set_small_problem_kernels(3)
    C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), k, 0)
    assert np.array_equal(host(C), Yq[:k])
    lab, best, second = O.assign(Yq, Yq[:k])
    labels_match(host(labels), lab, best, second, "labels of a fit without rounds")
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(labels), k)
    close(host(G), g_want, "gamma")
    close(host(Bt), b_want, "beta")


def test_shapes_outside_the_small_kernels_take_the_general_path(small_mask):
    """K * D above 4096 (fitting) or a D that is not 32, 64 or 128: same results, other kernels."""
    B.cat_set_small_problem_kernels(3)
    for n, d, k in [(2000, 128, 64), (1500, 96, 40)]:
        Yq, Yfp = _data(n + d, n, d)
        C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), k, 3)
        lab, best, second = O.assign(Yq, host(C))
        labels_match(host(labels), lab, best, second, f"labels, D = {d}, K = {k}")
        out = B.cat_apply(dev(Yq), C, G, Bt)
        want = O.affine_with_labels(Yq, host(labels), host(G), host(Bt))
        close(host(out), want, f"outputs, D = {d}, K = {k}")
