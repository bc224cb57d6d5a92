"""CUDA library vs CPU oracle, element by element, on the same seeded inputs.

Everything here goes through the C ABI (binding -> libcat.so).  Protocol:
  apply      : oracle parameters in, labels and corrected outputs compared
  one step   : both sides start from the oracle's centroids of round t; labels compared,
               the centroid update compared label-conditioned (oracle recomputes from the
               GPU's labels)
  final pass : gamma/beta compared label-conditioned; labels_out is the argmin against
               centroids_out
  end to end : direct comparison of all outputs when the oracle's trajectory has no row inside
               the near-tie band (1e-6 relative); when it has, direct comparison of the fit cut
               short before the first such assignment, and for the full fit the objective within
               1e-4 plus the label-conditioned checks above
"""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2509_26277_b200 import binding as B
from paper_2509_26277_b200 import workloads as W
from tests.parity import NEAR_REL, close, labels_match

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["fp32", "tensor"], autouse=True)
def contraction_path(request):
    """Every case runs twice: distance contraction forced onto the fp32 pipes, and forced onto
    the tensor cores wherever that path applies (D % 4 == 0, K <= 256)."""
    old = B.cat_get_tensor_core_min_k()
    B.cat_set_tensor_core_min_k(1 << 30 if request.param == "fp32" else 1)
    yield request.param
    B.cat_set_tensor_core_min_k(old)


def dev(a):
    return torch.as_tensor(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


# workloads the oracle finishes in seconds: configs 0-3 (config 1/2 apply sets cut to 8192
# rows, config 3 cut to 1/8 of its rows here; full sizes are in test_gpu_full_size.py) and
# a scaled config 4.
CASES = {
    "cfg0": dict(config=0, rows_scale=1.0),
    "cfg1": dict(config=1, rows_scale=1.0, apply_rows=8192),
    "cfg2": dict(config=2, rows_scale=1.0, apply_rows=8192),
    "cfg3": dict(config=3, rows_scale=0.125),
    "cfg4s": dict(config=4, rows_scale=1.0 / 256),
}
_cache = {}


def workload(name):
    if name not in _cache:
        c = CASES[name]
        w = W.make(c["config"], device="cpu", rows_scale=c["rows_scale"])
        if "apply_rows" in c:
            w.Yq_apply = w.Yq_apply[:c["apply_rows"]].contiguous()
        ora = O.fit(w.Yq_fit.numpy(), w.Yfp_fit.numpy(), w.K, w.iters, near_rel=NEAR_REL)
        _cache[name] = (w, ora)
    return _cache[name]


@pytest.mark.parametrize("name", list(CASES))
def test_apply_matches_oracle(name):
    w, ora = workload(name)
    Yq = w.Yq_apply.numpy()
    want, lab, best, second = O.apply(Yq, ora.centroids, ora.gamma, ora.beta)
    out, glab = B.cat_apply(dev(Yq), dev(ora.centroids), dev(ora.gamma), dev(ora.beta), want_labels=True)
    torch.cuda.synchronize()
    glab = host(glab)
    n_near, n_diff = labels_match(glab, lab, best, second, f"{name} apply labels")
    # rows whose label differs inside the near-tie band are checked against the GPU's own label
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, glab, ora.gamma, ora.beta)
    err = close(host(out), want2, f"{name} apply outputs")
    print(f"{name}: apply rows {len(Yq)} near-tie rows {n_near} (label differs on {n_diff}) max|err| {err:.2e}")


@pytest.mark.parametrize("name", list(CASES))
def test_one_lloyd_step_teacher_forced(name):
    w, _ = workload(name)
    Yq = w.Yq_fit.numpy()
    dYq = dev(Yq)
    for t in sorted({0, w.iters // 2, w.iters - 1}):
        C_t = O.fit(Yq, Yq, w.K, t).centroids if t else Yq[:w.K].copy()
        lab, best, second = O.assign(Yq, C_t)
        glab = B.cat_assign(dYq, dev(C_t))
        n_near, n_diff = labels_match(host(glab), lab, best, second, f"{name} round {t} labels")
        sums, counts = B.cat_cluster_sums(dYq, glab, w.K)
        C_gpu = dev(C_t)
        B.cat_centroids_from_sums(sums, counts, C_gpu)
        C_want, n_want = O.update_centroids(Yq, host(glab), C_t)
        assert np.array_equal(host(counts), n_want)
        close(host(C_gpu), C_want, f"{name} round {t} centroid update")
        print(f"{name}: round {t} near-tie rows {n_near} (differs on {n_diff})")


@pytest.mark.parametrize("name", list(CASES))
def test_fit_final_pass_and_end_to_end(name):
    w, ora = workload(name)
    Yq, Yfp = w.Yq_fit.numpy(), w.Yfp_fit.numpy()
    C, G, Bt, labels, diag = B.cat_fit(dev(Yq), dev(Yfp), w.K, w.iters, want_diag=True)
    torch.cuda.synchronize()
    C, G, Bt, labels = host(C), host(G), host(Bt), host(labels)
    assert diag["device_status"] == 0
    # labels_out is the argmin against centroids_out
    lab, best, second = O.assign(Yq, C)
    n_near, n_diff = labels_match(labels, lab, best, second, f"{name} fit labels_out")
    # gamma/beta, label-conditioned
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, labels, w.K)
    close(G, g_want, f"{name} gamma (label-conditioned)")
    close(Bt, b_want, f"{name} beta (label-conditioned)")
    assert diag["empty_clusters_final"] == int((np.bincount(labels, minlength=w.K) == 0).sum())
    # trajectory
    J_gpu = O.assign(Yq, C)[1].sum()
    ratio = J_gpu / ora.J[-1]
    agree = float((labels == ora.labels).mean())
    assert abs(ratio - 1) < 1e-4, (ratio, agree)
    with_near = np.flatnonzero(ora.near)          # assignments of the oracle's run that saw a near-tie row
    strict_rounds = w.iters if len(with_near) == 0 else int(with_near[0]) - 1
    if strict_rounds == w.iters:
        prefix, got = ora, (C, G, Bt, labels)
    elif strict_rounds >= 0:
        # a fit of this many rounds makes only clear-cut assignments: it must equal the oracle's outright
        prefix = O.fit(Yq, Yfp, w.K, strict_rounds, near_rel=NEAR_REL)
        assert int(prefix.near.sum()) == 0
        got = tuple(host(x) for x in B.cat_fit(dev(Yq), dev(Yfp), w.K, strict_rounds))
    else:
        prefix = None
    if prefix is not None:
        assert np.array_equal(got[3], prefix.labels), f"{name}: labels differ with no near-tie on the trajectory"
        close(got[0], prefix.centroids, f"{name} centroids end to end ({strict_rounds} rounds)")
        close(got[1], prefix.gamma, f"{name} gamma end to end ({strict_rounds} rounds)")
        close(got[2], prefix.beta, f"{name} beta end to end ({strict_rounds} rounds)")
    print(f"{name}: oracle near-tie rows per assignment {ora.near.tolist()} -> strict end-to-end over {strict_rounds} of "
          f"{w.iters} rounds; full fit: label agreement {agree:.6f}, J_gpu/J_oracle {ratio:.8f}, "
          f"rows through the exact pass {diag['refined_rows_total']}")


def test_fit_is_reproducible_run_to_run():
    w, _ = workload("cfg3")
    a = B.cat_fit(dev(w.Yq_fit.numpy()), dev(w.Yfp_fit.numpy()), w.K, 5)
    b = B.cat_fit(dev(w.Yq_fit.numpy()), dev(w.Yfp_fit.numpy()), w.K, 5)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


# ---------------------------------------------------------------- edge cases

def _rand(seed, n, d):
    return np.random.default_rng(seed).normal(size=(n, d)).astype(np.float32)


@pytest.mark.parametrize("n,d,k", [(1, 4, 1), (5, 1, 2), (127, 3, 3), (129, 7, 5), (300, 10, 9),
                                   (257, 1000, 17), (1000, 64, 65), (513, 36, 130), (64, 8, 64),
                                   (2000, 20, 1), (900, 1024, 256), (700, 12, 512), (600, 1540, 48), (300, 1100, 6),
                                   # N not a multiple of the rows a warp shares when a row takes fewer than 32 lanes
                                   (1001, 64, 65), (67, 8, 64), (515, 32, 40), (333, 120, 33)])
def test_ragged_shapes_apply_and_fit(n, d, k):
    Yq = _rand(n * 7 + d, n, d)
    Yfp = (Yq * 1.1 + 0.1 * _rand(n + d + 1, n, d)).astype(np.float32)
    C = _rand(k, k, d)
    g, b = _rand(k + 1, k, d), _rand(k + 2, k, d)
    want, lab, best, second = O.apply(Yq, C, g, b)
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(g), dev(b), want_labels=True)
    _, n_diff = labels_match(host(glab), lab, best, second, "labels")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), g, b)
    close(host(out), want2, "outputs")
    if n >= k:
        Cg, Gg, Bg, lg = B.cat_fit(dev(Yq), dev(Yfp), k, 3)
        lab2, best2, second2 = O.assign(Yq, host(Cg))
        labels_match(host(lg), lab2, best2, second2, "fit labels")
        g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(lg), k)
        close(host(Gg), g_want, "gamma")
        close(host(Bg), b_want, "beta")
        ora = O.fit(Yq, Yfp, k, 3, near_rel=NEAR_REL)
        if ora.near.sum() == 0:
            close(host(Cg), ora.centroids, "centroids")
            assert np.array_equal(host(lg), ora.labels)


@pytest.mark.parametrize("n,d,k,scale", [(600, 2048, 40, 1.0),      # rows longer than one streaming step
                                         (300, 120, 33, 1.0),       # short rows, 30 float4 (not a power of two)
                                         (700, 1032, 64, 1.0),      # last fp16 slab partly outside the matrix
                                         (520, 1028, 48, 1.0),      # D % 8 != 0: the fit stays on TF32 operands
                                         (3000, 256, 128, 1.0),
                                         (1500, 512, 256, 3.0e4),   # magnitudes far above the fp16 range
                                         (1500, 512, 256, 2.0e-7)])  # ... and far below it
def test_tensor_paths_shapes_and_scales(n, d, k, scale):
    """Shapes and magnitudes that steer the tensor-core kernels through their variants (fp16 copy of
    the rows with its power-of-two scale, TF32, short and long rows).  Tolerances scale with the data."""
    Yq = (_rand(n + d, n, d) * scale).astype(np.float32)
    Yfp = (Yq * 0.9 + 0.05 * scale * _rand(n + d + 1, n, d)).astype(np.float32)
    Cg, Gg, Bg, lg = B.cat_fit(dev(Yq), dev(Yfp), k, 4)
    lab, best, second = O.assign(Yq, host(Cg))
    labels_match(host(lg), lab, best, second, "fit labels")
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, host(lg), k)
    close(host(Gg), g_want, "gamma")
    close(host(Bg) / scale, b_want / scale, "beta")
    ora = O.fit(Yq, Yfp, k, 4, near_rel=1e-5)
    if ora.near.sum() == 0:
        assert np.array_equal(host(lg), ora.labels)
        close(host(Cg) / scale, ora.centroids / scale, "centroids")
    want, lab, best, second = O.apply(Yq, host(Cg), host(Gg), host(Bg))
    out, glab = B.cat_apply(dev(Yq), Cg, Gg, Bg, want_labels=True)
    _, n_diff = labels_match(host(glab), lab, best, second, "apply labels")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), host(Gg), host(Bg))
    close(host(out) / scale, want2 / scale, "outputs")


@pytest.mark.parametrize("d,k", [(64, 40), (1000, 16), (1024, 256), (4096, 64), (16384, 32)])
@pytest.mark.parametrize("scale", [1.0, 3.0e4, 1.0e-7])
def test_fast_scores_stay_within_their_error_bound(d, k, scale, contraction_path):
    """The label decision trusts a fast score only as far as its error bound e.  cat_assign_scores hands out
    the two smallest fast scores of every row and the e that was used; both must lie within e of the two
    smallest exact scores ||c||^2 - 2 y.c (fp64 here), whatever the operands: fp32 FMA chains, TF32 or
    fp16 tensor-core products.  Rows: near centroids, halfway between the origin and a centroid (where
    the two terms of a score cancel), exact copies of centroids, and plain noise."""
    rng = np.random.default_rng(d * 7 + k)
    n = 640
    cen = rng.normal(size=(k, d))
    pick = rng.integers(0, k, size=n)
    Y = np.empty((n, d))
    Y[:160] = cen[pick[:160]] + 0.3 * rng.normal(size=(160, d))
    Y[160:320] = 0.5 * cen[pick[160:320]] + 0.01 * rng.normal(size=(160, d))
    Y[320:480] = cen[pick[320:480]]
    Y[480:] = rng.normal(size=(160, d)) * rng.uniform(0.1, 4.0, size=(160, 1))
    Yq = (Y * scale).astype(np.float32)
    C = (cen * scale * 0.999).astype(np.float32)      # (stays below the largest magnitude of Yq)
    T = (C.astype(np.float64) ** 2).sum(1)[None, :] - 2.0 * Yq.astype(np.float64) @ C.astype(np.float64).T
    T.sort(axis=1)
    lab, best, second = O.assign(Yq, C)
    modes = [False, True] if (contraction_path == "tensor" and d % 8 == 0) else [False]
    for fp16 in modes:
        labels, rec = B.cat_assign_scores(dev(Yq), dev(C), fp16_operands=fp16)
        labels_match(host(labels), lab, best, second, "labels")
        e = host(rec["bound"]).astype(np.float64)
        fb, fs = host(rec["best"]).astype(np.float64), host(rec["second"]).astype(np.float64)
        assert np.isfinite(e).all() and (e > 0).all()
        slack = e * (1 + 1e-6)
        worst = max(float((np.abs(fb - T[:, 0]) / e).max()), float((np.abs(fs - T[:, 1]) / e).max()))
        assert (np.abs(fb - T[:, 0]) <= slack).all(), ("best", fp16, worst)
        assert (np.abs(fs - T[:, 1]) <= slack).all(), ("second", fp16, worst)
        print(f"d={d} k={k} scale={scale:g} {contraction_path}{' fp16' if fp16 else ''}: "
              f"largest |fast - exact| / e = {worst:.3f}")


def test_fit_diagnostics_per_assignment():
    """cat_fit_from's optional record of every assignment: objective, rows that went to the exact
    pass, rows inside the 1e-6 near-tie band -- against the oracle's J_t and near_t."""
    w, ora = workload("cfg1")
    Yq, Yfp = w.Yq_fit.numpy(), w.Yfp_fit.numpy()
    C, G, Bt, labels, diag = B.cat_fit(dev(Yq), dev(Yfp), w.K, w.iters, want_diag=True)
    assert diag["assignments_recorded"] == w.iters + 1
    if np.array_equal(host(labels), ora.labels):
        np.testing.assert_allclose(diag["objective"], ora.J, rtol=1e-10)
        assert diag["near_tie_rows"] == ora.near.tolist()
    J = np.array(diag["objective"])
    assert (np.diff(J) <= 1e-9 * J[:-1]).all()                       # Lloyd's objective never rises
    assert all(u >= t for u, t in zip(diag["undecided_rows"], diag["near_tie_rows"]))
    assert diag["refined_rows_total"] == sum(diag["undecided_rows"])
    assert diag["refined_rows_final"] == diag["undecided_rows"][-1]
    # more assignments than slots: the first 63 and the final one are kept
    C2, _, _, l2, d2 = B.cat_fit(dev(Yq[:300]), dev(Yfp[:300]), 4, 70, want_diag=True)
    assert d2["assignments_recorded"] == 64
    assert d2["objective"][-1] == pytest.approx(float(O.assign(Yq[:300], host(C2))[1].sum()), rel=1e-10)


@pytest.mark.parametrize("d,k", [(4096, 32), (4096, 256), (16384, 32), (16384, 256)])
def test_long_rows_against_the_oracle(d, k):
    """Rows of 4096 and 16384 columns (the longest the library takes) on both contraction paths:
    the error bound of the fast scores grows with D, the labels must not."""
    n = 600
    rng = np.random.default_rng(d + k)
    cen = rng.normal(size=(k, d)).astype(np.float32)
    Yq = (cen[rng.integers(0, k, size=n)] + 0.9 * rng.normal(size=(n, d))).astype(np.float32)
    C = (cen + 0.02 * rng.normal(size=cen.shape)).astype(np.float32)
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    ws = B.workspace("apply", n, d, k, "cuda")
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True, ws=ws)
    assert B.cat_workspace_report(ws)["device_status"] == 0
    n_near, n_diff = labels_match(host(glab), lab, best, second, "labels, long rows")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), G, Bt)
    close(host(out), want2, "outputs, long rows")
    glab2 = B.cat_assign(dev(Yq), dev(C))
    labels_match(host(glab2), lab, best, second, "cat_assign labels, long rows")


@pytest.mark.parametrize("cs", [2, 4])
@pytest.mark.parametrize("n,d,k", [(3000, 256, 48), (1111, 1024, 256), (700, 128, 32), (2500, 512, 200),
                                   (129, 128, 33), (40000, 256, 64)])
def test_apply_column_split_matches_oracle(n, d, k, cs):
    """The column-split form of the fused inference kernel (clusters of 2 or 4 CTAs share a 128-row
    tile and sum partial scores through distributed shared memory): ragged N, K that does not fill
    the cluster's centroid ranges, several tiles per cluster.  Same bar as the row-tile form, and
    bit-identical outputs to it."""
    rng = np.random.default_rng(n + d + k)
    cen = (rng.normal(size=(k, d)) * 2).astype(np.float32)
    Yq = (cen[rng.integers(0, k, size=n)] + rng.normal(size=(n, d))).astype(np.float32)
    C = (cen + 0.05 * rng.normal(size=cen.shape)).astype(np.float32)
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    assert B.cat_get_apply_column_split() == 0
    try:
        B.cat_set_apply_column_split(1)
        ref, _ = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True)
        B.cat_set_apply_column_split(cs)
        ws = B.workspace("apply", n, d, k, "cuda")
        out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True, ws=ws)
        rep = B.cat_workspace_report(ws)
    finally:
        B.cat_set_apply_column_split(0)
    assert rep["device_status"] == 0
    _, n_diff = labels_match(host(glab), lab, best, second, "apply labels (column split)")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), G, Bt)
    close(host(out), want2, "outputs (column split)")
    assert torch.equal(out, ref)


def test_apply_column_split_falls_back_where_the_shape_does_not_allow_it():
    """D not a multiple of 32 cs: the request is ignored and the row-tile kernel runs."""
    w, _ = workload("cfg2")
    C, G, Bt, _ = B.cat_fit(dev(w.Yq_fit.numpy()), dev(w.Yfp_fit.numpy()), w.K, 3)
    Y = dev(w.Yq_apply.numpy()[:5000])
    ref = B.cat_apply(Y, C, G, Bt)
    try:
        B.cat_set_apply_column_split(4)
        out = B.cat_apply(Y, C, G, Bt)
    finally:
        B.cat_set_apply_column_split(0)
    assert torch.equal(out, ref)


@pytest.mark.parametrize("d,k", [(256, 32), (1024, 64), (64, 40), (120, 33), (68, 40)])
def test_rows_between_two_centroids_are_decided_like_the_oracle(d, k):
    """Rows placed next to the bisector of two centroids, with relative distance gaps from 1e-6 to
    1e-4: all of them are undecidable for the tensor-core scores, and they straddle the margin
    below which the exact pass leaves its fp32 pre-decision for fp64."""
    rng = np.random.default_rng(d + k)
    C = rng.normal(size=(k, d)).astype(np.float32)
    n = 6000
    a = rng.integers(0, k, size=n)
    b = (a + 1 + rng.integers(0, k - 1, size=n)) % k
    s = (10.0 ** rng.uniform(-6.9, -4.9, size=n)) * rng.choice([-1.0, 1.0], size=n)
    Yq = ((C[a].astype(np.float64) + C[b]) / 2 + s[:, None] * (C[b].astype(np.float64) - C[a])).astype(np.float32)
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply(Yq, C, G, Bt)
    rel = (second - best) / second
    assert (rel < 1e-3).mean() > 0.9 and (rel > 2e-6).mean() > 0.5   # the rows are where they were meant to be
    ws = B.workspace("apply", n, d, k, "cuda")
    out, glab = B.cat_apply(dev(Yq), dev(C), dev(G), dev(Bt), want_labels=True, ws=ws)
    rep = B.cat_workspace_report(ws)
    assert rep["refined_rows_last"] > n // 2      # they did go through the exact pass
    _, n_diff = labels_match(host(glab), lab, best, second, "labels next to a bisector")
    want2 = want if n_diff == 0 else O.affine_with_labels(Yq, host(glab), G, Bt)
    close(host(out), want2, "outputs next to a bisector")
    glab2 = B.cat_assign(dev(Yq), dev(C))
    assert torch.equal(glab2, glab)


def test_fit_fp16_and_tf32_operands_agree():
    """The default start lets cat_fit assign from an fp16 copy of the rows; an explicit start (here the
    same first K rows) keeps TF32 operands.  Labels are decided exactly either way."""
    w, _ = workload("cfg4s")
    Yq, Yfp = dev(w.Yq_fit.numpy()), dev(w.Yfp_fit.numpy())
    a = B.cat_fit(Yq, Yfp, w.K, 6)
    b = B.cat_fit(Yq, Yfp, w.K, 6, init_centroids=Yq[:w.K].clone())
    assert torch.equal(a[3], b[3])
    for x, y in zip(a[:3], b[:3]):
        close(host(x), host(y), "fp16 vs tf32 fit")


def test_exact_ties_resolve_to_lowest_index():
    Yq = np.array([[0, 0, 0, 0], [1, 0, 0, 0], [5, 5, 5, 5]] * 50, np.float32)
    C = np.array([[-1, 0, 0, 0], [5, 5, 5, 5], [1, 0, 0, 0], [5, 5, 5, 5]], np.float32)
    glab = host(B.cat_assign(dev(Yq), dev(C)))
    assert glab.tolist() == [0, 2, 1] * 50


def test_identical_rows_all_ambiguous():
    """Every centroid equal: every row is an exact tie and goes through the fp64 pass."""
    Yq = np.tile(_rand(1, 1, 24), (700, 1))
    Yfp = Yq + 1
    C, G, Bt, labels, diag = B.cat_fit(dev(Yq), dev(Yfp), 6, 2, want_diag=True)
    assert not host(labels).any()
    assert diag["refined_rows_final"] == 700 and diag["empty_clusters_final"] == 5
    ora = O.fit(Yq, Yfp, 6, 2)
    close(host(C), ora.centroids, "centroids")
    close(host(G), ora.gamma, "gamma")
    close(host(Bt), ora.beta, "beta")


def test_empty_cluster_keeps_centroid_and_gets_identity_parameters():
    Yq = _rand(3, 200, 16)
    Yq[1] = Yq[0]
    Yfp = _rand(4, 200, 16)
    for iters in (0, 1, 4):
        C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), 4, iters)
        ora = O.fit(Yq, Yfp, 4, iters, near_rel=1e-5)
        assert np.array_equal(host(labels), ora.labels)
        close(host(C), ora.centroids, "centroids")
        close(host(G), ora.gamma, "gamma")
        close(host(Bt), ora.beta, "beta")
    C0, G0, B0, l0 = B.cat_fit(dev(Yq), dev(Yfp), 4, 0)
    assert torch.all(G0[1] == 1) and torch.all(B0[1] == 0)
    C1 = B.cat_fit(dev(Yq), dev(Yfp), 4, 1)[0]
    assert torch.equal(C1[1], dev(Yq)[1])


def test_k1_is_plain_affine_and_identity_inputs_give_identity_map():
    Yq = _rand(5, 1500, 40) * 3 + 1
    Yfp = (Yq * 0.5 - 2).astype(np.float32)
    C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), 1, 3)
    assert not host(labels).any()
    close(host(C)[0], Yq.astype(np.float64).mean(0), "K=1 centroid")
    close(host(G), np.full((1, 40), 0.5), "K=1 gamma")
    close(host(Bt), np.full((1, 40), -2.0), "K=1 beta", abs_tol=3e-6)
    C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yq), 7, 5)
    close(host(G), np.ones((7, 40)), "gamma for Yq == Yfp")
    close(host(Bt), np.zeros((7, 40)), "beta for Yq == Yfp")
    out = B.cat_apply(dev(Yq), C, torch.ones_like(G), torch.zeros_like(Bt))
    assert torch.equal(out, dev(Yq))          # identity parameters are bit-exact


def test_explicit_init_centroids():
    Yq, Yfp = _rand(6, 400, 12), _rand(7, 400, 12)
    init = _rand(8, 5, 12)
    C, G, Bt, labels = B.cat_fit(dev(Yq), dev(Yfp), 5, 4, init_centroids=dev(init))
    ora = O.fit(Yq, Yfp, 5, 4, init=init, near_rel=1e-5)
    if ora.near.sum() == 0:
        assert np.array_equal(host(labels), ora.labels)
        close(host(C), ora.centroids, "centroids")
        close(host(G), ora.gamma, "gamma")


@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.6, 1.0])
def test_alpha_blend(alpha):
    Yq = _rand(9, 999, 100)
    C, g, b = _rand(10, 12, 100), _rand(11, 12, 100), _rand(12, 12, 100)
    want, lab, best, second = O.apply(Yq, C, g, b, alpha=alpha)
    out, glab = B.cat_apply_blend(dev(Yq), dev(C), dev(g), dev(b), alpha, want_labels=True)
    labels_match(host(glab), lab, best, second, "labels")
    # The library folds the blend into fp32 coefficients g' = 1 + alpha (gamma - 1), b' = alpha beta
    # (formed in fp64, rounded once each) and evaluates fma(g', y, b'): three roundings instead of the
    # oracle's one, i.e. up to 2^-24 (|g' y| + |b'|) + half an ulp of the result.  Where the two terms
    # cancel that exceeds 1e-6 + 1e-5 |result|, so the bound is written out per element.
    gl, bl = g[lab].astype(np.float64), b[lab].astype(np.float64)
    gp, bp = 1 + alpha * (gl - 1), alpha * bl
    slack = 2.0 ** -24 * (np.abs(gp * Yq) + np.abs(bp))
    err = np.abs(host(out).astype(np.float64) - want)
    assert (err <= 1e-6 + 1e-5 * np.abs(want) + slack).all(), float((err - slack).max())
    if alpha == 0.0:
        assert torch.equal(out, dev(Yq))
    if alpha == 1.0:
        assert torch.equal(out, B.cat_apply(dev(Yq), dev(C), dev(g), dev(b)))


@pytest.mark.parametrize("n,d,k", [(3000, 1024, 64), (1111, 1000, 16), (500, 36, 5), (5000, 256, 200), (70, 130, 3)])
def test_apply_with_bf16_output(n, d, k):
    """cat_apply_bf16 on shapes that take the fused 64-row-tile kernel and on shapes that take the
    assignment followed by a second pass: labels as cat_apply, outputs equal to the oracle's bit for bit."""
    rng = np.random.default_rng(n + d + k)
    cen = (rng.normal(size=(k, d)) * 2).astype(np.float32)
    Yq = (cen[rng.integers(0, k, size=n)] + rng.normal(size=(n, d))).astype(np.float32)
    Yq[: n // 4] = (0.5 * (cen[rng.integers(0, k, size=n // 4)] + cen[rng.integers(0, k, size=n // 4)])
                    + 1e-4 * rng.normal(size=(n // 4, d))).astype(np.float32)     # undecided rows: midway between centroids
    G = rng.normal(size=(k, d)).astype(np.float32)
    Bt = rng.normal(size=(k, d)).astype(np.float32)
    want, lab, best, second = O.apply_bf16(Yq, cen, G, Bt)
    out, glab = B.cat_apply_bf16(dev(Yq), dev(cen), dev(G), dev(Bt), want_labels=True)
    assert out.dtype == torch.bfloat16
    _, n_diff = labels_match(host(glab), lab, best, second, "labels (bf16 output)")
    if n_diff:
        want = O.to_bf16(O.affine_with_labels(Yq, host(glab), G, Bt))
    np.testing.assert_array_equal(out.float().cpu().numpy(), want)


def test_step_level_moments_and_solve():
    Yq, Yfp = _rand(13, 3000, 48), _rand(14, 3000, 48)
    labels = np.random.default_rng(15).integers(0, 10, size=3000).astype(np.int32)
    labels[labels == 4] = 5                                  # cluster 4 empty
    dq, df, dl = dev(Yq), dev(Yfp), dev(labels)
    sq, n = B.cat_cluster_sums(dq, dl, 10)
    sf, _ = B.cat_cluster_sums(df, dl, 10)
    assert host(n).tolist() == np.bincount(labels, minlength=10).tolist()
    nn = n.clamp(min=1).double()[:, None]
    var, cov = B.cat_centred_moments(dq, df, dl, sq / nn, sf / nn)
    g, b = B.cat_solve_gamma_beta(sq, sf, var, cov, n)
    g_want, b_want = O.solve_gamma_beta(Yq, Yfp, labels, 10)
    close(host(g), g_want, "gamma")
    close(host(b), b_want, "beta")
    assert torch.all(g[4] == 1) and torch.all(b[4] == 0)


def test_host_buffer_entry_points():
    w, ora = workload("cfg1")
    Yq = w.Yq_apply[:5000].contiguous().pin_memory()
    out = torch.empty_like(Yq).pin_memory()
    labels = torch.empty(5000, dtype=torch.int32).pin_memory()
    B.cat_apply_host(Yq, torch.from_numpy(ora.centroids), torch.from_numpy(ora.gamma),
                     torch.from_numpy(ora.beta), out, labels)
    ref, rlab = B.cat_apply(Yq.cuda(), dev(ora.centroids), dev(ora.gamma), dev(ora.beta), want_labels=True)
    assert torch.equal(out, ref.cpu()) and torch.equal(labels, rlab.cpu())
    K, D = ora.centroids.shape
    C, G, Bt = (torch.empty((K, D)).pin_memory() for _ in range(3))
    lab = torch.empty(w.N_fit, dtype=torch.int32).pin_memory()
    B.cat_fit_host(w.Yq_fit.pin_memory(), w.Yfp_fit.pin_memory(), K, w.iters, C, G, Bt, lab)
    Cd, Gd, Bd, ld = B.cat_fit(w.Yq_fit.cuda(), w.Yfp_fit.cuda(), K, w.iters)
    assert torch.equal(C, Cd.cpu()) and torch.equal(G, Gd.cpu()) and torch.equal(Bt, Bd.cpu())
    assert torch.equal(lab, ld.cpu())


def test_host_apply_streams_many_chunks():
    """More chunks than staging slots: D = 16384 makes a chunk 1024 rows."""
    rng = np.random.default_rng(16)
    Yq = torch.from_numpy(rng.normal(size=(5000, 16384)).astype(np.float32)).pin_memory()
    C = torch.from_numpy(rng.normal(size=(3, 16384)).astype(np.float32))
    g = torch.from_numpy(rng.normal(size=(3, 16384)).astype(np.float32))
    b = torch.from_numpy(rng.normal(size=(3, 16384)).astype(np.float32))
    out = torch.empty_like(Yq).pin_memory()
    B.cat_apply_host(Yq, C, g, b, out)
    ref = B.cat_apply(Yq.cuda(), C.cuda(), g.cuda(), b.cuda())
    assert torch.equal(out, ref.cpu())


def test_non_default_stream_and_missing_labels_out():
    Yq = dev(_rand(17, 4000, 32))
    C = dev(_rand(18, 8, 32))
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        a = B.cat_assign(Yq, C)
        out = B.cat_apply(Yq, C, torch.ones_like(C), torch.zeros_like(C))
    s.synchronize()
    assert torch.equal(a, B.cat_assign(Yq, C)) and torch.equal(out, Yq)


def test_bounded_device_wait_reports_a_timeout_and_leaves_the_context_usable():
    """A device-side wait that can never be satisfied gives up after its limit: the kernel returns,
    the status word says CAT_ERR_DEVICE_TIMEOUT, and the next call on the same workspace works."""
    Yq = dev(_rand(21, 1000, 256))
    C = dev(_rand(22, 40, 256))
    ws = B.workspace("apply", 1000, 256, 40, "cuda")
    B.cat_selftest_wait_timeout(ws, limit_ms=20)
    rep = B.cat_workspace_report(ws)
    assert rep["device_status"] == 6
    labels = B.cat_assign(Yq, C, ws=ws)
    assert B.cat_workspace_report(ws)["device_status"] == 0
    lab, best, second = O.assign(host(Yq), host(C))
    labels_match(host(labels), lab, best, second, "labels after the self-test")
