"""The seeded input generators: shapes, determinism and the fake-quantisation
structure each configuration is specified to have."""
import numpy as np
import torch

from paper_2509_26277_b200 import workloads as W


def test_specs():
    assert W.spec(0) == dict(name="tiny", seed=0, D=1000, N_fit=1024, N_apply=1024, K=8, iters=20)
    assert W.spec(1)["N_apply"] == 50_000 and W.spec(1)["K"] == 16 and W.spec(1)["iters"] == 30
    assert W.spec(2)["N_fit"] == 4096 and W.spec(2)["K"] == 32
    assert W.spec(3) == dict(name="conv3x3x64_w2a2", seed=3, D=64, N_fit=200_704,
                             N_apply=200_704, K=64, iters=25)
    assert W.spec(4) == dict(name="bandwidth_stress", seed=4, D=1024, N_fit=262_144,
                             N_apply=4_194_304, K=256, iters=25)


def test_config0_shapes_and_determinism():
    a, b = W.make(0), W.make(0)
    assert a.Yq_fit.shape == (1024, 1000) and a.Yfp_fit.shape == (1024, 1000)
    assert a.Yq_apply.shape == (1024, 1000) and a.K == 8 and a.iters == 20
    assert a.Yq_fit.dtype == torch.float32 and a.Yq_fit.is_contiguous()
    assert torch.equal(a.Yq_fit, b.Yq_fit) and torch.equal(a.Yfp_fit, b.Yfp_fit)
    assert torch.equal(a.Yq_apply, b.Yq_apply)
    assert not torch.equal(a.Yq_apply, a.Yq_fit)
    # quantised outputs track the FP outputs but are not equal to them
    c = np.corrcoef(a.Yq_fit.numpy().ravel(), a.Yfp_fit.numpy().ravel())[0, 1]
    assert 0.5 < c < 0.999


def test_weight_and_activation_levels():
    g = torch.Generator().manual_seed(0)
    Wt = torch.randn((7, 64), generator=g)
    for bits, nlev in ((2, 4), (4, 16)):
        Wq = W.quantize_weight_rows(Wt, bits)
        for r in range(7):
            lv = torch.unique(Wq[r])
            assert len(lv) <= nlev
            top = 2.0 ** (bits - 1) - 0.5
            scale = Wt[r].abs().max() / top
            k = (lv / scale).numpy()
            assert np.allclose(k - np.floor(k), 0.5, atol=1e-4) and np.abs(k).max() <= top + 1e-4
        X = torch.relu(torch.randn((50, 64), generator=g))
        s = W.activation_scale(X, bits)
        Xq = W.quantize_activation(X * 1.5, bits, s)          # exceeds the calibrated range: clipped
        lv = torch.unique(Xq / s).numpy()
        assert np.allclose(lv, np.round(lv), atol=1e-4) and lv.min() >= 0 and lv.max() <= 2 ** bits - 1


def test_config3_is_row_scaled_and_apply_aliases_fit():
    w = W.make(3, rows_scale=0.01)
    assert w.Yq_fit.shape == (2007, 64) and w.Yq_apply is w.Yq_fit and w.K == 64


def test_mixture_small():
    w = W.gaussian_mixture("mix", 4, 4, 3000, 32, 16, 1000, 8, 5)
    assert w.Yq_apply.shape == (3000, 32) and w.Yq_fit.shape == (1000, 32)
    assert w.Yfp_fit.shape == (1000, 32)
    assert w.Yq_fit.data_ptr() == w.Yq_apply.data_ptr()
    for j in range(32):
        assert len(torch.unique(w.Yq_apply[:, j])) <= 4
    # quantisation error is bounded by half a step of the column's range
    step = (w.Yq_apply.amax(0) - w.Yq_apply.amin(0)) / 3
    assert torch.all((w.Yq_fit - w.Yfp_fit).abs() <= step / 2 + 1e-4)
    w2 = W.gaussian_mixture("mix", 4, 4, 3000, 32, 16, 1000, 8, 5)
    assert torch.equal(w.Yq_apply, w2.Yq_apply)


def test_make_config4_scaled():
    w = W.make(4, rows_scale=1 / 2048)
    assert w.Yq_apply.shape == (2048, 1024) and w.Yq_fit.shape[0] == 256 and w.K == 256
