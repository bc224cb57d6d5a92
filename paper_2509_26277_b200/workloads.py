"""Seeded synthetic workloads shaped like CAT's inputs.

CAT consumes two matrices of model outputs for the same samples: the low-bit
(LQ) outputs ``Yq`` and the full-precision (FP) outputs ``Yfp`` (Algorithm 1,
"all_q", "all_fp").  The paper takes them from quantised ImageNet classifiers
(D = 1000 logits, 10 ... 100 000 calibration rows, K = 1 ... 256 clusters);
those networks and images are not available here, so these generators stand in
for them: a random linear head evaluated with fake-quantised weights and
activations, or a Gaussian mixture with per-column fake quantisation.

This module holds input generation only -- none of CAT's own arithmetic -- and
is the one piece of code that the CPU checker's tests and the CUDA library's
tests both use: a workload is generated once and the same bytes go to both.

Five configurations (index = ``config``):

0  tiny            seed 0  linear head Din=512  D=1000 W2A2  fit 1024 rows   K=8   20 iters  apply 1024
1  ResNet-18 head  seed 1  linear head Din=512  D=1000 W2A2  fit 1024 rows   K=16  30 iters  apply 50 000
2  ResNet-50 head  seed 2  linear head Din=2048 D=1000 W4A4  fit 4096 rows   K=32  30 iters  apply 50 000
3  conv feature    seed 3  im2col 3x3x64->64: Din=576 D=64 W2A2, 200 704 rows, K=64 25 iters, apply same rows
4  bandwidth       seed 4  256-component Gaussian mixture, 4 194 304 x 1024, per-column 2-bit
                           fake quantisation; fit on the first 262 144 rows, K=256 25 iters; apply on all rows
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import torch


@dataclass
class Workload:
    name: str
    config: int
    K: int
    iters: int
    Yq_fit: torch.Tensor            # [N_fit, D] fp32
    Yfp_fit: torch.Tensor           # [N_fit, D] fp32
    Yq_apply: torch.Tensor          # [N_apply, D] fp32 (may alias Yq_fit)

    @property
    def D(self) -> int:
        return int(self.Yq_fit.shape[1])

    @property
    def N_fit(self) -> int:
        return int(self.Yq_fit.shape[0])

    @property
    def N_apply(self) -> int:
        return int(self.Yq_apply.shape[0])


# (seed, Din, D, weight bits, activation bits, fit rows, apply rows (None = the fit rows), K, iters)
_LINEAR = {
    0: ("tiny", 0, 512, 1000, 2, 2, 1024, 1024, 8, 20),
    1: ("resnet18_head_w2a2", 1, 512, 1000, 2, 2, 1024, 50_000, 16, 30),
    2: ("resnet50_head_w4a4", 2, 2048, 1000, 4, 4, 4096, 50_000, 32, 30),
    3: ("conv3x3x64_w2a2", 3, 576, 64, 2, 2, 200_704, None, 64, 25),
}
_MIXTURE = ("bandwidth_stress", 4, 4_194_304, 1024, 256, 262_144, 256, 25)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def quantize_weight_rows(W: torch.Tensor, bits: int) -> torch.Tensor:
    """Per-row symmetric mid-rise fake quantisation: 2**bits levels
    {+-0.5, +-1.5, ...} * scale with scale = max|w_row| / (2**(bits-1) - 0.5)."""
    top = 2.0 ** (bits - 1) - 0.5
    scale = W.abs().amax(dim=1, keepdim=True) / top
    scale = torch.where(scale > 0, scale, torch.ones_like(scale))
    q = torch.clamp(torch.floor(W / scale) + 0.5, -top, top)
    return q * scale


def activation_scale(X: torch.Tensor, bits: int) -> float:
    """Per-tensor unsigned scale = max(X) / (2**bits - 1), taken on the fit set."""
    s = float(X.max().item()) / (2.0 ** bits - 1.0)
    return s if s > 0 else 1.0


def quantize_activation(X: torch.Tensor, bits: int, scale: float) -> torch.Tensor:
    """Unsigned per-tensor fake quantisation with a given scale (round half to
    even, clipped to 0 ... 2**bits - 1)."""
    return torch.clamp(torch.round(X / scale), 0.0, 2.0 ** bits - 1.0) * scale


def _matmul_rows(X: torch.Tensor, Wt: torch.Tensor, chunk: int = 65536) -> torch.Tensor:
    out = torch.empty((X.shape[0], Wt.shape[1]), dtype=torch.float32, device=X.device)
    for r in range(0, X.shape[0], chunk):
        out[r:r + chunk] = X[r:r + chunk] @ Wt
    return out


def linear_head(name: str, config: int, seed: int, din: int, d: int, wbits: int, abits: int,
                n_fit: int, n_apply: Optional[int], K: int, iters: int, device="cpu") -> Workload:
    """Outputs of a random linear layer, FP and fake-quantised.

    X = ReLU(N(0,1)) [n, din]; W ~ N(0, 1/din) [d, din]; Yfp = X W^T;
    Yq = Xq Wq^T.  The apply set draws a second X (seed + 1000), shares W and
    reuses the fit set's activation scale (calibration-time ranges are kept
    at inference time)."""
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        g = _gen(seed, device)
        X = torch.relu(torch.randn((n_fit, din), generator=g, device=device, dtype=torch.float32))
        W = torch.randn((d, din), generator=g, device=device, dtype=torch.float32) * (din ** -0.5)
        Wq = quantize_weight_rows(W, wbits)
        s = activation_scale(X, abits)
        Yfp = _matmul_rows(X, W.t().contiguous())
        Yq = _matmul_rows(quantize_activation(X, abits, s), Wq.t().contiguous())
        if n_apply is None:
            Yq_apply = Yq
        else:
            g2 = _gen(seed + 1000, device)
            X2 = torch.relu(torch.randn((n_apply, din), generator=g2, device=device,
                                        dtype=torch.float32))
            Yq_apply = _matmul_rows(quantize_activation(X2, abits, s), Wq.t().contiguous())
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev
    return Workload(name, config, K, iters, Yq.contiguous(), Yfp.contiguous(),
                    Yq_apply.contiguous())


_MIX_CHUNK = 65536  # rows per generator chunk; fixed so that bytes do not depend on memory size


def _mixture_chunk(seed: int, c: int, rows: int, means: torch.Tensor, stds: torch.Tensor,
                   device) -> torch.Tensor:
    g = _gen(seed * 1_000_003 + 17 + c, device)
    comp = torch.randint(0, means.shape[0], (rows,), generator=g, device=device)
    z = torch.randn((rows, means.shape[1]), generator=g, device=device, dtype=torch.float32)
    return means[comp] + stds[comp] * z


def gaussian_mixture(name: str, config: int, seed: int, n: int, d: int, components: int,
                     n_fit: int, K: int, iters: int, device="cpu") -> Workload:
    """Rows drawn from a `components`-component Gaussian mixture (uniform
    weights; means ~ N(0, 4) i.e. std 2; per-component diagonal std ~
    U(0.5, 2)), and their per-column 2-bit uniform fake quantisation over the
    column's [min, max] across all n rows.  Generated in fixed chunks in two
    passes (ranges, then quantisation) so that only Yq (all rows) and the
    first n_fit rows of Yfp are ever held."""
    g = _gen(seed, device)
    means = torch.randn((components, d), generator=g, device=device, dtype=torch.float32) * 2.0
    stds = torch.rand((components, d), generator=g, device=device, dtype=torch.float32) * 1.5 + 0.5
    lo = torch.full((d,), float("inf"), device=device)
    hi = torch.full((d,), float("-inf"), device=device)
    nchunks = (n + _MIX_CHUNK - 1) // _MIX_CHUNK
    for c in range(nchunks):
        rows = min(_MIX_CHUNK, n - c * _MIX_CHUNK)
        y = _mixture_chunk(seed, c, rows, means, stds, device)
        lo = torch.minimum(lo, y.amin(dim=0))
        hi = torch.maximum(hi, y.amax(dim=0))
        del y
    step = (hi - lo) / 3.0
    step = torch.where(step > 0, step, torch.ones_like(step))
    Yq = torch.empty((n, d), dtype=torch.float32, device=device)
    Yfp_fit = torch.empty((n_fit, d), dtype=torch.float32, device=device)
    for c in range(nchunks):
        r0 = c * _MIX_CHUNK
        rows = min(_MIX_CHUNK, n - r0)
        y = _mixture_chunk(seed, c, rows, means, stds, device)
        if r0 < n_fit:
            m = min(rows, n_fit - r0)
            Yfp_fit[r0:r0 + m] = y[:m]
        Yq[r0:r0 + rows] = lo + step * torch.clamp(torch.round((y - lo) / step), 0.0, 3.0)
        del y
    return Workload(name, config, K, iters, Yq[:n_fit], Yfp_fit, Yq)


def make(config: int, device="cpu", rows_scale: float = 1.0, seed_offset: int = 0) -> Workload:
    """Build workload `config` (0-4) on `device`.

    rows_scale < 1 shrinks the row counts (never below K) for CPU-sized test
    cases; shapes D, K, iters and the value recipe stay as specified.
    seed_offset draws different rows from the same recipe (one shard per rank)."""
    if config in _LINEAR:
        name, seed, din, d, wb, ab, n_fit, n_apply, K, iters = _LINEAR[config]
        seed += seed_offset
        n_fit = max(K, int(round(n_fit * rows_scale)))
        if n_apply is not None:
            n_apply = max(1, int(round(n_apply * rows_scale)))
        return linear_head(name, config, seed, din, d, wb, ab, n_fit, n_apply, K, iters, device)
    if config == 4:
        name, seed, n, d, comps, n_fit, K, iters = _MIXTURE
        seed += seed_offset
        n = max(K, int(round(n * rows_scale)))
        n_fit = max(K, min(n, int(round(n_fit * rows_scale))))
        return gaussian_mixture(name, config, seed, n, d, comps, n_fit, K, iters, device)
    raise ValueError(f"unknown config {config}")


def spec(config: int) -> dict:
    """Shapes of workload `config` without generating it."""
    if config in _LINEAR:
        name, seed, din, d, wb, ab, n_fit, n_apply, K, iters = _LINEAR[config]
        return dict(name=name, seed=seed, D=d, N_fit=n_fit,
                    N_apply=n_fit if n_apply is None else n_apply, K=K, iters=iters)
    if config == 4:
        name, seed, n, d, comps, n_fit, K, iters = _MIXTURE
        return dict(name=name, seed=seed, D=d, N_fit=n_fit, N_apply=n, K=K, iters=iters)
    raise ValueError(f"unknown config {config}")
