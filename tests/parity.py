"""Helpers for comparing the CUDA library with the CPU oracle.

Tolerances (fp32 results): |a - b| <= 1e-6 + 1e-5 |b|.  Labels must be equal except
on rows the oracle marks as near-ties (best-vs-second gap <= 1e-6 relative), which
are counted and reported."""
import numpy as np

ABS_TOL = 1e-6
REL_TOL = 1e-5
NEAR_REL = 1e-6


def close(a, b, what, abs_tol=ABS_TOL, rel_tol=REL_TOL):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape, f"{what}: shape {a.shape} vs {b.shape}"
    err = np.abs(a - b)
    bound = abs_tol + rel_tol * np.abs(b)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), a.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {a.size} outside tolerance; worst at {i}: "
                             f"got {a[i]!r}, want {b[i]!r}, |diff| {err[i]:.3e}")
    return float(err.max()) if a.size else 0.0


def labels_match(gpu_labels, ora_labels, best, second, what, near_rel=NEAR_REL):
    """Bit-exact except near-tie rows.  Returns (#near-tie rows, #mismatches among them)."""
    gpu_labels = np.asarray(gpu_labels)
    near = (second - best) <= near_rel * second
    diff = gpu_labels != ora_labels
    hard = diff & ~near
    if hard.any():
        i = int(np.flatnonzero(hard)[0])
        raise AssertionError(f"{what}: {int(hard.sum())} label mismatches outside the near-tie band; "
                             f"first at row {i}: gpu {gpu_labels[i]}, oracle {ora_labels[i]}, "
                             f"best {best[i]!r}, second {second[i]!r}")
    return int(near.sum()), int((diff & near).sum())
