"""B200-native CAT (Cluster-based Affine Transformation) hot path.

`cat_fit` / `cat_apply` and the step-level entry points live in a C-ABI CUDA
library (csrc/, built in-tree as libcat.so); `binding` marshals torch device
tensors into it.  Nothing here computes on the CPU: if the CUDA library is
missing the calls raise.
"""
from . import workloads  # noqa: F401  (input generation only)

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
