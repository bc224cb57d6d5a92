"""The C-ABI library: builds, loads, exports every function include/cat.h declares,
and rejects bad arguments on the host before anything reaches a GPU."""
import ctypes
import os
import re

import pytest

from paper_2509_26277_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cat_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    L = ctypes.CDLL(path)
    names = declared_functions()
    assert "cat_fit" in names and "cat_apply" in names and len(names) >= 15
    for n in names:
        assert hasattr(L, n), f"{n} declared in cat.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_version_and_status_strings():
    L = binding.lib()
    assert b"sm_100a" in L.cat_version()
    seen = {L.cat_status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert L.cat_status_string(99) == b"unknown status"


def test_kernel_selection_settings_are_host_state():
    """Both selectors are process-wide host settings: readable and writable without a GPU."""
    assert binding.cat_get_apply_column_split() == 0
    try:
        for cs in (1, 2, 4):
            binding.cat_set_apply_column_split(cs)
            assert binding.cat_get_apply_column_split() == cs
        for bad in (3, 8, -1, 100):
            binding.cat_set_apply_column_split(bad)
            assert binding.cat_get_apply_column_split() == 0
    finally:
        binding.cat_set_apply_column_split(0)
    k = binding.cat_get_tensor_core_min_k()
    try:
        binding.cat_set_tensor_core_min_k(64)
        assert binding.cat_get_tensor_core_min_k() == 64
        binding.cat_set_tensor_core_min_k(0)
        assert binding.cat_get_tensor_core_min_k() == 1
    finally:
        binding.cat_set_tensor_core_min_k(k)


def test_workspace_queries_are_pure_host_functions():
    L = binding.lib()
    a = L.cat_apply_workspace_bytes(50_000, 1000, 16)
    f = L.cat_fit_workspace_bytes(1024, 1000, 16)
    assert a > 2 * 50_000 * 4 and f > a // 50 and a % 256 == 0 and f % 256 == 0
    big = L.cat_fit_workspace_bytes(262_144, 1024, 256)
    # the fp16 copy of the rows (N*D*2 bytes) plus modest sort tables and partial sums
    assert 262_144 * 1024 * 2 < big < 262_144 * 1024 * 2 + 128 * 2 ** 20
    assert L.cat_apply_host_workspace_bytes(4_194_304, 1024, 256) < 2 ** 30
    assert L.cat_fit_host_workspace_bytes(1024, 1000, 8) > 2 * 1024 * 1000 * 4
    # cat_fit sorts up to 2N entries with 32-bit positions: N < 2^30
    assert L.cat_fit_workspace_bytes(2 ** 30, 4, 2) == 0 and L.cat_fit_workspace_bytes(2 ** 30 - 1, 4, 2) > 0
    assert L.cat_apply_workspace_bytes(2 ** 31 - 1, 4, 2) > 0
    # unsupported or nonsensical sizes give 0
    assert L.cat_apply_workspace_bytes(10, 4, binding.MAX_K + 1) == 0
    assert L.cat_apply_workspace_bytes(10, binding.MAX_D + 1, 2) == 0
    assert L.cat_apply_workspace_bytes(2 ** 31, 4, 2) == 0
    assert L.cat_fit_workspace_bytes(0, 4, 2) == 0
    assert L.cat_fit_workspace_bytes(10, 0, 2) == 0
    assert L.cat_fit_workspace_bytes(10, 4, 0) == 0


def test_argument_errors_return_before_any_device_work():
    L = binding.lib()
    vp = ctypes.c_void_p
    fake = vp(0x1000)        # never dereferenced: every call below fails validation first
    odd = vp(0x1004)
    before = L.cat_kernel_launches()
    # NULL pointers
    assert L.cat_apply(None, 8, 4, 2, fake, fake, fake, fake, None, fake, 1 << 20, None) == 1
    assert L.cat_fit(fake, None, 8, 4, 2, 1, fake, fake, fake, None, fake, 1 << 20, None) == 1
    assert L.cat_assign(fake, 8, 4, 2, fake, None, fake, 1 << 20, None) == 1
    # shapes
    assert L.cat_fit(fake, fake, 3, 4, 5, 1, fake, fake, fake, None, fake, 1 << 20, None) == 2   # N < K
    assert L.cat_fit(fake, fake, 8, 4, 0, 1, fake, fake, fake, None, fake, 1 << 20, None) == 2   # K < 1
    assert L.cat_fit(fake, fake, 8, 0, 2, 1, fake, fake, fake, None, fake, 1 << 20, None) == 2   # D < 1
    assert L.cat_fit(fake, fake, 8, 4, 2, -1, fake, fake, fake, None, fake, 1 << 20, None) == 2  # iters < 0
    assert L.cat_apply_blend(fake, 8, 4, 2, fake, fake, fake, ctypes.c_float(1.5), fake, None,
                             fake, 1 << 20, None) == 2
    assert L.cat_apply_blend(fake, 8, 4, 2, fake, fake, fake, ctypes.c_float(float("nan")), fake, None,
                             fake, 1 << 20, None) == 2
    # limits
    assert L.cat_apply(fake, 8, 4, binding.MAX_K + 1, fake, fake, fake, fake, None, fake, 1 << 20, None) == 7
    assert L.cat_apply(fake, 2 ** 31, 4, 2, fake, fake, fake, fake, None, fake, 1 << 20, None) == 7
    # alignment
    assert L.cat_apply(odd, 8, 4, 2, fake, fake, fake, fake, None, fake, 1 << 20, None) == 3
    assert L.cat_fit(fake, fake, 8, 4, 2, 1, fake, odd, fake, None, fake, 1 << 20, None) == 3
    # workspace
    assert L.cat_apply(fake, 8, 4, 2, fake, fake, fake, fake, None, None, 1 << 20, None) == 4
    assert L.cat_apply(fake, 8, 4, 2, fake, fake, fake, fake, None, fake, 16, None) == 4
    assert L.cat_fit(fake, fake, 8, 4, 2, 1, fake, fake, fake, None, fake, 16, None) == 4
    assert L.cat_cluster_sums(fake, fake, 8, 4, 2, fake, fake, fake, 16, None) == 4
    assert L.cat_apply_host(fake, 8, 4, 2, fake, fake, fake, fake, None, fake, 16, None) == 4
    assert L.cat_fit_host(fake, fake, 8, 4, 2, 1, fake, fake, fake, None, None, 0, None) == 4
    # init must not alias the output
    assert L.cat_fit_from(fake, fake, 8, 4, 2, 1, fake, fake, fake, fake, None, None, fake, 1 << 20, None) == 2
    assert L.cat_kernel_launches() == before


def test_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros((8, 4))
    with pytest.raises(TypeError):
        binding.cat_assign(x, x[:2].contiguous(), ws=torch.zeros(1024, dtype=torch.uint8))
