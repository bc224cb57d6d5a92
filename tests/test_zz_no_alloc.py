"""cat_assign_noalloc, the entry point for callers that cannot allocate device memory
(it keeps its scratch in a fixed array inside the library).  Collected last on purpose.

The check: through the C ABI, its labels equal cat_assign's (and the CPU oracle's) on the same
inputs, twice in a row -- the second call right after one that filled the shared scratch with a long queue of
exact-pass rows, so anything the first call left behind would show."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2509_26277_b200 import binding as B
from tests.parity import labels_match


def test_noalloc_rejects_sizes_beyond_its_limits_on_the_host():
    L = B.lib()
    fake = ctypes.c_void_p(0x1000)   # never dereferenced: validation fails first
    before = L.cat_kernel_launches()
    assert L.cat_assign_noalloc(fake, B.NOALLOC_MAX_ROWS + 1, 8, 2, fake, fake, None) == 7
    assert L.cat_assign_noalloc(fake, 16, 8, B.MAX_K + 1, fake, fake, None) == 7
    assert L.cat_assign_noalloc(fake, 16, B.MAX_D + 1, 2, fake, fake, None) == 7
    assert L.cat_assign_noalloc(None, 16, 8, 2, fake, fake, None) == 1
    assert L.cat_assign_noalloc(fake, 0, 8, 2, fake, fake, None) == 2
    assert L.cat_assign_noalloc(ctypes.c_void_p(0x1004), 16, 8, 2, fake, fake, None) == 3
    assert b"limits" in L.cat_status_string(7)
    assert L.cat_kernel_launches() == before


@pytest.mark.gpu
def test_noalloc_labels_equal_cat_assign_on_two_calls_in_a_row():
    rng = np.random.default_rng(2024)
    # call 1: every row identical and every centroid identical -> all 5000 rows go through
    # the exact pass, which fills the shared queue
    Y1 = torch.from_numpy(np.tile(rng.normal(size=(1, 40)).astype(np.float32), (5000, 1))).cuda()
    C1 = Y1[:6].clone()
    # call 2: ordinary data, ragged row count, K not a multiple of the tile
    Y2 = torch.from_numpy(rng.normal(size=(70001, 100)).astype(np.float32)).cuda()
    C2 = torch.from_numpy(rng.normal(size=(37, 100)).astype(np.float32)).cuda()
    want1 = B.cat_assign(Y1, C1)
    want2 = B.cat_assign(Y2, C2)
    got1 = torch.full((5000,), -7, dtype=torch.int32, device="cuda")
    got2 = torch.full((70001,), -7, dtype=torch.int32, device="cuda")
    B.cat_assign_noalloc(Y1, C1, got1)
    B.cat_assign_noalloc(Y2, C2, got2)
    torch.cuda.synchronize()
    assert torch.equal(got1, want1) and int(got1.max()) == 0
    assert torch.equal(got2, want2)
    # and against the CPU oracle, which shares nothing with either entry point
    lab, best, second = O.assign(Y2.cpu().numpy(), C2.cpu().numpy())
    labels_match(got2.cpu().numpy(), lab, best, second, "cat_assign_noalloc labels")
    # and once more in the opposite order, at the row limit
    Y3 = torch.from_numpy(rng.normal(size=(B.NOALLOC_MAX_ROWS, 16)).astype(np.float32)).cuda()
    C3 = Y3[:200].clone()
    got3 = torch.empty((B.NOALLOC_MAX_ROWS,), dtype=torch.int32, device="cuda")
    B.cat_assign_noalloc(Y3, C3, got3)
    B.cat_assign_noalloc(Y1, C1, got1)
    torch.cuda.synchronize()
    assert torch.equal(got3, B.cat_assign(Y3, C3)) and torch.equal(got1, want1)
    with pytest.raises(B.CatError) as e:
        B.cat_assign_noalloc(torch.zeros((B.NOALLOC_MAX_ROWS + 1, 4), device="cuda"), C3[:2, :4].contiguous(),
                             torch.empty((B.NOALLOC_MAX_ROWS + 1,), dtype=torch.int32, device="cuda"))
    assert e.value.status == 7
