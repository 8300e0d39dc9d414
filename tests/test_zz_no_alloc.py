"""lsgd_topk_select_static: the selector for callers that cannot allocate device
memory (no cudaMalloc allowed where they run, or no allocator of their own).

It must give exactly what lsgd_topk_select gives, call after call, although all
calls share one scratch array inside the library that still holds the previous
call's data.  This file is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2508_08540_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2508_08540_b200 import lsgd

    lsgd.lib()
    return lsgd


def test_static_selector_matches_the_workspace_one_twice_in_a_row(L):
    # two different pools back to back: the second call meets the first call's leftovers in the scratch
    cases = [(200_003, 50_000, 21), (131_072, 131_072, 22), (50_000, 12_500, 23), (3_000, 700, 24)]
    for order in (L.ORDER_LOSS_DESC, L.ORDER_INDEX_ASC):
        for N, k, seed in cases:
            v = torch.from_numpy(wl.loss_like_vector(seed, N, dup_frac=0.05, specials=True)).cuda()
            want_idx, want_vals = L.topk_select(v, k, order)
            idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
            vals = torch.full((k,), -1.0, dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            before = torch.cuda.memory_stats()["allocation.all.allocated"]  # allocations made so far
            L.topk_select_static(v, k, idx, vals, order)
            L.topk_select_static(v, k, idx, vals, order)  # and once more over its own leftovers
            torch.cuda.synchronize()
            assert torch.cuda.memory_stats()["allocation.all.allocated"] == before  # none was made by the calls
            # integer work: the tolerance of the selector tests is bit-exactness
            assert torch.equal(idx, want_idx)
            assert torch.equal(vals.view(torch.int32), want_vals.view(torch.int32))


def test_static_selector_limits(L):
    lib = L.lib()
    ptr = ctypes.c_void_p(0x1000)
    n = L.STATIC_TOPK_MAX_N
    # one past the built-in scratch: refused on the host, nothing launched
    assert lib.lsgd_topk_select_static(ptr, n + 1, 5, 0, ptr, None, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_topk_select_static(ptr, 10, 11, 0, ptr, None, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_topk_select_static(ptr, 10, 0, 0, None, None, None) == L.OK
    # the largest pool it takes
    v = torch.from_numpy(wl.loss_like_vector(31, n, dup_frac=0.01)).cuda()
    k = n // 3
    want_idx, _ = L.topk_select(v, k, L.ORDER_LOSS_DESC, want_vals=False)
    idx = torch.empty(k, dtype=torch.int32, device="cuda")
    L.topk_select_static(v, k, idx, None, L.ORDER_LOSS_DESC)
    assert torch.equal(idx, want_idx)
