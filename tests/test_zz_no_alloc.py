"""lsgd_topk_select_static: the selector for callers that cannot allocate device
memory (no cudaMalloc allowed where they run, or no allocator of their own).

It must give exactly what lsgd_topk_select gives (and what the CPU oracle gives),
call after call, although all calls share one scratch array inside the library
that still holds the previous call's data.  This file is collected last on purpose.
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


CASES = [(200_003, 50_000, 21), (131_072, 131_072, 22), (50_000, 12_500, 23), (3_000, 700, 24), (900, 300, 25)]


def test_static_selector_matches_the_workspace_one_twice_in_a_row(L, oracle):
    # two different pools back to back: the second call meets the first call's leftovers in the scratch
    for order in (L.ORDER_LOSS_DESC, L.ORDER_INDEX_ASC):
        for N, k, seed in CASES:
            h = wl.loss_like_vector(seed, N, dup_frac=0.05, specials=True)
            v = torch.from_numpy(h).cuda()
            o_idx, o_vals = oracle.topk(h, k, order)           # what the plain definition selects
            want_idx, want_vals = L.topk_select(v, k, order)   # what the entry point with a workspace selects
            for _ in range(2):                                 # the second call runs over the first one's leftovers
                idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
                vals = torch.full((k,), -1.0, dtype=torch.float32, device="cuda")
                L.topk_select_static(v, k, idx, vals, order)
                # integer work: the tolerance of the selector tests is bit-exactness
                assert torch.equal(idx, want_idx)
                assert torch.equal(vals.view(torch.int32), want_vals.view(torch.int32))
                np.testing.assert_array_equal(idx.cpu().numpy(), o_idx)
                np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), o_vals.view(np.uint32))


def test_static_selector_allocates_nothing(L):
    """Neither torch's allocator nor the driver's count of free device memory moves across the calls."""
    pools = [(torch.from_numpy(wl.loss_like_vector(seed, N, dup_frac=0.05)).cuda(), k,
              torch.empty(k, dtype=torch.int32, device="cuda"), torch.empty(k, dtype=torch.float32, device="cuda"))
             for N, k, seed in CASES]
    # first calls: the scratch address is looked up and the kernels of both orders are loaded onto the device
    for order in (L.ORDER_LOSS_DESC, L.ORDER_INDEX_ASC):
        for v, k, idx, vals in pools:
            L.topk_select_static(v, k, idx, vals, order)
    torch.cuda.synchronize()
    torch_before = torch.cuda.memory_stats()["allocation.all.allocated"]  # allocations torch made so far
    free_before, _ = torch.cuda.mem_get_info()                            # the driver's view: cudaMalloc would lower it
    for order in (L.ORDER_LOSS_DESC, L.ORDER_INDEX_ASC):
        for v, k, idx, vals in pools:
            L.topk_select_static(v, k, idx, vals, order)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == torch_before
    assert free_after == free_before


def test_static_selector_limits(L, oracle):
    lib = L.lib()
    ptr = ctypes.c_void_p(0x1000)
    n = L.STATIC_TOPK_MAX_N
    # one past the built-in scratch: refused on the host, nothing launched
    assert lib.lsgd_topk_select_static(ptr, n + 1, 5, 0, ptr, None, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_topk_select_static(ptr, 10, 11, 0, ptr, None, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_topk_select_static(ptr, 10, 0, 0, None, None, None) == L.OK
    # the largest pool it takes
    h = wl.loss_like_vector(31, n, dup_frac=0.01)
    v = torch.from_numpy(h).cuda()
    for k in (n // 3, n):
        want_idx, _ = L.topk_select(v, k, L.ORDER_LOSS_DESC, want_vals=False)
        idx = torch.empty(k, dtype=torch.int32, device="cuda")
        L.topk_select_static(v, k, idx, None, L.ORDER_LOSS_DESC)
        assert torch.equal(idx, want_idx)
        np.testing.assert_array_equal(idx.cpu().numpy(), oracle.topk(h, k, oracle.LOSS_DESC)[0])
