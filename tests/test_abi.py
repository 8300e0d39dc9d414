"""The C-ABI library loads and exports what include/lsgd.h declares; host-side
argument checks and host-only entry points work without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2508_08540_b200 import build

    build.build_library()
    from paper_2508_08540_b200 import lsgd

    return lsgd


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lsgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"LSGD_API\s+[\w\s\*]+?\b(lsgd_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert set(names) == set(L.EXPORTS) and len(names) == 19
    lib = ctypes.CDLL(L.LIB_PATH)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings_and_version(L):
    assert L.version() >= 100
    seen = {L.status_string(s) for s in range(7)}
    assert len(seen) == 7 and L.status_string(0) == "ok"
    assert L.status_string(99) == "unknown status"


def test_workspace_queries(L):
    assert L.score_workspace_bytes(1000, 1, 10) == 256
    assert L.score_workspace_bytes(1024, 128, 30522) >= 256 + 4 * 1024 * 128
    assert L.score_workspace_bytes(-1, 1, 10) == 0 and L.score_workspace_bytes(5, 0, 10) == 0
    assert L.topk_workspace_bytes(10, 11) == 0 and L.topk_workspace_bytes(-1, 0) == 0
    a = L.topk_workspace_bytes(1_281_167, 320_000)
    assert a >= 4 * 4 * 320_000 and a % 256 == 0
    assert L.score_topk_workspace_bytes(1024, 128, 30522, 256) == L.topk_workspace_bytes(1024, 256) + 4 * 1024 * 128
    # monotone in k and N
    assert L.topk_workspace_bytes(50_000, 12_500) <= L.topk_workspace_bytes(50_000, 50_000)


def test_weights_from_steps_host_only(L):
    w = L.weights_from_steps([32] * 8 + [1] * 2)  # Section 5.1 setting: tau_F = 32, tau_S = 1
    import numpy as np

    assert np.float32(w[0]) == np.float32(32 / 258) and np.float32(w[9]) == np.float32(1 / 258)
    assert abs(sum(w) - 1.0) < 1e-6
    with pytest.raises(L.LsgdError) as e:
        L.weights_from_steps([0, 0, 0])
    assert e.value.status == L.ERR_INVALID_ARG
    with pytest.raises(L.LsgdError):
        L.weights_from_steps([3, -1])


def test_argument_errors_are_found_before_any_cuda_call(L):
    lib = L.lib()
    one = ctypes.c_float(1.0)
    ptr = ctypes.c_void_p(0x1000)
    arr = (ctypes.c_void_p * 1)(0x1000)
    arrp = ctypes.cast(arr, ctypes.c_void_p)
    wp = ctypes.cast(ctypes.pointer(one), ctypes.c_void_p)
    # replica count out of range, NULLs, negative size
    assert lib.lsgd_aggregate(arrp, wp, 0, 16, ptr, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_aggregate(arrp, wp, 65, 16, ptr, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_aggregate(None, wp, 1, 16, ptr, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_aggregate(arrp, wp, 1, -1, ptr, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_aggregate(arrp, wp, 1, 0, None, None) == L.OK
    # partial overlap of out with a replica; misaligned replica
    assert lib.lsgd_aggregate(arrp, wp, 1, 16, ctypes.c_void_p(0x1010), None) == L.ERR_INVALID_ARG
    bad = (ctypes.c_void_p * 1)(0x1002)
    assert lib.lsgd_aggregate(ctypes.cast(bad, ctypes.c_void_p), wp, 1, 16, ctypes.c_void_p(0x9000), None) == L.ERR_ALIGNMENT
    # selector
    assert lib.lsgd_topk_select(ptr, 10, 11, 0, ptr, None, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_topk_select(ptr, 10, -1, 0, ptr, None, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_topk_select(ptr, 10, 5, 7, ptr, None, ptr, 1 << 20, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_topk_select(ptr, 1 << 31, 5, 0, ptr, None, ptr, 1 << 20, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_topk_select(ptr, 10, 0, 0, None, None, None, 0, None) == L.OK
    assert lib.lsgd_topk_select(None, 10, 5, 0, ptr, None, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_topk_select(ptr, 10, 5, 0, ptr, None, ctypes.c_void_p(0x2000), 16, None) == L.ERR_WORKSPACE
    assert lib.lsgd_topk_select(ptr, 10, 5, 0, ptr, None, ctypes.c_void_p(0x2010), 1 << 20, None) == L.ERR_ALIGNMENT
    assert lib.lsgd_topk_select(ctypes.c_void_p(0x1001), 10, 5, 0, ptr, None, ptr, 1 << 20, None) == L.ERR_ALIGNMENT
    # scorer
    big = ctypes.c_void_p(0x100000)
    assert lib.lsgd_score_losses(ptr, 5, ptr, 4, 1, 10, -100, big, ptr, 1 << 20, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_score_losses(ptr, 0, ptr, 4, 0, 10, -100, big, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_score_losses(ptr, 0, ptr, 4, 1, 0, -100, big, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_score_losses(ptr, 0, None, 4, 1, 10, -100, big, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_score_losses(ptr, 0, ptr, 0, 1, 10, -100, None, None, 0, None) == L.OK
    assert lib.lsgd_score_losses(ptr, 0, ptr, 4, 1, 10, -100, ctypes.c_void_p(0x1008), ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_score_losses(ctypes.c_void_p(0x1002), 0, ptr, 4, 1, 10, -100, big, ptr, 1 << 20, None) == L.ERR_ALIGNMENT
    assert lib.lsgd_score_losses(ptr, 0, ptr, 4, 1, 10, -100, big, ptr, 16, None) == L.ERR_WORKSPACE
    assert lib.lsgd_score_topk(ptr, 0, ptr, 4, 1, 10, -100, 5, 0, big, ptr, None, ptr, 1 << 20, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_read_device_status(None, None, None) == L.ERR_INVALID_ARG


def test_allocation_sizes_and_shares_host_only(L):
    # Section 5.1's setting (tau_F = 32 on 8 fast workers, tau_S = 1 on 2 slow ones): N_F / N = 256 / 258
    assert L.allocation_sizes(50_000, 32, 8, 1, 2, 1.0) == (49_612, 388, 49_612)
    nf, ns, k = L.allocation_sizes(1_281_167, 16, 4, 4, 4, 0.3)
    assert nf + ns == 1_281_167 and nf == 1_281_167 * 64 // 80 and k == int(0.3 * nf)
    assert L.allocation_sizes(1000, 5, 0, 2, 3, 0.5) == (0, 1000, 0)
    # decimal lambdas give the decimal product rounded down (0.29 * 100 is 28.999999999999996 in double)
    from fractions import Fraction

    for n in (100, 49_612, 1_281_167, 2_000_000_000):
        for lam in [f"{i / 100:.2f}" for i in range(101)] + ["0.333", "0.0007"]:
            assert L.allocation_sizes(n, 1, 1, 0, 1, float(lam))[2] == (Fraction(lam) * n).__floor__(), (n, lam)
    for bad in [(-1, 1, 1, 1, 1, 0.5), (10, 0, 0, 0, 0, 0.5), (10, 1, 1, 1, 1, 1.5), (10, 1, 1, 1, 1, float("nan")),
                (10, -1, 1, 1, 1, 0.5)]:
        with pytest.raises(L.LsgdError) as e:
            L.allocation_sizes(*bad)
        assert e.value.status == L.ERR_INVALID_ARG
    parts = [L.worker_share(49_612, 8, p) for p in range(8)]
    assert parts[0][0] == 0 and parts[-1][1] == 49_612 and all(parts[p][1] == parts[p + 1][0] for p in range(7))
    assert {e - b for b, e in parts} <= {6201, 6202}
    for bad in [(10, 0, 0), (10, 2, 2), (10, 2, -1), (-1, 2, 0)]:
        with pytest.raises(L.LsgdError):
            L.worker_share(*bad)


def test_draw_argument_errors_are_found_before_any_cuda_call(L):
    lib = L.lib()
    ptr = ctypes.c_void_p(0x1000)
    big = 1 << 24
    assert L.draw_workspace_bytes(10, 11) == 0 and L.draw_workspace_bytes(-1, 0) == 0
    assert L.draw_workspace_bytes(50_000, 388) >= L.topk_workspace_bytes(50_000, 388) + 4 * 50_000
    assert L.fast_allocation_workspace_bytes(100, 60, 41) == 0
    assert L.fast_allocation_workspace_bytes(50_000, 12_403, 37_209) == L.draw_workspace_bytes(50_000, 37_209)
    assert lib.lsgd_draw_uniform(10, 11, 1, 0, None, 0, ptr, ptr, big, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_draw_uniform(10, 8, 1, 0, ptr, 3, ptr, ptr, big, None) == L.ERR_INVALID_ARG  # only 7 candidates
    assert lib.lsgd_draw_uniform(10, 2, 1, 0, None, 3, ptr, ptr, big, None) == L.ERR_INVALID_ARG  # list missing
    assert lib.lsgd_draw_uniform(10, 0, 1, 0, None, 0, None, None, 0, None) == L.OK
    assert lib.lsgd_draw_uniform(1 << 31, 5, 1, 0, None, 0, ptr, ptr, big, None) == L.ERR_UNSUPPORTED
    assert lib.lsgd_draw_uniform(10, 5, 1, 0, None, 0, ptr, ptr, 16, None) == L.ERR_WORKSPACE
    assert lib.lsgd_draw_uniform(10, 5, 1, 0, None, 0, ctypes.c_void_p(0x1002), ptr, big, None) == L.ERR_ALIGNMENT
    assert lib.lsgd_draw_uniform(10, 5, 1, 0, None, 0, ptr, ctypes.c_void_p(0x1010), big, None) == L.ERR_ALIGNMENT
    assert lib.lsgd_fast_allocation(ptr, 10, 6, 5, 1, 0, ptr, ptr, big, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_fast_allocation(None, 10, 6, 2, 1, 0, ptr, ptr, big, None) == L.ERR_INVALID_ARG
    assert lib.lsgd_fast_allocation(ptr, 10, 0, 0, 1, 0, None, None, 0, None) == L.OK
    assert lib.lsgd_fast_allocation(ptr, 10, 6, 2, 1, 0, ptr, ptr, 16, None) == L.ERR_WORKSPACE


def test_aggregate_round_argument_errors(L):
    lib = L.lib()
    one = ctypes.c_float(1.0)
    wp = ctypes.cast(ctypes.pointer(one), ctypes.c_void_p)
    two = (ctypes.c_float * 2)(0.5, 0.5)
    w2 = ctypes.cast(two, ctypes.c_void_p)
    arr = (ctypes.c_void_p * 1)(0x10000)
    arrp = ctypes.cast(arr, ctypes.c_void_p)
    far = ctypes.c_void_p(0x90000)
    f = lib.lsgd_aggregate_round
    assert f(arrp, 7, wp, 1, 16, None, far, 0, None) == L.ERR_UNSUPPORTED
    assert f(arrp, 0, wp, 0, 16, None, far, 0, None) == L.ERR_INVALID_ARG
    assert f(arrp, 0, wp, 1, 16, None, None, 0, None) == L.ERR_INVALID_ARG       # no destination at all
    assert f(arrp, 0, wp, 1, 0, None, None, 1, None) == L.OK
    assert f(arrp, 1, wp, 1, 16, None, ctypes.c_void_p(0x10000), 0, None) == L.ERR_INVALID_ARG  # bf16 replica aliasing fp32 out
    assert f(arrp, 0, wp, 1, 16, None, ctypes.c_void_p(0x10010), 0, None) == L.ERR_INVALID_ARG  # partial overlap
    assert f(arrp, 0, wp, 1, 16, ctypes.c_void_p(0x10020), far, 0, None) == L.ERR_INVALID_ARG   # base overlaps the replica
    assert f(arrp, 0, wp, 1, 16, ctypes.c_void_p(0x90010), far, 0, None) == L.ERR_INVALID_ARG   # base overlaps out
    assert f(arrp, 0, wp, 1, 16, None, ctypes.c_void_p(0x90002), 0, None) == L.ERR_ALIGNMENT
    odd = (ctypes.c_void_p * 1)(0x10001)
    assert f(ctypes.cast(odd, ctypes.c_void_p), 1, wp, 1, 16, None, far, 0, None) == L.ERR_ALIGNMENT
    twice = (ctypes.c_void_p * 2)(0x10000, 0x10000)
    assert f(ctypes.cast(twice, ctypes.c_void_p), 0, w2, 2, 16, None, far, 1, None) == L.ERR_INVALID_ARG  # broadcast into aliased replicas


def test_binding_fails_loudly_without_the_library(tmp_path):
    """There is no CPU or library fallback: without liblsgd.so every entry point raises."""
    import subprocess
    import sys

    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "from paper_2508_08540_b200 import lsgd\n"
        "lsgd.LIB_PATH = %r\n"
        "try:\n"
        "    lsgd.weights_from_steps([1, 2])\n"
        "except ImportError as e:\n"
        "    print('raised', 'missing' in str(e))\n"
        "else:\n"
        "    print('no error')\n"
    ) % (ROOT, str(tmp_path / "liblsgd.so"))
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    assert out.stdout.strip() == "raised True", out.stdout + out.stderr


def test_library_sources_never_allocate_device_memory():
    """The library's contract: the caller owns every buffer.  No source of liblsgd may name an allocating or freeing
    runtime call (the GPU tests can only watch torch's allocator and the driver's free-memory count)."""
    import glob

    banned = re.compile(r"\b(cudaMalloc\w*|cudaFree\w*|cudaMemPool\w*|cudaHostAlloc|cudaHostRegister|cuMemAlloc\w*|"
                        r"cuMemCreate|cuMemMap|cuMemFree\w*)\s*\(")
    files = sorted(glob.glob(os.path.join(ROOT, "paper_2508_08540_b200", "csrc", "*.cu*")))
    assert len(files) >= 8
    for path in files:
        text = open(path).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        hit = banned.search(text)
        assert hit is None, f"{os.path.basename(path)} calls {hit.group(1)}"
