"""Parity of the per-epoch data allocation (Section 4.2) on the GPU with the CPU oracle: integer work, so every
index must match exactly.  Sizes span the single-CTA path, several tiles with a ragged tail, and the five
configurations' pool sizes."""
import numpy as np
import pytest
import torch

from paper_2508_08540_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2508_08540_b200 import lsgd

    lsgd.lib()
    return lsgd


DRAWS = [
    # N, n_draw, n_exclude
    (1, 1, 0), (2, 1, 1), (5, 5, 0), (37, 10, 20), (4096, 1000, 96), (4097, 4097, 0), (4099, 2000, 2099),
    (50_000, 388, 0), (50_000, 388, 49_612), (50_000, 37_209, 12_403), (100_003, 100_003, 0), (262_147, 5, 262_000),
    (1_281_167, 256_233, 0), (1_281_167, 704_934, 320_000),
]


@pytest.mark.parametrize("N,m,nex", DRAWS)
def test_draw_matches_oracle(L, oracle, N, m, nex):
    seed, stream = 0x9E3779B97F4A7C15 ^ N, (m << 33) | 5  # 64-bit seed and stream: both halves are used
    excl = None
    if nex:
        excl = np.random.default_rng(N + m).permutation(N)[:nex].astype(np.int32)
    want = oracle.draw_uniform(N, m, seed, stream, excl)
    got = L.draw_uniform(N, m, seed, stream, torch.from_numpy(excl).cuda() if nex else None)
    np.testing.assert_array_equal(got.cpu().numpy(), want)


def test_draw_ignores_out_of_range_exclusions_and_reuses_a_workspace(L, oracle):
    N, m = 10_000, 3_000
    excl = np.array([5, -1, N, 2**31 - 1, 17, -(2**31)], dtype=np.int32)
    ws = L.workspace(L.draw_workspace_bytes(N, m))
    ws.fill_(0xFF)  # the workspace needs no initialisation
    out = torch.empty(m, dtype=torch.int32, device="cuda")
    for stream in (0, 1, 0):  # the same workspace, three calls in a row
        L.draw_uniform(N, m - 4, 77, stream, torch.from_numpy(excl).cuda(), out_idx=out[:m - 4], ws=ws)
        np.testing.assert_array_equal(out[:m - 4].cpu().numpy(), oracle.draw_uniform(N, m - 4, 77, stream, excl))


FAST = [
    # N, k_high, n_fill
    (1, 1, 0), (9, 4, 5), (4096, 1024, 3072), (4097, 0, 1500), (4097, 1500, 0), (10_001, 2_500, 7_000),
    (50_000, 12_403, 37_209), (50_000, 49_612, 0), (1_281_167, 320_000, 704_934),
]


@pytest.mark.parametrize("N,k,fill", FAST)
def test_fast_allocation_matches_oracle(L, oracle, N, k, fill):
    losses = wl.loss_like_vector(4000 + N, N, dup_frac=0.02, specials=N >= 16)
    want = oracle.fast_allocation(losses, k, fill, 20250808, N)
    ws = L.workspace(L.fast_allocation_workspace_bytes(N, k, fill))
    ws.fill_(0xA5)
    got = L.fast_allocation(torch.from_numpy(losses).cuda(), k, fill, 20250808, N, ws=ws).cpu().numpy()
    np.testing.assert_array_equal(got, want)
    assert np.unique(got).size == got.size
    # split over 8 fast workers: the shares are the oracle's ranges and cover the list once
    cuts = [L.worker_share(got.size, 8, p) for p in range(8)]
    assert cuts == [oracle.worker_share(got.size, 8, p) for p in range(8)]


def test_epoch_allocation_end_to_end(L, oracle):
    """One epoch's allocation for config 2's pool in the paper's setting (8 fast workers with tau_F = 32, 2 slow
    ones with tau_S = 1): scorer -> fast allocation on the GPU's own losses, slow draw on an independent stream,
    and the unified-sampling variant where the slow workers draw from what the fast workers left."""
    cfg = wl.CONFIGS[2]
    x, y = wl.pool_rows(cfg)
    nf, ns, k = L.allocation_sizes(cfg.N, 32, 8, 1, 2, 0.25)
    assert (nf, ns, k) == oracle.allocation_sizes(cfg.N, 32, 8, 1, 2, 0.25)
    losses = L.score_losses(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda())
    fast = L.fast_allocation(losses, k, nf - k, 1234, 10)
    slow = L.draw_uniform(cfg.N, ns, 1234, 11, device="cuda")
    unified = L.draw_uniform(cfg.N, ns, 1234, 11, exclude_idx=fast)
    lh = losses.cpu().numpy()
    np.testing.assert_array_equal(fast.cpu().numpy(), oracle.fast_allocation(lh, k, nf - k, 1234, 10))
    np.testing.assert_array_equal(slow.cpu().numpy(), oracle.draw_uniform(cfg.N, ns, 1234, 11))
    np.testing.assert_array_equal(unified.cpu().numpy(), oracle.draw_uniform(cfg.N, ns, 1234, 11, fast.cpu().numpy()))
    # unified sampling partitions the epoch: fast and slow allocations are disjoint and cover the pool
    assert np.array_equal(np.sort(np.concatenate([fast.cpu().numpy(), unified.cpu().numpy()])), np.arange(cfg.N))
    # every high-loss sample is at least as hard as every sample the selection left out (the GPU's own losses)
    sel = fast.cpu().numpy()[:k]
    rest = np.setdiff1d(np.arange(cfg.N), sel)
    assert lh[sel].min() >= lh[rest].max()


@pytest.mark.parametrize("cfg_id,lam", [(1, 1.0), (2, 0.5)])
def test_high_loss_to_slow_workers_variant(L, oracle, cfg_id, lam):
    """The appendix's other data allocation (table of data sampling methods, row "High-loss -> CPU"): the SLOW
    group takes the highest-loss samples, the fast group draws at random; with separated sampling the fast draw is
    independent, with unified sampling it comes from what the slow group left.  The library has no mode switch:
    the variant is the same three calls with the groups' sizes exchanged, and every list must match the oracle."""
    cfg = wl.scaled(wl.CONFIGS[cfg_id], N=20_011)
    x, y = wl.pool_rows(cfg)
    nf, ns, _ = L.allocation_sizes(cfg.N, 32, 8, 1, 2, lam)
    assert (nf, ns) == oracle.allocation_sizes(cfg.N, 32, 8, 1, 2, lam)[:2] and nf + ns == cfg.N
    k_slow = int(lam * ns)  # the high-loss part of the SLOW allocation
    losses = L.score_losses(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda())
    lh = losses.cpu().numpy()
    slow = L.fast_allocation(losses, k_slow, ns - k_slow, 99, 2)          # top-k_slow, then the random fill
    fast_separated = L.draw_uniform(cfg.N, nf, 99, 3, device="cuda")      # independent of the slow list
    fast_unified = L.draw_uniform(cfg.N, nf, 99, 3, exclude_idx=slow)     # from what the slow group left
    np.testing.assert_array_equal(slow.cpu().numpy(), oracle.fast_allocation(lh, k_slow, ns - k_slow, 99, 2))
    np.testing.assert_array_equal(fast_separated.cpu().numpy(), oracle.draw_uniform(cfg.N, nf, 99, 3))
    np.testing.assert_array_equal(fast_unified.cpu().numpy(), oracle.draw_uniform(cfg.N, nf, 99, 3, slow.cpu().numpy()))
    # the slow group's first k_slow samples are the hardest of the pool (the library's own losses, ties by index)
    np.testing.assert_array_equal(slow.cpu().numpy()[:k_slow], oracle.topk(lh, k_slow, oracle.LOSS_DESC)[0])
    # unified: the two groups partition the epoch; separated: the fast draw may overlap the slow list
    assert np.array_equal(np.sort(np.concatenate([slow.cpu().numpy(), fast_unified.cpu().numpy()])), np.arange(cfg.N))
    assert np.unique(fast_separated.cpu().numpy()).size == nf
    # split over the 2 slow and the 8 fast workers
    assert [L.worker_share(ns, 2, p) for p in range(2)] == [oracle.worker_share(ns, 2, p) for p in range(2)]
    assert [L.worker_share(nf, 8, p) for p in range(8)] == [oracle.worker_share(nf, 8, p) for p in range(8)]
