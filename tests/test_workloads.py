"""The synthetic input generators: position-addressable, seeded, right shapes."""
import numpy as np

from paper_2508_08540_b200 import workloads as wl


def test_pool_is_position_addressable():
    cfg = wl.scaled(wl.CONFIGS[2], N=30_000)  # C = 100: 10485 rows per keyed block, so 3 blocks
    full_x, full_y = wl.pool_rows(cfg)
    part_x, part_y = wl.pool_rows(cfg, 10_400, 21_111)
    np.testing.assert_array_equal(part_x, full_x[10_400:21_111])
    np.testing.assert_array_equal(part_y, full_y[10_400:21_111])
    one_x, one_y = wl.pool_samples(cfg, [0, 10_485, 29_999])
    np.testing.assert_array_equal(one_x, full_x[[0, 10_485, 29_999]])
    np.testing.assert_array_equal(one_y, full_y[[0, 10_485, 29_999]])
    assert full_x.dtype == np.float32 and full_x.shape == (30_000, 1, 100)
    assert 0 <= full_y.min() and full_y.max() < 100
    # N(0, 2) plus 1.0 on the true class
    assert abs(full_x.std() - 2.0) < 0.02
    true = np.take_along_axis(full_x[:, 0, :], full_y, axis=1)
    assert abs(true.mean() - 1.0) < 0.05


def test_sequence_pool_masks_and_bf16():
    cfg = wl.scaled(wl.CONFIGS[4], N=6, T=16, C=4096)
    x, y = wl.pool_rows(cfg)
    assert x.dtype == np.uint16 and x.shape == (6, 16, 4096) and y.shape == (6, 16)
    big = wl.scaled(wl.CONFIGS[4], N=64, T=128, C=8)
    _, yb = wl.pool_rows(big)
    frac = (yb == wl.IGNORE_INDEX).mean()
    assert 0.07 < frac < 0.13
    assert abs(wl.bf16_bits_to_f32(x).std() - 3.0) < 0.05


def test_duplicate_rows_are_exact_copies():
    cfg = wl.scaled(wl.CONFIGS[3], N=5_000)
    x, y = wl.pool_rows(cfg)
    dst, src = wl._dup_map(cfg)
    assert dst.size == 50 and not set(dst.tolist()) & set(src.tolist())
    np.testing.assert_array_equal(x[dst], x[src])
    np.testing.assert_array_equal(y[dst], y[src])
    px, py = wl.pool_rows(cfg, int(dst[0]), int(dst[0]) + 1)
    np.testing.assert_array_equal(px[0], x[dst[0]])


def test_replicas_and_weights():
    cfg = wl.scaled(wl.CONFIGS[1], D=(1 << 20) + 777)
    r3 = wl.replica_slice(cfg, 3)
    np.testing.assert_array_equal(wl.replica_slice(cfg, 3, 1_048_000, 1_049_000), r3[1_048_000:1_049_000])
    r4 = wl.replica_slice(cfg, 4)
    assert abs(r3.std() - 0.05) < 1e-3
    assert abs((r3 - r4).std() - np.sqrt(2) * 1e-3) < 1e-4
    w = wl.weight_draws(cfg)
    assert w.shape == (10,) and w.dtype == np.float32 and abs(w.sum() - 1) < 1e-6 and (w > 0).all()
    tau = wl.step_counts(wl.CONFIGS[5])
    assert tau.shape == (16,) and tau.min() >= 1 and tau.max() <= 64
    np.testing.assert_array_equal(tau, wl.step_counts(wl.CONFIGS[5]))
