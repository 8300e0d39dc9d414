"""Element-by-element parity of the CUDA library (through its C ABI) with the CPU
oracle on the same seeded inputs: small and ragged shapes, several tiles, edge
cases.  Tolerances (from the arithmetic: 2-ulp exponentials and a tree sum for the losses, a chain of P fused multiply-adds for Eq. 3):
  losses       |g - o| <= 1e-5 |o| + C 2^-52   (C 2^-52: the oracle's own double rounding when it sums C terms next to 1;
               losses below that floor are checked against the closed form log1p(sum_j!=y exp(x_j - x_y)) instead)
  aggregation  |g - o| <= 1e-6 * sum_i |w_i x_i[j]|  and  ||g - o||_2 <= 1e-6 ||o||_2
  top-k        indices and values bit-exact
"""
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


def dev_logits(x: np.ndarray) -> torch.Tensor:
    if x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(x).cuda()


def assert_losses_close(got: np.ndarray, want: np.ndarray, C: int):
    nan = np.isnan(want)
    np.testing.assert_array_equal(np.isnan(got), nan)
    err = np.abs(got[~nan].astype(np.float64) - want[~nan])
    tol = 1e-5 * np.abs(want[~nan]) + C * 2.0 ** -52
    bad = err > tol
    assert not bad.any(), f"{bad.sum()} losses off; worst rel {np.max(err / np.maximum(np.abs(want[~nan]), 1e-300)):.3e}"


def random_pool(seed, N, T, C, dtype, sigma=2.0, bump=1.0, mask_p=0.0):
    cfg = wl.RoundConfig(900 + seed, "t", 2, 8, "softmax", N, T, C, dtype, sigma, bump, mask_p, 0)
    return wl.pool_rows(cfg)


# --------------------------------------------------------------------------- #
# scorer
# --------------------------------------------------------------------------- #
SCORE_SHAPES = [
    # N, T, C, dtype            path
    (1, 1, 1, "f32"), (33, 1, 2, "f32"), (1000, 1, 3, "f32"), (777, 1, 7, "bf16"), (5000, 1, 10, "f32"),
    (300, 1, 32, "bf16"), (2000, 1, 4, "f32"), (1111, 1, 5, "bf16"), (999, 1, 12, "f32"), (640, 1, 16, "bf16"), (1500, 1, 20, "f32"),
    (901, 1, 24, "bf16"), (1300, 1, 28, "f32"), (77, 1, 31, "f32"),             # rows of at most 32 elements: one lane per row, in registers
    (500, 1, 33, "bf16"), (700, 1, 101, "bf16"), (400, 1, 104, "f32"), (300, 1, 105, "f32"), (1200, 1, 50, "bf16"), (900, 1, 52, "f32"),
    (2500, 1, 208, "bf16"), (1000, 1, 103, "f32"),                              # one lane per row out of shared memory, units of 16/8/4/2 bytes
    (31, 1, 33, "f32"), (2049, 1, 100, "f32"), (513, 1, 100, "bf16"),
    (1000, 1, 36, "f32"), (333, 2, 40, "bf16"), (4099, 1, 64, "f32"), (777, 1, 102, "f32"), (650, 1, 128, "bf16"),
    (129, 3, 128, "f32"), (1031, 1, 132, "f32"), (500, 1, 200, "f32"), (97, 2, 201, "f32"), (420, 1, 256, "f32"),
    (801, 1, 256, "bf16"), (65, 1, 255, "bf16"), (900, 1, 102, "bf16"), (211, 1, 300, "f32"), (150, 2, 512, "f32"),
    (300, 1, 1000, "bf16"), (77, 3, 1024, "bf16"), (190, 1, 450, "bf16"), (100, 1, 511, "f32"),
                                                                                 # lane groups: 16/8/4-byte rows or not, 4/8/16 lanes
    (257, 1, 1000, "f32"),
    (65, 3, 1016, "f32"), (40, 2, 2031, "bf16"), (129, 1, 999, "bf16"),          # warp rows, odd alignments
    (37, 1, 1017, "f32"), (19, 2, 2500, "f32"), (24, 3, 4099, "bf16"), (40, 1, 1500, "f32"), (33, 2, 3001, "bf16"),
    (9, 1, 8191, "f32"), (300, 1, 2048, "bf16"), (21, 1, 16384, "bf16"), (7, 2, 8000, "f32"),  # streamed rows (<= 32 KB)
    (6, 5, 30522, "bf16"),
    (5, 1, 50001, "f32"),
    (3, 2, 60011, "f32"), (2, 1, 120013, "bf16"),                                # the longest streamed rows
    (2, 1, 70001, "f32"), (3, 1, 140001, "bf16"),                                # beyond 256 KB: one CTA per row
]


@pytest.mark.parametrize("N,T,C,dtype", SCORE_SHAPES)
def test_score_matches_oracle(L, oracle, N, T, C, dtype):
    x, y = random_pool(C % 97, N, T, C, dtype, mask_p=0.15 if T > 1 else 0.0)
    want, bad = oracle.score(x, y)
    ws = L.workspace(L.score_workspace_bytes(N, T, C))
    got = L.score_losses(dev_logits(x), torch.from_numpy(y).cuda(), ws=ws)
    assert L.read_device_status(ws) == bad == 0
    assert_losses_close(got.cpu().numpy(), want, C)


@pytest.mark.parametrize("C,dtype", [(10, "f32"), (7, "bf16"), (32, "f32"), (32, "bf16"), (100, "f32"), (100, "bf16"), (101, "bf16"), (104, "f32"),
                                     (300, "bf16"), (1000, "bf16"), (5000, "f32"), (30522, "bf16")])
@pytest.mark.parametrize("off", [1, 2, 3, 4, 5])
def test_score_misaligned_base(L, oracle, C, dtype, off):
    # the pool starts `off` elements into an allocation: rows start at every 4-byte (2-byte) phase
    N = 41 if C > 1000 else 777
    x, y = random_pool(7, N, 1, C, dtype)
    flat = dev_logits(x).reshape(-1)
    buf = torch.zeros(flat.numel() + 8, dtype=flat.dtype, device="cuda")
    buf[off:off + flat.numel()] = flat
    view = buf[off:off + flat.numel()].view(N, C)
    want, _ = oracle.score(x, y)
    got = L.score_losses(view, torch.from_numpy(y).cuda())
    assert_losses_close(got.cpu().numpy(), want, C)


def test_score_closed_forms_and_small_losses(L, oracle):
    for C in (10, 100, 1000, 30522):
        x = torch.full((4, C), 0.7, device="cuda")
        y = torch.tensor([0, 1, C // 2, C - 1], device="cuda")
        got = L.score_losses(x, y).cpu().numpy()
        np.testing.assert_allclose(got, np.log(C), rtol=1e-5)
    # confident rows: losses from 1e-1 down to 1e-12 keep their relative accuracy
    for C in (8, 100, 1000, 2500, 6000):
        rows = []
        for gap in (2.0, 5.0, 10.0, 20.0, 30.0):
            r = np.random.default_rng(int(gap)).normal(0, 1, C).astype(np.float32)
            r[3] = r.max() + gap
            rows.append(r)
        x = np.stack(rows)
        y = np.full(len(rows), 3)
        want, _ = oracle.score(x, y)
        got = L.score_losses(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()).cpu().numpy()
        assert_losses_close(got, want, C)
        # the true class is the maximum here, so the loss has a cancellation-free closed form
        xd = x.astype(np.float64)
        exact = np.log1p(np.exp(np.delete(xd, 3, axis=1) - xd[:, 3:4]).sum(axis=1))
        np.testing.assert_allclose(got, exact, rtol=1e-5, atol=0)
        assert (got > 0).all()
    # huge logits stay finite; duplicated maxima
    x = np.array([[1e4, -1e4, 0, 0], [-1e4, 1e4, 0, 0], [1e4, 1e4, 1e4, -1e4], [9995.0, 1e4, 0, 0]], dtype=np.float32)
    y = np.array([1, 1, 0, 1])
    want, _ = oracle.score(x, y)
    got = L.score_losses(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()).cpu().numpy()
    assert_losses_close(got, want, 4)
    for C in (64, 3000, 9000):  # several copies of the maximum in the warp and CTA kernels
        x = np.zeros((2, C), dtype=np.float32)
        x[:, [5, C // 2, C - 1]] = 3.0
        y = np.array([5, 6])
        want, _ = oracle.score(x, y)
        got = L.score_losses(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()).cpu().numpy()
        assert_losses_close(got, want, C)


@pytest.mark.parametrize("C,dtype", [(10, "f32"), (32, "bf16"), (100, "f32"), (100, "bf16"), (500, "f32"), (1000, "bf16"), (5000, "f32"),
                                     (9000, "bf16"), (70_001, "f32")])
def test_score_at_the_documented_logit_bound(L, oracle, C, dtype):
    """Logits as large as the header allows (|x| <= 1e8; here +-2^26, exact in bf16), in every scorer kernel: ties at
    the top, the true class at the top, at the bottom and in between."""
    big = np.float32(2.0 ** 26)
    rng = np.random.default_rng(C)
    N = 64
    x = rng.choice(np.array([big, -big, big * np.float32(0.9921875), 0.0, 1.0, -3.0], np.float32), size=(N, C)).astype(np.float32)
    x[:, 0] = big                    # every row has the bound itself ...
    x[::2, C // 2] = big             # ... half of them twice
    y = rng.integers(0, C, N)
    y[:8] = 0                        # the true class is the maximum
    y[8:16] = C // 2
    xs = wl.f32_to_bf16_bits(x) if dtype == "bf16" else x
    want, bad = oracle.score(xs, y)
    assert bad == 0 and np.isfinite(want).all()
    got = L.score_losses(dev_logits(xs), torch.from_numpy(y).cuda()).cpu().numpy()
    assert_losses_close(got, want, C)


@pytest.mark.parametrize("C,dtype", [(10, "f32"), (40, "bf16"), (100, "f32"), (102, "bf16"), (500, "f32"), (1000, "bf16"),
                                     (1500, "f32"), (5000, "bf16"), (30522, "bf16"), (70001, "f32")])
@pytest.mark.parametrize("off", [0, 1, 3])
def test_score_true_class_anywhere_confident_or_not(L, oracle, C, dtype, off):
    """The true class is the one term every kernel leaves out of its sum: put it at the row's ends (the partial
    vectors of unaligned rows), next to them and in the middle, as the dominant class, as a runner-up, tied with the
    maximum, and far below it."""
    ys = sorted({0, 1, 2, 3, 7, 8, C // 2, C - 9, C - 8, C - 4, C - 3, C - 2, C - 1} & set(range(C)))
    rows, labels = [], []
    rng = np.random.default_rng(C + off)
    for y in ys:
        for kind in range(4):
            r = rng.normal(0, 2, C).astype(np.float32)
            top = float(r.max())
            if kind == 0:
                r[y] = top + 12.0      # dominant: a loss of about 1e-4, relative accuracy needed
            elif kind == 1:
                r[y] = top - 0.5       # runner-up
            elif kind == 2:
                r[y] = top             # tied with the maximum (unless y already is the maximum)
            else:
                r[y] = top - 30.0      # hopeless
            rows.append(r)
            labels.append(y)
    x = np.stack(rows)
    y = np.array(labels, dtype=np.int64)
    if dtype == "bf16":
        x = wl.f32_to_bf16_bits(x)
    want, bad = oracle.score(x, y)
    assert bad == 0
    flat = dev_logits(x).reshape(-1)
    buf = torch.zeros(flat.numel() + 8, dtype=flat.dtype, device="cuda")
    buf[off:off + flat.numel()] = flat
    got = L.score_losses(buf[off:off + flat.numel()].view(len(rows), C), torch.from_numpy(y).cuda()).cpu().numpy()
    assert_losses_close(got, want, C)
    # dominant rows: the cancellation-free closed form, to 1e-5 relative whatever the oracle's own floor
    xd = (wl.bf16_bits_to_f32(x) if dtype == "bf16" else x).astype(np.float64)
    dom = np.arange(0, len(rows), 4)
    others = np.array([np.exp(np.delete(xd[i], y[i]) - xd[i, y[i]]).sum() for i in dom])
    np.testing.assert_allclose(got[dom], np.log1p(others), rtol=1e-5, atol=0)


@pytest.mark.parametrize("C,dtype", [(10, "f32"), (100, "f32"), (5000, "bf16")])
def test_score_masks_bad_labels_and_sequences(L, oracle, C, dtype):
    N, T = 9, 6
    x, y = random_pool(11, N, T, C, dtype, mask_p=0.3)
    y[2, :] = -100          # a sample with every token ignored scores 0
    y[4, 1] = C             # out of range: NaN, counted
    y[5, 0] = -7
    want, bad = oracle.score(x, y)
    ws = L.workspace(L.score_workspace_bytes(N, T, C))
    got = L.score_losses(dev_logits(x), torch.from_numpy(y).cuda(), ws=ws).cpu().numpy()
    assert bad == 2 and L.read_device_status(ws) == 2
    assert got[2] == 0.0 and np.isnan(got[4]) and np.isnan(got[5])
    assert_losses_close(got, want, C)
    # T = 1 with ignored labels
    x1, y1 = random_pool(12, 50, 1, C, dtype)
    y1[::7] = -100
    want1, _ = oracle.score(x1, y1)
    got1 = L.score_losses(dev_logits(x1), torch.from_numpy(y1).cuda()).cpu().numpy()
    assert (got1[::7] == 0).all()
    assert_losses_close(got1, want1, C)


def test_score_is_position_independent_and_deterministic(L):
    # identical rows at different positions give identical bits (16-byte-aligned rows: C = 100, 1000 fp32)
    for C in (100, 1000, 6000):
        r = torch.randn(C, device="cuda", generator=torch.Generator("cuda").manual_seed(C))
        x = r.repeat(777, 1).contiguous()
        y = torch.full((777,), 5, device="cuda")
        a = L.score_losses(x, y)
        assert (a == a[0]).all()
        b = L.score_losses(x, y)
        assert torch.equal(a, b)


# --------------------------------------------------------------------------- #
# selector
# --------------------------------------------------------------------------- #
TOPK_CASES = [(1, 1), (2, 1), (31, 30), (1000, 1), (1000, 1000), (4096, 777), (4097, 1), (4097, 4097), (5000, 4999),
              (50_000, 12_500), (50_000, 5_000), (70_001, 35_000), (300_000, 299_999), (1_000_003, 250_000)]


@pytest.mark.parametrize("N,k", TOPK_CASES)
@pytest.mark.parametrize("order", [0, 1])
def test_topk_bit_exact(L, oracle, N, k, order):
    v = wl.loss_like_vector(N + k, N, dup_frac=0.01, specials=True)
    want_idx, want_vals = oracle.topk(v, k, order)
    idx, vals = L.topk_select(torch.from_numpy(v).cuda(), k, order)
    np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
    np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))


@pytest.mark.parametrize("N", [3000, 40_000])
def test_topk_ties_straddle_the_cut(L, oracle, N):
    rng = np.random.default_rng(N)
    v = rng.gamma(2.0, 1.0, N).astype(np.float32)
    k = N // 4
    kth = np.sort(v)[::-1][k - 1]
    pos = rng.permutation(N)[:64]
    v[pos] = kth  # 64 extra copies of the k-th value, on both sides of any cut
    for order in (0, 1):
        for kk in (k - 20, k, k + 20):
            want_idx, _ = oracle.topk(v, kk, order)
            idx, _ = L.topk_select(torch.from_numpy(v).cuda(), kk, order)
            np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
    # all equal: the k lowest indices
    same = torch.full((N,), 0.25, device="cuda")
    idx, _ = L.topk_select(same, 100, 0)
    assert idx.cpu().tolist() == list(range(100))
    # strictly increasing: the last k, reversed
    inc = torch.arange(N, device="cuda", dtype=torch.float32)
    idx, _ = L.topk_select(inc, 5, 0)
    assert idx.cpu().tolist() == [N - 1, N - 2, N - 3, N - 4, N - 5]


def test_topk_zero_k_and_no_vals(L):
    v = torch.rand(10_000, device="cuda")
    idx, vals = L.topk_select(v, 0)
    assert idx.numel() == 0
    idx, vals = L.topk_select(v, 10, want_vals=False)
    assert vals is None and idx.cpu().tolist() == torch.topk(v, 10).indices.cpu().tolist()


def test_topk_guards_stay_untouched(L, oracle):
    # outputs and workspace sit between sentinel pads that must come back unchanged
    N, k = 123_457, 30_001
    v = wl.loss_like_vector(5, N)
    pad = 1024
    out = torch.full((k + 2 * pad,), -7, dtype=torch.int32, device="cuda")
    vals = torch.full((k + 2 * pad,), -7.0, dtype=torch.float32, device="cuda")
    need = L.topk_workspace_bytes(N, k)
    wsbuf = torch.full((need + 2 * 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    ws = wsbuf[4096:4096 + need]
    L.topk_select(torch.from_numpy(v).cuda(), k, 0, out_idx=out[pad:pad + k], out_vals=vals[pad:pad + k], ws=ws)
    torch.cuda.synchronize()
    assert (out[:pad] == -7).all() and (out[pad + k:] == -7).all()
    assert (vals[:pad] == -7).all() and (vals[pad + k:] == -7).all()
    assert (wsbuf[:4096] == 0x5A).all() and (wsbuf[4096 + need:] == 0x5A).all()
    np.testing.assert_array_equal(out[pad:pad + k].cpu().numpy(), oracle.topk(v, k, 0)[0])


# --------------------------------------------------------------------------- #
# fused scorer + selector
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("N,T,C,dtype,k", [(3000, 1, 10, "f32", 750), (20_000, 1, 100, "f32", 5000),
                                           (9000, 1, 1000, "bf16", 2000), (4500, 2, 300, "f32", 4500),
                                           (700, 4, 5000, "bf16", 99), (5000, 1, 4100, "f32", 1234)])
@pytest.mark.parametrize("order", [0, 1])
def test_score_topk_equals_the_two_calls_and_the_oracle(L, oracle, N, T, C, dtype, k, order):
    x, y = random_pool(3, N, T, C, dtype, mask_p=0.1 if T > 1 else 0.0)
    xd, yd = dev_logits(x), torch.from_numpy(y).cuda()
    losses, idx, vals = L.score_topk(xd, yd, k, order)
    sep_losses = L.score_losses(xd, yd)
    sep_idx, sep_vals = L.topk_select(sep_losses, k, order)
    assert torch.equal(losses, sep_losses) and torch.equal(idx, sep_idx) and torch.equal(vals, sep_vals)
    # the selector is exact on the library's own losses
    g = losses.cpu().numpy()
    want_idx, _ = oracle.topk(g, k, order)
    np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
    # end to end against the oracle's losses: selected >= unselected - 1e-5 * max(1, |threshold|)
    o, _ = oracle.score(x, y)
    assert_losses_close(g, o, C)
    sel = np.zeros(N, bool)
    sel[idx.cpu().numpy()] = True
    if 0 < k < N:
        thr = o[sel].min()
        assert thr >= o[~sel].max() - 1e-5 * max(1.0, abs(thr))


# --------------------------------------------------------------------------- #
# aggregation
# --------------------------------------------------------------------------- #
def assert_aggregate_close(got, out64, mag):
    err = np.abs(got.astype(np.float64) - out64)
    assert (err <= 1e-6 * mag + 1e-45).all(), f"worst {np.max(err / np.maximum(mag, 1e-300)):.3e}"
    assert np.linalg.norm(err) <= 1e-6 * np.linalg.norm(out64) + 1e-45


@pytest.mark.parametrize("P", [1, 2, 3, 10, 16, 17, 33, 64])
@pytest.mark.parametrize("D", [1, 3, 4, 5, 1023, 272_474, 1_000_003])
def test_aggregate_matches_oracle(L, oracle, P, D):
    cfg = wl.RoundConfig(800 + P, "t", P, D, "softmax", 1, 1, 2, "f32", 1, 0, 0, 0)
    reps = [wl.replica_slice(cfg, i) for i in range(P)]
    w = wl.weight_draws(cfg)
    out64, _, mag = oracle.aggregate(reps, w)
    got = L.aggregate([torch.from_numpy(r).cuda() for r in reps], w.tolist()).cpu().numpy()
    assert_aggregate_close(got, out64, mag)


def test_aggregate_special_weights_and_in_place(L, oracle):
    P, D = 10, 100_003
    cfg = wl.RoundConfig(850, "t", P, D, "softmax", 1, 1, 2, "f32", 1, 0, 0, 0)
    reps = [wl.replica_slice(cfg, i) for i in range(P)]
    dev = [torch.from_numpy(r).cuda() for r in reps]
    for i in (0, 4, 9):  # one-hot weight: that replica, bit for bit
        w = [0.0] * P
        w[i] = 1.0
        assert torch.equal(L.aggregate(dev, w), dev[i])
    # step-count weights of the paper's (32, 1) setting, and equal steps = plain mean
    for tau in ([32] * 8 + [1] * 2, [5] * 10):
        w = L.weights_from_steps(tau)
        np.testing.assert_array_equal(np.array(w, np.float32), oracle.weights_from_steps(tau))
        out64, _, mag = oracle.aggregate(reps, np.array(w, np.float32))
        assert_aggregate_close(L.aggregate(dev, w).cpu().numpy(), out64, mag)
    # identical replicas with weights summing to 1 reproduce the replica
    got = L.aggregate([dev[0]] * 4, [0.5, 0.25, 0.125, 0.125])
    np.testing.assert_allclose(got.cpu().numpy(), reps[0], rtol=4 * 2.0 ** -24, atol=0)  # P roundings of the fp32 chain
    # in place: out is exactly replica 3
    w = wl.weight_draws(cfg)
    out64, _, mag = oracle.aggregate(reps, w)
    target = dev[3].clone()
    L.aggregate(dev[:3] + [target] + dev[4:], w.tolist(), out=target)
    assert_aggregate_close(target.cpu().numpy(), out64, mag)
    # weights are used as given: not normalised
    got = L.aggregate(dev[:2], [2.0, -1.0]).cpu().numpy()
    o64, _, m = oracle.aggregate(reps[:2], np.array([2.0, -1.0], np.float32))
    assert_aggregate_close(got, o64, m)


@pytest.mark.parametrize("off", [1, 2, 3])
def test_aggregate_misaligned_and_guards(L, oracle, off):
    P, D = 5, 70_001
    cfg = wl.RoundConfig(860, "t", P, D, "softmax", 1, 1, 2, "f32", 1, 0, 0, 0)
    reps = [wl.replica_slice(cfg, i) for i in range(P)]
    w = wl.weight_draws(cfg)
    dev = []
    for i, r in enumerate(reps):
        buf = torch.zeros(D + 8, device="cuda")
        o = off if i % 2 == 0 else 0
        buf[o:o + D] = torch.from_numpy(r).cuda()
        dev.append(buf[o:o + D])
    pad = 256
    outbuf = torch.full((D + 2 * pad + 4,), -7.0, device="cuda")
    out = outbuf[pad + off:pad + off + D]
    L.aggregate(dev, w.tolist(), out=out)
    out64, _, mag = oracle.aggregate(reps, w)
    assert_aggregate_close(out.cpu().numpy(), out64, mag)
    assert (outbuf[:pad + off] == -7).all() and (outbuf[pad + off + D:] == -7).all()


def test_errors_raise(L):
    x = torch.zeros(4, 10, device="cuda")
    y = torch.zeros(4, dtype=torch.int64, device="cuda")
    with pytest.raises(L.LsgdError) as e:
        L.score_losses(x, y, ws=torch.empty(256, dtype=torch.uint8, device="cuda")[:16])
    assert e.value.status in (L.ERR_WORKSPACE, L.ERR_ALIGNMENT)
    with pytest.raises(L.LsgdError):
        L.topk_select(torch.zeros(10, device="cuda"), 11)
    with pytest.raises(L.LsgdError):
        L.aggregate([torch.zeros(8, device="cuda")] * 65, [0.0] * 65)
    # a failed call leaves the context usable
    assert L.score_losses(x, y).shape == (4,)


def test_score_random_shapes_offsets_and_masks(L, oracle):
    """A seeded sweep over row lengths of every kernel's range, both types, pools starting at every element offset
    inside an allocation, ignored and out-of-range labels: every loss against the oracle."""
    rng = np.random.default_rng(20250808)
    lengths = list(range(1, 40)) + [rng.integers(40, 210) for _ in range(40)] + [rng.integers(210, 1100) for _ in range(25)] + \
              [int(x) for x in rng.integers(1100, 9000, 8)]
    for case, C in enumerate(lengths):
        C = int(C)
        dtype = "bf16" if case % 2 else "f32"
        N = int(rng.integers(1, 400 if C < 1100 else 60))
        T = 1 if case % 5 else 3
        off = int(rng.integers(0, 8))
        x, y = random_pool(1000 + case, N, T, C, dtype, sigma=float(rng.choice([0.5, 2.0, 8.0])), bump=float(rng.choice([0.0, 3.0])),
                           mask_p=0.2 if T > 1 else 0.0)
        y = y.copy()
        if case % 7 == 0:
            y.reshape(-1)[rng.integers(0, y.size)] = C + 5  # one label out of range
        flat = dev_logits(x).reshape(-1)
        buf = torch.zeros(flat.numel() + 8, dtype=flat.dtype, device="cuda")
        buf[off:off + flat.numel()] = flat
        view = buf[off:off + flat.numel()].view(N, T, C)
        want, bad = oracle.score(x, y)
        ws = L.workspace(L.score_workspace_bytes(N, T, C))
        got = L.score_losses(view, torch.from_numpy(y).cuda(), ws=ws).cpu().numpy()
        assert L.read_device_status(ws) == bad, (case, C, dtype, N, T, off)
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan), (case, C, dtype, N, T, off)
        err = np.abs(got[~nan].astype(np.float64) - want[~nan])
        assert (err <= 1e-5 * np.abs(want[~nan]) + C * 2.0 ** -52).all(), (case, C, dtype, N, T, off, float(err.max()))


@pytest.mark.parametrize("N", [500, 5_000, 100_000])
def test_fused_call_reports_bad_labels_and_a_selection_alone_reports_none(L, oracle, N):
    """The status block after lsgd_score_topk carries the scorer's count through every selector variant (one block,
    one cluster, cooperative); after a selection on its own it reads zero, whatever the workspace held before."""
    C = 10
    x, y = random_pool(5, N, 1, C, "f32")
    y = y.copy()
    y[[1, N // 2, N - 1]] = C + 1
    xd, yd = dev_logits(x), torch.from_numpy(y).cuda()
    k = N // 4
    ws = L.workspace(L.score_topk_workspace_bytes(N, 1, C, k))
    ws.fill_(0xFF)
    losses, idx, _ = L.score_topk(xd, yd, k, L.ORDER_LOSS_DESC, ws=ws)
    assert L.read_device_status(ws) == 3
    g = losses.cpu().numpy()
    assert np.isnan(g).sum() == 3
    np.testing.assert_array_equal(idx.cpu().numpy(), oracle.topk(g, k, oracle.LOSS_DESC)[0])  # NaN ranks highest
    ws.fill_(0xFF)
    idx2, _ = L.topk_select(losses, k, L.ORDER_LOSS_DESC, ws=ws)
    assert L.read_device_status(ws) == 0
    assert torch.equal(idx, idx2)
