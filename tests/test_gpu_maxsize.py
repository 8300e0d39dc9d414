"""The sizes at which 32-bit index arithmetic would wrap: Eq. 3 over more than 2^31 parameters, the selector on a
loss table of 2^31 - 1 entries (the largest the header admits), the scorer on more than 2^31 token rows.

Whole-input oracle runs are out of reach at these sizes, so each test checks, against the oracle, windows of the
output placed where an index or a byte offset crosses 2^31, 2^32 or 2^33 (and the two ends), plus a property that
holds at any size and covers every element (a one-hot weight reproduces its replica bit for bit; the selected set
is exactly the planted entries).  Inputs are made on the device in slabs.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def L():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2508_08540_b200 import lsgd

    lsgd.lib()
    return lsgd


def need_free_gb(gb):
    free, _ = torch.cuda.mem_get_info()
    if free < gb * (1 << 30):
        pytest.skip(f"needs {gb} GB of free device memory")


def fill_normal(t, seed, sigma=1.0, slab=1 << 28):
    g = torch.Generator(device="cuda").manual_seed(seed)
    flat = t.view(-1)
    for a in range(0, flat.numel(), slab):
        b = min(flat.numel(), a + slab)
        flat[a:b] = (torch.randn(b - a, device="cuda", generator=g) * sigma).to(t.dtype)


def windows(total, marks, half):
    """[a, b) ranges of `half` elements either side of each mark, clipped to [0, total), plus both ends."""
    out = [(0, min(total, 2 * half)), (max(0, total - 2 * half), total)]
    out += [(max(0, m - half), min(total, m + half)) for m in marks if 0 < m < total]
    return out


def test_aggregate_beyond_2_to_31_parameters(L, oracle):
    """Eq. 3 with D = 2^31 + 7 (element indices beyond int32, byte offsets beyond 2^33, a ragged tail of three)."""
    need_free_gb(30)
    D = (1 << 31) + 7
    reps = [torch.empty(D, dtype=torch.float32, device="cuda") for _ in range(2)]
    for i, r in enumerate(reps):
        fill_normal(r, 4100 + i, 0.05)
    w = [0.75, 0.5]
    out = torch.full((D,), float("nan"), dtype=torch.float32, device="cuda")
    L.aggregate(reps, w, out=out)
    torch.cuda.synchronize()
    for a, b in windows(D, [1 << 30, 1 << 31, (1 << 31) + (1 << 30) // 2], 4096):
        xs = [r[a:b].cpu().numpy() for r in reps]
        want, _, mag = oracle.aggregate(xs, np.array(w, dtype=np.float32))
        got = out[a:b].cpu().numpy().astype(np.float64)
        assert (np.abs(got - want) <= 1e-6 * mag + 1e-45).all(), (a, b)
    # a one-hot weight reproduces that replica bit for bit, over the whole vector
    L.aggregate(reps, [0.0, 1.0], out=out)
    for a in range(0, D, 1 << 29):
        b = min(D, a + (1 << 29))
        assert torch.equal(out[a:b], reps[1][a:b]), (a, b)
    del reps, out
    torch.cuda.empty_cache()


def test_topk_on_the_largest_table(L, oracle):
    """N = 2^31 - 1 losses (8 GiB).  Every entry lies in [0, 1) except some 1,500 planted ones above 1 (at both ends, either
    side of 2^30, in runs and scattered, with a group of equal values that the cut of k = 1,000 divides), so the
    selection is the oracle's selection among the planted entries, mapped back to their positions."""
    need_free_gb(14)
    N = (1 << 31) - 1
    losses = torch.empty(N, dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(77)
    for a in range(0, N, 1 << 28):
        b = min(N, a + (1 << 28))
        losses[a:b] = torch.rand(b - a, device="cuda", generator=g)
    rng = np.random.default_rng(5)
    pos = np.unique(np.concatenate([
        np.array([0, 1, 2, N - 1, N - 2, (1 << 30) - 1, 1 << 30, (1 << 30) + 1], dtype=np.int64),
        np.arange((1 << 30) + (1 << 29), (1 << 30) + (1 << 29) + 200, dtype=np.int64),
        rng.integers(0, N, size=1292, dtype=np.int64)]))
    vals = (1.0 + rng.random(pos.size) * 9.0).astype(np.float32)
    k = 1000
    cut = np.sort(vals)[::-1][k - 1]
    tied = rng.choice(pos.size, size=16, replace=False)
    vals[tied] = cut                       # sixteen equal values at the cut: some selected, some not
    losses[torch.from_numpy(pos).cuda()] = torch.from_numpy(vals).cuda()
    ws = L.workspace(L.topk_workspace_bytes(N, k))
    for order, o_order in ((L.ORDER_LOSS_DESC, oracle.LOSS_DESC), (L.ORDER_INDEX_ASC, oracle.INDEX_ASC)):
        want_sub, want_vals = oracle.topk(vals, k, o_order)   # pos ascends, so ties keep their order by index
        idx, got_vals = L.topk_select(losses, k, order, ws=ws)
        assert L.read_device_status(ws) == 0
        np.testing.assert_array_equal(idx.cpu().numpy().astype(np.int64), pos[want_sub])
        np.testing.assert_array_equal(got_vals.cpu().numpy(), want_vals)
    # all planted entries and the first of the rest: k beyond them, where the whole table decides
    k2 = pos.size + 3
    idx, got_vals = L.topk_select(losses, k2, L.ORDER_LOSS_DESC, ws=L.workspace(L.topk_workspace_bytes(N, k2)))
    idx = idx.cpu().numpy().astype(np.int64)
    want_sub, _ = oracle.topk(vals, pos.size, oracle.LOSS_DESC)
    np.testing.assert_array_equal(idx[:pos.size], pos[want_sub])
    losses[torch.from_numpy(pos).cuda()] = -1.0   # what is left: the three largest of the unplanted entries
    rest = got_vals[pos.size:].cpu().numpy()
    top = 0.0
    for a in range(0, N, 1 << 28):
        top = max(top, float(losses[a:min(N, a + (1 << 28))].max()))
    assert rest[0] == np.float32(top) and (np.diff(rest) <= 0).all()
    assert (losses[torch.from_numpy(idx[pos.size:]).cuda()].cpu().numpy() == rest).all()
    del losses
    torch.cuda.empty_cache()


def test_scorer_beyond_2_to_31_token_rows(L, oracle):
    """N x T = 1,048,579 x 2,049 = 2,148,538,371 token rows of two bf16 classes (row indices beyond int32; the token
    losses alone are 8 GiB), a tenth of the tokens ignored: the sequences at both ends and those around row 2^31
    against the oracle, and every loss of the pool inside the range two classes allow."""
    need_free_gb(40)
    N, T, C = (1 << 20) + 3, 2049, 2
    logits = torch.empty((N, T, C), dtype=torch.bfloat16, device="cuda")
    fill_normal(logits, 9001, 2.0)
    labels = torch.empty((N, T), dtype=torch.int64, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(9002)
    flat = labels.view(-1)
    for a in range(0, flat.numel(), 1 << 27):
        b = min(flat.numel(), a + (1 << 27))
        y = torch.randint(0, C, (b - a,), device="cuda", generator=g)
        y[torch.rand(b - a, device="cuda", generator=g) < 0.1] = -100
        flat[a:b] = y
    labels[5, :] = -100  # a sequence with every token ignored scores 0
    ws = L.workspace(L.score_workspace_bytes(N, T, C))
    got = L.score_losses(logits, labels, ws=ws)
    assert L.read_device_status(ws) == 0
    mid = (1 << 31) // T
    for a, b in windows(N, [mid], 48):
        x = logits[a:b].view(torch.int16).cpu().numpy().view(np.uint16)
        want, bad = oracle.score(x, labels[a:b].cpu().numpy())
        assert bad == 0
        g_ = got[a:b].cpu().numpy().astype(np.float64)
        assert (np.abs(g_ - want) <= 1e-5 * np.abs(want) + C * 2.0 ** -52).all(), (a, b)
    assert float(got[5]) == 0.0
    # a mean of 1,844 softplus values of N(0, 2.8) differences: every sample's loss is finite and near 1.3
    assert bool(torch.isfinite(got).all()) and 0.9 < float(got[6:].min()) and float(got.max()) < 1.8
    del logits, labels, ws
    torch.cuda.empty_cache()
