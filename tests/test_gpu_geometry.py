"""Stand-ins for a memory checker and a race detector.

  * Launch geometry must not change a single bit: every scorer kernel and the selector are run with their
    default grid and again with the thread-block count capped (and, for the selector, with the single-cluster
    variant switched off), through the library's test hooks; outputs must be bit-identical and equal the oracle's
    selection.  A race or an order that depends on which block ran first would show up here.
  * Outputs and workspaces sit between 4 KiB sentinel pads that must come back untouched: the scorer's loss
    table and its token-loss workspace, the fused call's workspace, and the round aggregation's outputs.
"""
import os
from contextlib import contextmanager

import numpy as np
import pytest
import torch

from paper_2508_08540_b200 import workloads as wl

pytestmark = pytest.mark.gpu

PAD = 4096  # bytes of sentinel on each side


@pytest.fixture(scope="module")
def L():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2508_08540_b200 import lsgd

    lsgd.lib()
    return lsgd


@contextmanager
def geometry(max_ctas=None, no_cluster=False, narrow_cluster=False):
    """The library reads these at every launch; they change grid sizes only."""
    old = {k: os.environ.get(k) for k in ("LSGD_TEST_MAX_CTAS", "LSGD_TEST_NO_CLUSTER", "LSGD_TEST_NARROW_CLUSTER")}
    try:
        if max_ctas is not None:
            os.environ["LSGD_TEST_MAX_CTAS"] = str(max_ctas)
        if no_cluster:
            os.environ["LSGD_TEST_NO_CLUSTER"] = "1"
        if narrow_cluster:
            os.environ["LSGD_TEST_NARROW_CLUSTER"] = "1"
        yield
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


def dev_logits(x):
    return torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16) if x.dtype == np.uint16 else torch.from_numpy(x).cuda()


def pool(seed, N, T, C, dtype, mask_p=0.0):
    cfg = wl.RoundConfig(700 + seed, "g", 2, 8, "softmax", N, T, C, dtype, 2.0, 1.0, mask_p, 0)
    return wl.pool_rows(cfg)


def guarded(nbytes, fill=0x5A):
    """(whole buffer, the nbytes in its middle), the rest filled with a sentinel; offsets are multiples of 256."""
    buf = torch.full((nbytes + 2 * PAD,), fill, dtype=torch.uint8, device="cuda")
    return buf, buf[PAD:PAD + nbytes]


def pads_intact(buf, nbytes, fill=0x5A):
    return bool((buf[:PAD] == fill).all()) and bool((buf[PAD + nbytes:] == fill).all())


# one shape per scorer kernel, each several tiles with a ragged tail
SCORER_SHAPES = [(20_011, 1, 10, "f32"), (9_001, 1, 32, "bf16"), (30_011, 1, 100, "f32"), (20_003, 1, 100, "bf16"), (7_001, 1, 101, "bf16"),
                 (6_007, 1, 103, "f32"),
                 (5_003, 1, 200, "f32"), (4_001, 1, 1000, "bf16"), (3_001, 1, 5000, "f32"), (257, 4, 30_522, "bf16"),
                 (37, 1, 70_001, "f32")]


@pytest.mark.parametrize("N,T,C,dtype", SCORER_SHAPES)
def test_scorer_bits_do_not_depend_on_the_grid(L, oracle, N, T, C, dtype):
    x, y = pool(C % 89, N, T, C, dtype, mask_p=0.1 if T > 1 else 0.0)
    xd, yd = dev_logits(x), torch.from_numpy(y).cuda()
    ref = L.score_losses(xd, yd)
    for cap in (1, 3, 37):
        with geometry(max_ctas=cap):
            got = L.score_losses(xd, yd)
        assert torch.equal(got.view(torch.int32), ref.view(torch.int32)), f"losses change with {cap} thread blocks"
    want, _ = oracle.score(x, y)
    g = ref.cpu().numpy()
    assert (np.abs(g - want) <= 1e-5 * np.abs(want) + C * 2.0 ** -52).all()


@pytest.mark.parametrize("N,k", [(1500, 700), (8192, 8192), (8193, 100), (50_000, 12_500), (65_536, 40_000), (65_537, 30_000),
                                 (300_007, 100_003), (1_281_167, 320_000)])
@pytest.mark.parametrize("order", [0, 1])
def test_selector_is_the_same_in_every_geometry(L, oracle, N, k, order):
    h = wl.loss_like_vector(N ^ k, N, dup_frac=0.02, specials=True)
    v = torch.from_numpy(h).cuda()
    want_idx, want_vals = oracle.topk(h, k, order)
    runs = [dict(), dict(narrow_cluster=True), dict(no_cluster=True), dict(max_ctas=3), dict(max_ctas=1), dict(max_ctas=8),
            dict(no_cluster=True, max_ctas=5), dict(no_cluster=True, max_ctas=1)]
    for kw in runs:
        with geometry(**kw):
            idx, vals = L.topk_select(v, k, order)
        np.testing.assert_array_equal(idx.cpu().numpy(), want_idx, err_msg=str(kw))
        np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32), err_msg=str(kw))


def test_selector_sort_pass_counts(L, oracle):
    """The loss-descending sort runs as many 9-bit passes as the selected keys' range needs: none (all selected
    losses equal), one, two, three and four."""
    N, k = 40_000, 9_000
    rng = np.random.default_rng(9)
    base = np.float32(1.0)
    for bits in (0, 5, 14, 23, 31):
        lo = base.view(np.uint32)
        off = rng.integers(0, 1 << bits, N, dtype=np.uint64).astype(np.uint32) if bits else np.zeros(N, np.uint32)
        h = (lo + off).astype(np.uint32).view(np.float32).copy()
        h[rng.permutation(N)[:k // 2]] = h.max()  # many ties at the top as well
        if bits == 31:
            h[:100] = -h[:100]
            h[100:110] = np.nan
        h = np.where(np.isfinite(h) | np.isnan(h), h, np.float32(3.0)).astype(np.float32)
        v = torch.from_numpy(h).cuda()
        for kw in (dict(), dict(narrow_cluster=True), dict(no_cluster=True)):
            with geometry(**kw):
                idx, vals = L.topk_select(v, k, L.ORDER_LOSS_DESC)
            want_idx, want_vals = oracle.topk(h, k, oracle.LOSS_DESC)
            np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
            np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))


def test_selector_when_the_candidates_outnumber_the_selection(L, oracle):
    """Loss-descending output of pools of up to 65,536 entries sorts every key that shares the k-th key's leading 22
    (or, where that leaves few enough, 11) bits or lies above them, and keeps the first k.  Pools where those candidates are far more than k, up to the
    whole pool (every count then sits at the limit of the 16-bit halves the blocks exchange), in sorted and reversed
    order (all candidates in the last or the first block), in the wide and the narrow cluster and without one."""
    rng = np.random.default_rng(65)
    N = 65_536
    pools = {
        "all equal": np.full(N, 1.75, np.float32),
        "two values": np.where(rng.random(N) < 0.5, np.float32(2.0), np.float32(2.0000002)).astype(np.float32),
        "37 values": rng.choice(rng.gamma(2.0, 1.0, 37).astype(np.float32), N),
        "within 1024 keys": (np.float32(3.0).view(np.uint32) + rng.integers(0, 1024, N).astype(np.uint32)).view(np.float32),
        "ascending": np.sort(rng.gamma(2.0, 1.0, N).astype(np.float32)),
        "descending": np.sort(rng.gamma(2.0, 1.0, N).astype(np.float32))[::-1].copy(),
    }
    for name, h in pools.items():
        v = torch.from_numpy(h).cuda()
        for k in (1, 100, 16_384, 40_000, N):
            want_idx, want_vals = oracle.topk(h, k, oracle.LOSS_DESC)
            for kw in (dict(), dict(narrow_cluster=True), dict(no_cluster=True)):
                with geometry(**kw):
                    idx, vals = L.topk_select(v, k, L.ORDER_LOSS_DESC)
                np.testing.assert_array_equal(idx.cpu().numpy(), want_idx, err_msg=f"{name} k={k} {kw}")
                np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32), err_msg=f"{name} k={k} {kw}")
    # the same through the fused call (the scorer's histogram resolves the first digit): identical rows score identical bits
    for N2, C in ((65_536, 10), (50_001, 7)):
        row = rng.normal(0, 2, C).astype(np.float32)
        x = np.tile(row, (N2, 1))
        x[N2 // 3] += 1.0  # two rows that differ, so that the pool is not one value only
        x[N2 - 5] -= 1.0
        y = np.full((N2, 1), 3, np.int64)
        d_x, d_y = torch.from_numpy(x).cuda().view(N2, 1, C), torch.from_numpy(y).cuda()
        for k in (1, 3, 20_000, N2):
            for kw in (dict(), dict(narrow_cluster=True)):
                with geometry(**kw):
                    losses, idx, vals = L.score_topk(d_x, d_y, k, L.ORDER_LOSS_DESC)
                g = losses.cpu().numpy()
                want_idx, want_vals = oracle.topk(g, k, oracle.LOSS_DESC)
                np.testing.assert_array_equal(idx.cpu().numpy(), want_idx, err_msg=f"fused N={N2} k={k} {kw}")
                np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))


@pytest.mark.parametrize("N,T,C,dtype,k", [(20_000, 1, 100, "f32", 5_000), (300, 16, 5000, "bf16", 64), (70_000, 1, 10, "f32", 17_500)])
def test_fused_call_is_the_same_in_every_geometry(L, oracle, N, T, C, dtype, k):
    x, y = pool(5, N, T, C, dtype, mask_p=0.1 if T > 1 else 0.0)
    xd, yd = dev_logits(x), torch.from_numpy(y).cuda()
    ref_l, ref_i, ref_v = L.score_topk(xd, yd, k, L.ORDER_LOSS_DESC)
    np.testing.assert_array_equal(ref_i.cpu().numpy(), oracle.topk(ref_l.cpu().numpy(), k, oracle.LOSS_DESC)[0])
    for kw in (dict(max_ctas=2), dict(narrow_cluster=True), dict(no_cluster=True), dict(no_cluster=True, max_ctas=3)):
        with geometry(**kw):
            l, i, v = L.score_topk(xd, yd, k, L.ORDER_LOSS_DESC)
        assert torch.equal(l.view(torch.int32), ref_l.view(torch.int32)) and torch.equal(i, ref_i)
        assert torch.equal(v.view(torch.int32), ref_v.view(torch.int32))


@pytest.mark.parametrize("N,T,C,dtype", [(5_003, 1, 10, "f32"), (3_001, 1, 100, "bf16"), (1_001, 1, 1000, "f32"), (129, 7, 3000, "bf16"),
                                         (9, 2, 70_001, "f32")])
def test_scorer_outputs_and_workspace_stay_inside_their_guards(L, oracle, N, T, C, dtype):
    x, y = pool(11, N, T, C, dtype, mask_p=0.15 if T > 1 else 0.0)
    xd, yd = dev_logits(x), torch.from_numpy(y).cuda()
    lbuf, lmid = guarded(4 * N)
    need = L.score_workspace_bytes(N, T, C)
    wbuf, ws = guarded(need, 0xC3)
    losses = lmid.view(torch.float32)
    L.score_losses(xd, yd, losses=losses, ws=ws)
    assert L.read_device_status(ws) == 0
    assert pads_intact(lbuf, 4 * N) and pads_intact(wbuf, need, 0xC3)
    want, _ = oracle.score(x, y)
    g = losses.cpu().numpy()
    assert (np.abs(g - want) <= 1e-5 * np.abs(want) + C * 2.0 ** -52).all()
    # the fused call: loss table, indices, values and the joint workspace
    k = max(1, N // 3)
    need = L.score_topk_workspace_bytes(N, T, C, k)
    wbuf, ws = guarded(need, 0xC3)
    lbuf, lmid = guarded(4 * N)
    ibuf, imid = guarded(4 * k)
    vbuf, vmid = guarded(4 * k)
    losses2 = lmid.view(torch.float32)
    L.score_topk(xd, yd, k, L.ORDER_LOSS_DESC, losses=losses2, out_idx=imid.view(torch.int32), out_vals=vmid.view(torch.float32), ws=ws)
    torch.cuda.synchronize()
    assert pads_intact(lbuf, 4 * N) and pads_intact(wbuf, need, 0xC3) and pads_intact(ibuf, 4 * k) and pads_intact(vbuf, 4 * k)
    assert torch.equal(losses2, losses)
    np.testing.assert_array_equal(imid.view(torch.int32).cpu().numpy(), oracle.topk(g, k, oracle.LOSS_DESC)[0])


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("D,P", [(1, 2), (1023, 3), (50_001, 10), (272_474, 17)])
def test_round_aggregation_stays_inside_its_guards(L, oracle, D, P, bf16):
    cfg = wl.scaled(wl.CONFIGS[2], D=D, P=P)
    reps = [wl.replica_slice(cfg, i) for i in range(P)]
    base = wl.replica_slice(cfg, 63)
    if bf16:
        reps = [wl.f32_to_bf16_bits(r) for r in reps]
    w = np.full(P, 1.0 / P, np.float32)
    es = 2 if bf16 else 4
    bufs = [guarded(es * D, 0x3C) for _ in range(P)]
    d_reps = []
    for (buf, mid), r in zip(bufs, reps):
        t = mid.view(torch.bfloat16 if bf16 else torch.float32)
        t.copy_(torch.from_numpy(r.view(np.int16)).view(torch.bfloat16) if bf16 else torch.from_numpy(r))
        d_reps.append(t)
    obuf, omid = guarded(4 * D)
    out = omid.view(torch.float32)
    L.aggregate_round(d_reps, w.tolist(), base=torch.from_numpy(base).cuda(), out=out, broadcast=True)
    torch.cuda.synchronize()
    assert pads_intact(obuf, 4 * D) and all(pads_intact(b, es * D, 0x3C) for b, _ in bufs)
    o64, _, _, mag = oracle.aggregate_round(reps, w, base)
    err = np.abs(out.cpu().numpy().astype(np.float64) - o64)
    assert (err <= 1e-6 * mag + 2.0 ** -24 * 1.01 * np.abs(o64)).all()


def test_selector_barrier_gives_up_cleanly(L, oracle):
    """The cooperative selector's barrier is bounded: made to wait for a thread block that does not exist (a test
    hook; nothing on the device is harmed), every block gives up after its poll limit, the status block reports
    LSGD_ERR_TIMEOUT, and the next call on the same context works."""
    N, k = 200_003, 50_000
    h = wl.loss_like_vector(77, N, dup_frac=0.01)
    v = torch.from_numpy(h).cuda()
    ws = L.workspace(L.topk_workspace_bytes(N, k))
    os.environ["LSGD_TEST_PHANTOM_BLOCK"] = "1"
    try:
        L.topk_select(v, k, L.ORDER_LOSS_DESC, ws=ws)
        with pytest.raises(L.LsgdError) as e:
            L.read_device_status(ws)
        assert e.value.status == L.ERR_TIMEOUT
    finally:
        del os.environ["LSGD_TEST_PHANTOM_BLOCK"]
    idx, _ = L.topk_select(v, k, L.ORDER_LOSS_DESC, ws=ws)
    assert L.read_device_status(ws) == 0
    np.testing.assert_array_equal(idx.cpu().numpy(), oracle.topk(h, k, oracle.LOSS_DESC)[0])


BOUNDARY_N = [1025, 4095, 4096, 4097, 8191, 8192, 8193, 32_767, 32_768, 32_769, 65_535, 65_536, 65_537, 150_001]


@pytest.mark.parametrize("N", BOUNDARY_N)
def test_selector_at_block_and_tile_boundaries(L, oracle, N):
    """Pool sizes around the selector's block sizes (4,096 / 8,192 entries, the 65,536-entry limit of the cluster
    variants) and selection sizes around its sort tiles, on four kinds of tables: loss-like with copies and special
    values, all equal, strictly increasing, strictly decreasing."""
    rng = np.random.default_rng(N)
    tables = {
        "loss-like": wl.loss_like_vector(N, N, dup_frac=0.03, specials=True),
        "all equal": np.full(N, 1.25, np.float32),
        "increasing": np.arange(N, dtype=np.float32),
        "decreasing": np.arange(N, 0, -1).astype(np.float32),
    }
    ks = sorted({1, 2, 1023, 1024, 1025, 2048, 2049, 4096, 4097, 8192, 8193, N // 3, N - 1, N} & set(range(1, N + 1)))
    ks = [k for k in ks if k <= N]
    for name, h in tables.items():
        v = torch.from_numpy(h).cuda()
        for k in (ks if name == "loss-like" else [ks[int(rng.integers(len(ks)))], N]):
            for order in (L.ORDER_LOSS_DESC, L.ORDER_INDEX_ASC):
                want_idx, want_vals = oracle.topk(h, k, order)
                for kw in (dict(), dict(narrow_cluster=True)) if N <= 65_536 else (dict(),):
                    with geometry(**kw):
                        idx, vals = L.topk_select(v, k, order)
                    np.testing.assert_array_equal(idx.cpu().numpy(), want_idx, err_msg=f"{name} N={N} k={k} order={order} {kw}")
                    np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32),
                                                  err_msg=f"{name} N={N} k={k} order={order} {kw}")
