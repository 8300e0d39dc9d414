"""The five synthetic rounds at their full sizes, through the same calls bench.py times
(lsgd_score_topk in loss-descending order, then lsgd_aggregate).

The oracle cannot score a whole 8 GB pool in seconds, so losses and aggregated parameters are
checked on samples it computes one by one (the generators are position-addressable), while the
selection, which is exact, is checked in full against the oracle run on the library's own loss
vector.  Tolerances as in test_gpu_parity.py.
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


def upload_pool(cfg):
    """The whole pool on the device, generated in slabs of about 256 MB."""
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    d_logits = torch.empty((cfg.N, cfg.T, cfg.C), dtype=tdt, device="cuda")
    labels = np.empty((cfg.N, cfg.T), dtype=np.int64)
    es = 4 if cfg.dtype == "f32" else 2
    step = max(1, (1 << 28) // (cfg.T * cfg.C * es))
    for s0 in range(0, cfg.N, step):
        s1 = min(cfg.N, s0 + step)
        x, y = wl.pool_rows(cfg, s0, s1)
        t = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) if cfg.dtype == "bf16" else torch.from_numpy(x)
        d_logits[s0:s1].copy_(t)
        labels[s0:s1] = y
    return d_logits, labels


@pytest.mark.parametrize("cfg_id", [1, 2, 3, 4, 5])
def test_full_config(L, oracle, cfg_id):
    cfg = wl.CONFIGS[cfg_id]
    rng = np.random.default_rng(cfg.seed)

    # ---------------- score + top-k, as benchmarked ----------------
    d_logits, labels = upload_pool(cfg)
    d_labels = torch.from_numpy(labels).cuda()
    ws = L.workspace(L.score_topk_workspace_bytes(cfg.N, cfg.T, cfg.C, cfg.k))
    losses, idx, vals = L.score_topk(d_logits, d_labels, cfg.k, L.ORDER_LOSS_DESC, ws=ws)
    assert L.read_device_status(ws) == 0
    g = losses.cpu().numpy()
    assert np.isfinite(g).all() and (g >= 0).all()

    # sampled losses against the oracle, one sample at a time (first, last, and random ones)
    n_check = 24 if cfg.T > 1 else 400
    pick = np.unique(np.concatenate([[0, cfg.N - 1], rng.integers(0, cfg.N, n_check)]))
    if cfg.dup_frac:
        dst, src = wl._dup_map(cfg)
        pick = np.unique(np.concatenate([pick, dst[:50], src[:50]]))
        assert np.array_equal(g[dst], g[src]), "copied rows must score identical bits"
    x, y = wl.pool_samples(cfg, pick)
    np.testing.assert_array_equal(y, labels[pick])
    want, bad = oracle.score(x, y)
    assert bad == 0
    err = np.abs(g[pick].astype(np.float64) - want)
    assert (err <= 1e-5 * np.abs(want) + cfg.C * 2.0 ** -52).all(), f"worst rel {np.max(err / want):.3e}"

    # the selection is exact on the library's own loss vector, in both orders; values are the losses' bits
    want_idx, want_vals = oracle.topk(g, cfg.k, oracle.LOSS_DESC)
    np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
    np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))
    idx_asc, _ = L.topk_select(losses, cfg.k, L.ORDER_INDEX_ASC, want_vals=False)
    np.testing.assert_array_equal(idx_asc.cpu().numpy(), np.sort(want_idx))
    sel = np.zeros(cfg.N, bool)
    sel[want_idx] = True
    assert g[sel].min() >= g[~sel].max()  # every selected loss >= every unselected one, no slack needed
    # against the oracle's own losses on the sampled rows: slack 1e-5 * max(1, |threshold|)
    thr = g[sel].min()
    slack = 1e-5 * max(1.0, abs(thr))
    in_sel = sel[pick]
    assert (want[in_sel] >= thr - slack).all() and (want[~in_sel] <= thr + slack).all()

    # same bits on a second run and through the two separate entry points
    losses2, idx2, _ = L.score_topk(d_logits, d_labels, cfg.k, L.ORDER_LOSS_DESC, ws=ws)
    assert torch.equal(losses, losses2) and torch.equal(idx, idx2)
    sep = L.score_losses(d_logits, d_labels)
    assert torch.equal(sep, losses)
    del d_logits, losses2, sep
    torch.cuda.empty_cache()

    # ---------------- aggregation, as benchmarked ----------------
    if cfg.weight_mode == "steps":
        tau = wl.step_counts(cfg)
        w = np.array(L.weights_from_steps(tau.tolist()), np.float32)
        np.testing.assert_array_equal(w, oracle.weights_from_steps(tau))
    else:
        w = wl.weight_draws(cfg)
    reps = []
    for i in range(cfg.P):
        reps.append(torch.from_numpy(wl.replica_slice(cfg, i)).cuda())
    out = L.aggregate(reps, w.tolist())
    out2 = L.aggregate(reps, w.tolist())
    assert torch.equal(out, out2)
    # three windows (start, a ragged middle, the end) recomputed by the oracle from regenerated slices
    span = 200_000
    for lo in sorted({0, max(0, cfg.D // 2 - 12_345), max(0, cfg.D - span)}):
        hi = min(cfg.D, lo + span)
        sl = [wl.replica_slice(cfg, i, lo, hi) for i in range(cfg.P)]
        np.testing.assert_array_equal(sl[0], reps[0][lo:hi].cpu().numpy())
        o64, _, mag = oracle.aggregate(sl, w)
        got = out[lo:hi].cpu().numpy()
        err = np.abs(got.astype(np.float64) - o64)
        assert (err <= 1e-6 * mag).all(), f"worst {np.max(err / mag):.3e}"
        assert np.linalg.norm(err) <= 1e-6 * np.linalg.norm(o64)
        big = np.abs(o64) >= 1e-2
        assert (err[big] <= 1e-6 * np.abs(o64[big])).all()  # plain relative error where nothing cancels
    del reps, out, out2
    torch.cuda.empty_cache()
