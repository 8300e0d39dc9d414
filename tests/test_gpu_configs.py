"""The five synthetic rounds at their full sizes, through the same calls bench.py times
(lsgd_score_topk in loss-descending order, then lsgd_aggregate), checked in FULL:

  every per-sample loss of the whole pool against the oracle (Algorithm 1's loss record),
  the selection, exact, against the oracle run on the library's own loss vector, and the end-to-end
  inequality "every selected loss >= every unselected loss" in the oracle's losses of the whole pool,
  every aggregated parameter of the whole vector against the oracle (Eq. 3).

The oracle is the unchanged single-threaded routine; it is called on disjoint sample / parameter
ranges from a few host threads so that the five rounds finish in minutes.
Tolerances as in test_gpu_parity.py.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from paper_2508_08540_b200 import workloads as wl

pytestmark = pytest.mark.gpu

HOST_THREADS = max(1, min(16, os.cpu_count() or 1))


@pytest.fixture(scope="module")
def L():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2508_08540_b200 import lsgd

    lsgd.lib()
    return lsgd


def oracle_losses(oracle, x, y):
    """oracle.score over the samples of (x, y), split into contiguous ranges over the host threads."""
    n = x.shape[0]
    cuts = np.linspace(0, n, min(n, HOST_THREADS) + 1).astype(np.int64)
    with ThreadPoolExecutor(HOST_THREADS) as ex:
        parts = list(ex.map(lambda ab: oracle.score(x[ab[0]:ab[1]], y[ab[0]:ab[1]]), zip(cuts[:-1], cuts[1:])))
    return np.concatenate([p[0] for p in parts]), sum(p[1] for p in parts)


def upload_pool_and_score_it(cfg, oracle):
    """The whole pool on the device, generated in slabs of about 256 MB, each slab scored by the oracle on the way."""
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    d_logits = torch.empty((cfg.N, cfg.T, cfg.C), dtype=tdt, device="cuda")
    labels = np.empty((cfg.N, cfg.T), dtype=np.int64)
    want = np.empty(cfg.N, dtype=np.float64)
    bad = 0
    es = 4 if cfg.dtype == "f32" else 2
    step = max(1, (1 << 28) // (cfg.T * cfg.C * es))
    for s0 in range(0, cfg.N, step):
        s1 = min(cfg.N, s0 + step)
        x, y = wl.pool_rows(cfg, s0, s1)
        t = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) if cfg.dtype == "bf16" else torch.from_numpy(x)
        d_logits[s0:s1].copy_(t)
        labels[s0:s1] = y
        want[s0:s1], b = oracle_losses(oracle, x, y)
        bad += b
    return d_logits, labels, want, bad


@pytest.mark.parametrize("cfg_id", [1, 2, 3, 4, 5])
def test_full_config(L, oracle, cfg_id):
    cfg = wl.CONFIGS[cfg_id]

    # ---------------- score + top-k, as benchmarked ----------------
    d_logits, labels, want, bad = upload_pool_and_score_it(cfg, oracle)
    assert bad == 0
    d_labels = torch.from_numpy(labels).cuda()
    ws = L.workspace(L.score_topk_workspace_bytes(cfg.N, cfg.T, cfg.C, cfg.k))
    losses, idx, vals = L.score_topk(d_logits, d_labels, cfg.k, L.ORDER_LOSS_DESC, ws=ws)
    assert L.read_device_status(ws) == 0
    g = losses.cpu().numpy()
    assert g.shape == (cfg.N,) and np.isfinite(g).all() and (g >= 0).all()

    # every loss of the pool against the oracle
    err = np.abs(g.astype(np.float64) - want)
    tol = 1e-5 * np.abs(want) + cfg.C * 2.0 ** -52
    assert (err <= tol).all(), f"{(err > tol).sum()} of {cfg.N} losses off; worst rel {np.max(err / want):.3e}"
    if cfg.dup_frac:
        dst, src = wl._dup_map(cfg)
        assert dst.size == round(cfg.dup_frac * cfg.N)
        assert np.array_equal(g[dst], g[src]), "copied rows must score identical bits"

    # the selection is exact on the library's own loss vector, in both orders; values are the losses' bits
    want_idx, want_vals = oracle.topk(g, cfg.k, oracle.LOSS_DESC)
    np.testing.assert_array_equal(idx.cpu().numpy(), want_idx)
    np.testing.assert_array_equal(vals.cpu().numpy().view(np.uint32), want_vals.view(np.uint32))
    idx_asc, _ = L.topk_select(losses, cfg.k, L.ORDER_INDEX_ASC, want_vals=False)
    np.testing.assert_array_equal(idx_asc.cpu().numpy(), np.sort(want_idx))
    sel = np.zeros(cfg.N, bool)
    sel[want_idx] = True
    assert g[sel].min() >= g[~sel].max()  # every selected loss >= every unselected one, no slack needed
    # end to end, in the oracle's own losses of the whole pool: slack 1e-5 * max(1, |threshold|)
    thr = float(g[sel].min())
    slack = 1e-5 * max(1.0, abs(thr))
    assert want[sel].min() >= want[~sel].max() - slack
    assert (want[sel] >= thr - slack).all() and (want[~sel] <= thr + slack).all()
    # and against the selection the oracle makes from its own losses: the two sets differ only by samples whose
    # loss lies within the slack of the cut
    o_idx, _ = oracle.topk(want.astype(np.float32), cfg.k, oracle.LOSS_DESC)
    o_sel = np.zeros(cfg.N, bool)
    o_sel[o_idx] = True
    moved = sel != o_sel
    assert (np.abs(want[moved] - thr) <= slack).all(), f"{moved.sum()} samples moved across the cut beyond the slack"

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
    h_reps = [wl.replica_slice(cfg, i) for i in range(cfg.P)]
    reps = [torch.from_numpy(r).cuda() for r in h_reps]
    out = L.aggregate(reps, w.tolist())
    out2 = L.aggregate(reps, w.tolist())
    assert torch.equal(out, out2)
    got = out.cpu().numpy()
    assert got.shape == (cfg.D,)
    del reps, out, out2
    torch.cuda.empty_cache()

    # every parameter against the oracle, in windows of 4 M elements spread over the host threads
    span = 1 << 22

    def window(lo):
        hi = min(cfg.D, lo + span)
        o64, _, mag = oracle.aggregate([r[lo:hi] for r in h_reps], w)
        e = np.abs(got[lo:hi].astype(np.float64) - o64)
        big = np.abs(o64) >= 1e-2  # plain relative error where nothing cancels
        return (int((e > 1e-6 * mag).sum()), float(np.max(e / mag)), float(e @ e), float(o64 @ o64),
                int((e[big] > 1e-6 * np.abs(o64[big])).sum()), hi - lo)

    with ThreadPoolExecutor(HOST_THREADS) as ex:
        res = list(ex.map(window, range(0, cfg.D, span)))
    assert sum(r[5] for r in res) == cfg.D
    assert sum(r[0] for r in res) == 0, f"worst {max(r[1] for r in res):.3e} of sum_i |w_i x_i|"
    assert np.sqrt(sum(r[2] for r in res)) <= 1e-6 * np.sqrt(sum(r[3] for r in res))
    assert sum(r[4] for r in res) == 0
