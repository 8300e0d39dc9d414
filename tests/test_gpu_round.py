"""Parity of lsgd_aggregate_round with the CPU oracle: Eq. 3 and its form around x_t, fp32 and bf16 replicas,
with and without the write-back into the replicas.  Tolerances (fp32 accumulation: one rounding per difference, P fused multiply-adds, one final add):
  plain form   |g - o| <= 1e-6 * sum_i |w_i x_i[j]|
  delta form   |g - o| <= 1e-6 * sum_i |w_i (x_i[j] - b[j])| + 2^-24 * 1.01 * |o|      (the last term: the final add)
  write-back   fp32 replicas hold `out` bit for bit; bf16 replicas hold `out` rounded to nearest even, bit for bit
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


def replicas_for(D, P, bf16, seed=3):
    cfg = wl.scaled(wl.CONFIGS[seed], D=D, P=P)
    reps = [wl.replica_slice(cfg, i) for i in range(P)]
    base = wl.replica_slice(cfg, 63)  # x_t: the common part plus its own small noise
    if bf16:
        reps = [wl.f32_to_bf16_bits(r) for r in reps]
    w = np.random.default_rng(D + P).random(P).astype(np.float32)
    w /= np.float32(w.sum() * (1.0 if P % 2 else 0.9))  # some cases with weights that do not sum to one
    return reps, base, w


def to_dev(r):
    return torch.from_numpy(r.view(np.int16)).cuda().view(torch.bfloat16) if r.dtype == np.uint16 else torch.from_numpy(r).cuda()


def to_host(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.cpu().numpy()


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("use_base,bcast", [(False, False), (True, False), (False, True), (True, True)])
@pytest.mark.parametrize("D,P", [(1, 1), (7, 2), (1023, 3), (4100, 8), (272_474, 10), (1_000_003, 16), (50_001, 17), (9_999, 64)])
def test_round_matches_oracle(L, oracle, D, P, use_base, bcast, bf16):
    reps, base, w = replicas_for(D, P, bf16)
    o64, _, _, mag = oracle.aggregate_round(reps, w, base if use_base else None)
    d_reps = [to_dev(r) for r in reps]
    out = L.aggregate_round(d_reps, w.tolist(), base=torch.from_numpy(base).cuda() if use_base else None, broadcast=bcast)
    g = out.cpu().numpy()
    tol = 1e-6 * mag + (2.0 ** -24 * 1.01 * np.abs(o64) if use_base else 0.0)
    err = np.abs(g.astype(np.float64) - o64)
    assert np.all(err <= tol), f"worst err/tol {np.max(err / np.maximum(tol, 1e-300)):.3f}"
    for i, d in enumerate(d_reps):
        h = to_host(d)
        if bcast:
            np.testing.assert_array_equal(h, wl.f32_to_bf16_bits(g) if bf16 else g)
        else:
            np.testing.assert_array_equal(h, reps[i])  # untouched


def test_round_fixed_points_and_agreement_with_plain_aggregate(L):
    D, P = 300_007, 10
    reps, base, w = replicas_for(D, P, False)
    d_reps = [to_dev(r) for r in reps]
    wn = (w / w.sum()).astype(np.float32).tolist()
    # nobody moved: x_{t+1} = x_t bit for bit, whatever the weights
    b = torch.from_numpy(base).cuda()
    same = [b.clone() for _ in range(P)]
    assert torch.equal(L.aggregate_round(same, (w * 3).tolist(), base=b), b)
    # the plain form is the Eq. 3 entry point, bit for bit (same order of operations)
    assert torch.equal(L.aggregate_round(d_reps, wn), L.aggregate(d_reps, wn))
    # one-hot weight in the delta form: b + (x_i - b) is x_i up to the roundings of the difference and of the sum
    e = [0.0] * P
    e[4] = 1.0
    got = L.aggregate_round(d_reps, e, base=b).cpu().numpy().astype(np.float64)
    x4 = reps[4].astype(np.float64)
    assert np.all(np.abs(got - x4) <= 2.0 ** -24 * 1.01 * (np.abs(x4) + np.abs(x4 - base.astype(np.float64))))


def test_round_in_place_and_misaligned(L, oracle):
    D, P = 100_003, 4
    reps, base, w = replicas_for(D, P, False)
    o64, _, _, mag = oracle.aggregate_round(reps, w, base)
    tol = 1e-6 * mag + 2.0 ** -24 * 1.01 * np.abs(o64)
    # x_t updated in place (out == base), replicas refreshed in the same pass, no separate output
    d_reps = [to_dev(r) for r in reps]
    b = torch.from_numpy(base).cuda()
    L.aggregate_round(d_reps, w.tolist(), base=b, out=b, broadcast=True)
    assert np.all(np.abs(b.cpu().numpy().astype(np.float64) - o64) <= tol)
    assert all(torch.equal(d, b) for d in d_reps)
    # broadcast without an fp32 output: the replicas alone hold the result
    d_reps = [to_dev(r) for r in reps]
    assert L.aggregate_round(d_reps, w.tolist(), base=torch.from_numpy(base).cuda(), broadcast=True, want_out=False) is None
    assert np.all(np.abs(d_reps[0].cpu().numpy().astype(np.float64) - o64) <= tol)
    # pointers that are only element-aligned take the element path: same numbers
    for bf16 in (False, True):
        reps, base, w = replicas_for(D, P, bf16)
        o64, _, _, mag = oracle.aggregate_round(reps, w, base)
        bufs = [torch.empty(D + 8, dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda") for _ in range(P)]
        views = [buf[1 + i % 3: 1 + i % 3 + D] for i, buf in enumerate(bufs)]
        for v, r in zip(views, reps):
            v.copy_(to_dev(r))
        out = L.aggregate_round(views, w.tolist(), base=torch.from_numpy(base).cuda(), broadcast=True).cpu().numpy()
        assert np.all(np.abs(out.astype(np.float64) - o64) <= 1e-6 * mag + 2.0 ** -24 * 1.01 * np.abs(o64))
        for v in views:
            np.testing.assert_array_equal(to_host(v), wl.f32_to_bf16_bits(out) if bf16 else out)
