"""Pins of the oracle's round aggregation (Eq. 3 and its form around x_t, fp32 or bf16 replicas) to facts
from outside it: the already pinned Eq. 3 routine, numpy in float64, fixed points, and a library's bf16 rounding."""
import numpy as np
import torch

from paper_2508_08540_b200 import workloads as wl


def make(P=5, D=1001, seed=0, bf16=False):
    rng = np.random.default_rng(seed)
    base = rng.normal(0, 0.05, D).astype(np.float32)
    reps = [(base + rng.normal(0, 1e-3, D).astype(np.float32)).astype(np.float32) for _ in range(P)]
    if bf16:
        reps = [wl.f32_to_bf16_bits(r) for r in reps]
    w = rng.random(P).astype(np.float32)
    return base, reps, w


def as_f64(r):
    return (wl.bf16_bits_to_f32(r) if r.dtype == np.uint16 else r).astype(np.float64)


def test_plain_form_is_eq3(oracle):
    for bf16 in (False, True):
        base, reps, w = make(bf16=bf16)
        out, out32, _, mag = oracle.aggregate_round(reps, w)
        ref = np.einsum("i,ij->j", w.astype(np.float64), np.stack([as_f64(r) for r in reps]))
        np.testing.assert_allclose(out, ref, rtol=0, atol=1e-15)
        np.testing.assert_array_equal(out32, out.astype(np.float32))
        np.testing.assert_allclose(mag, np.abs(w.astype(np.float64)[:, None] * np.stack([as_f64(r) for r in reps])).sum(0),
                                   rtol=1e-14)
        if not bf16:
            np.testing.assert_array_equal(out, oracle.aggregate(reps, w)[0])


def test_delta_form_closed_form_and_fixed_points(oracle):
    for bf16 in (False, True):
        base, reps, w = make(seed=1, bf16=bf16)
        X = np.stack([as_f64(r) for r in reps])
        wd, bd = w.astype(np.float64), base.astype(np.float64)
        out, _, _, mag = oracle.aggregate_round(reps, w, base)
        # b + sum w_i (x_i - b) = (1 - sum w) b + sum w_i x_i
        np.testing.assert_allclose(out, (1.0 - wd.sum()) * bd + wd @ X, rtol=0, atol=1e-15)
        np.testing.assert_allclose(mag, np.abs(wd[:, None] * (X - bd)).sum(0), rtol=1e-13)
        # weights that sum to one: the delta form is Eq. 3
        wn = (w / w.sum()).astype(np.float32)
        out1, *_ = oracle.aggregate_round(reps, wn, base)
        np.testing.assert_allclose(out1, wn.astype(np.float64) @ X + (1.0 - wn.astype(np.float64).sum()) * bd, rtol=0, atol=1e-15)
        np.testing.assert_allclose(out1, oracle.aggregate_round(reps, wn)[0], rtol=0, atol=1e-8)
        # one-hot weight: that replica; zero weights: the base itself
        e = np.zeros(len(reps), np.float32)
        e[2] = 1.0
        np.testing.assert_allclose(oracle.aggregate_round(reps, e, base)[0], X[2], rtol=0, atol=1e-17)
        np.testing.assert_array_equal(oracle.aggregate_round(reps, np.zeros(len(reps), np.float32), base)[0], bd)
    # nobody moved: every replica equals the base, so x_{t+1} = x_t exactly, whatever the weights
    base, reps, w = make(seed=2)
    same = [base.copy() for _ in reps]
    out, out32, _, mag = oracle.aggregate_round(same, w * 7.0, base)
    np.testing.assert_array_equal(out32, base)
    assert np.all(mag == 0.0)


def test_bf16_rounding_matches_a_library(oracle):
    rng = np.random.default_rng(3)
    D = 70_000
    x = (rng.normal(0, 1, D) * np.exp(rng.normal(0, 8, D))).astype(np.float32)
    u = x.view(np.uint32)
    u[:3000] = (u[:3000] & 0xFFFF0000) | 0x8000  # exact ties: the low half is exactly one half ulp
    x = u.view(np.float32)
    x[-4:] = [0.0, 1e-40, np.inf, -np.inf]  # (the sum starts from +0, so a lone -0 comes out as +0: left out)
    _, out32, out16, _ = oracle.aggregate_round([x], np.ones(1, np.float32))
    np.testing.assert_array_equal(out32, x)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(out16, lib)
    np.testing.assert_array_equal(out16, wl.f32_to_bf16_bits(x))  # the input generator's rounding agrees too
