"""Pins of the CPU oracle to facts that do not come from the oracle itself.

Closed forms, invariances, library routines (scipy log-sum-exp, numpy einsum and
stable argsort), values fixed by the paper (tests/golden/paper_values.txt) and
brute force on tiny inputs.  Chosen so that a dropped term, a wrong sign or
index, or a transposed operand fails at least one of them.
"""
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden():
    d = {}
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            d[k.strip()] = float(v)
    return d


# --------------------------------------------------------------------------- #
# scorer
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("C,lnC", [(10, 2.302585092994046), (100, 4.605170185988092), (1000, 6.907755278982137),
                                   (30522, 10.32620301405082)])
def test_uniform_logits_give_ln_C(oracle, C, lnC):
    # softmax of equal logits is 1/C for every class, so CE = ln C whatever the label
    assert abs(lnC - math.log(C)) < 1e-15
    x = np.full((3, C), 0.7, dtype=np.float32)
    y = np.array([0, C // 2, C - 1])
    loss, bad = oracle.score(x, y)
    assert bad == 0
    np.testing.assert_allclose(loss, lnC, rtol=1e-14)


def test_known_probabilities(oracle):
    # logits = ln(1), ln(2), ln(3)  =>  softmax = 1/6, 2/6, 3/6
    x = np.log(np.array([[1.0, 2.0, 3.0]] * 3)).astype(np.float32)
    loss, _ = oracle.score(x, np.array([0, 1, 2]))
    xd = x.astype(np.float64)
    z = np.exp(xd[0]).sum()
    np.testing.assert_allclose(loss, [math.log(z / math.exp(xd[0, j])) for j in range(3)], rtol=1e-14)
    np.testing.assert_allclose(loss, [math.log(6), math.log(3), math.log(2)], rtol=1e-6)  # fp32 rounding of ln 2, ln 3


def test_two_class_softplus(oracle):
    rng = np.random.default_rng(1)
    x = rng.normal(0, 4, size=(200, 2)).astype(np.float32)
    y = rng.integers(0, 2, size=200)
    loss, _ = oracle.score(x, y)
    xd = x.astype(np.float64)
    other = xd[np.arange(200), 1 - y]
    true = xd[np.arange(200), y]
    np.testing.assert_allclose(loss, np.logaddexp(0.0, other - true), rtol=1e-13, atol=4e-16)  # log(1+eps) in double


def test_single_class_is_zero(oracle):
    loss, _ = oracle.score(np.array([[3.5], [-2.0]], dtype=np.float32), np.array([0, 0]))
    assert np.all(loss == 0.0)


def test_matches_library_logsumexp_and_layout(oracle):
    # [N, T, C] row-major with N, T, C all different catches any transposition
    rng = np.random.default_rng(2)
    N, T, C = 5, 3, 17
    x = rng.normal(0, 3, size=(N, T, C)).astype(np.float32)
    y = rng.integers(0, C, size=(N, T))
    loss, bad, tok = oracle.score(x, y, return_tokens=True)
    xd = x.astype(np.float64)
    ref_tok = logsumexp(xd, axis=2) - np.take_along_axis(xd, y[..., None], axis=2)[..., 0]
    np.testing.assert_allclose(tok, ref_tok, rtol=1e-13)
    np.testing.assert_allclose(loss, ref_tok.mean(axis=1), rtol=1e-13)
    assert bad == 0


def test_shift_and_permutation_invariance(oracle):
    rng = np.random.default_rng(3)
    # multiples of 1/8 so that the shifted logits stay exact in fp32
    x = (rng.integers(-64, 64, size=(50, 33)) / 8.0).astype(np.float32)
    y = rng.integers(0, 33, size=50)
    base, _ = oracle.score(x, y)
    shifted, _ = oracle.score(x + np.float32(100.0), y)
    np.testing.assert_allclose(shifted, base, rtol=1e-13)
    perm = rng.permutation(33)
    inv = np.argsort(perm)
    permuted, _ = oracle.score(np.ascontiguousarray(x[:, perm]), inv[y])
    np.testing.assert_allclose(permuted, base, rtol=1e-13)


def test_huge_logits_stay_finite(oracle):
    x = np.array([[1e4, -1e4], [-1e4, 1e4], [1e4, 1e4]], dtype=np.float32)
    loss, _ = oracle.score(x, np.array([1, 1, 0]))
    np.testing.assert_allclose(loss, [2e4, 0.0, math.log(2)], rtol=1e-15, atol=0)


def test_dominant_class_first_order_and_small_losses(oracle):
    # true class far ahead: loss = log1p(sum_j!=y exp(x_j - x_y)) ~ that sum; checks tiny losses are resolved
    x = np.array([[20.0, 0.0, 1.0, -1.0]], dtype=np.float32)
    loss, _ = oracle.score(x, np.array([0]))
    eps = math.exp(-20) + math.exp(-19) + math.exp(-21)
    # the definition evaluates log(1 + eps) in double: absolute resolution ~2^-52
    np.testing.assert_allclose(loss, math.log1p(eps), rtol=1e-12, atol=4e-16)
    assert abs(loss[0] - eps) < 4e-16 + eps * eps


def test_losses_nonnegative(oracle):
    rng = np.random.default_rng(4)
    x = rng.normal(0, 10, size=(300, 7)).astype(np.float32)
    y = rng.integers(0, 7, size=300)
    loss, _ = oracle.score(x, y)
    assert np.all(loss >= 0.0)


def test_masking_equals_deleting_tokens(oracle):
    rng = np.random.default_rng(5)
    N, T, C = 4, 6, 11
    x = rng.normal(0, 2, size=(N, T, C)).astype(np.float32)
    y = rng.integers(0, C, size=(N, T))
    ym = y.copy()
    ym[0, 1] = ym[0, 4] = ym[2, 0] = -100
    ym[3, :] = -100  # a sample with every token ignored scores 0 (library convention)
    loss, bad, tok = oracle.score(x, ym, return_tokens=True)
    assert bad == 0
    # the same tokens scored one by one as plain classification
    flat, _ = oracle.score(x.reshape(N * T, C), y.reshape(N * T))
    flat = flat.reshape(N, T)
    np.testing.assert_allclose(loss[0], flat[0, [0, 2, 3, 5]].mean(), rtol=1e-14)
    np.testing.assert_allclose(loss[1], flat[1].mean(), rtol=1e-14)
    np.testing.assert_allclose(loss[2], flat[2, 1:].mean(), rtol=1e-14)
    assert loss[3] == 0.0
    assert tok[0, 1] == 0.0 and tok[3].sum() == 0.0


def test_bf16_bits_are_widened_exactly(oracle):
    from paper_2508_08540_b200.workloads import bf16_bits_to_f32, f32_to_bf16_bits

    rng = np.random.default_rng(6)
    x = rng.normal(0, 3, size=(20, 40)).astype(np.float32)
    bits = f32_to_bf16_bits(x).reshape(20, 40)
    back = bf16_bits_to_f32(bits)
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    # 1.5 = 0x3FC0, -2.0 = 0xC000 in bf16
    assert f32_to_bf16_bits(np.array([1.5, -2.0], np.float32)).tolist() == [0x3FC0, 0xC000]
    y = rng.integers(0, 40, size=20)
    a, _ = oracle.score(bits, y)
    b, _ = oracle.score(back, y)
    np.testing.assert_array_equal(a, b)


def test_bad_labels_are_nan_and_counted(oracle):
    x = np.zeros((3, 2, 4), dtype=np.float32)
    y = np.array([[0, 4], [1, -1], [2, 3]])
    loss, bad = oracle.score(x, y)
    assert bad == 2
    assert np.isnan(loss[0]) and np.isnan(loss[1]) and loss[2] == pytest.approx(math.log(4))


# --------------------------------------------------------------------------- #
# selector
# --------------------------------------------------------------------------- #
def brute_topk(v, k):
    """k rounds of 'scan for the best remaining': higher value first, then lower index.
    -0 == +0; NaN above everything."""
    def key(x):
        return (2, 0.0) if x != x else (1, float(x))

    left = list(range(len(v)))
    out = []
    for _ in range(k):
        best = left[0]
        for i in left[1:]:
            if key(v[i]) > key(v[best]):
                best = i
        out.append(best)
        left.remove(best)
    return out


@pytest.mark.parametrize("seed", range(6))
def test_topk_against_brute_force(oracle, seed):
    from paper_2508_08540_b200.workloads import loss_like_vector

    n = [1, 2, 17, 64, 257, 600][seed]
    v = loss_like_vector(100 + seed, n, dup_frac=0.3, specials=(n >= 16))
    for k in sorted({0, 1, n // 3, n - 1 if n > 1 else 1, n}):
        idx, vals = oracle.topk(v, k, oracle.LOSS_DESC)
        ref = brute_topk(v, k)
        assert idx.tolist() == ref
        np.testing.assert_array_equal(vals.view(np.uint32), v[ref].view(np.uint32) if k else np.empty(0, np.uint32))
        idx2, _ = oracle.topk(v, k, oracle.INDEX_ASC)
        assert idx2.tolist() == sorted(ref)


def test_topk_special_orders(oracle):
    n = 1000
    v = np.full(n, 0.25, dtype=np.float32)
    assert oracle.topk(v, 10)[0].tolist() == list(range(10))  # all tied: lowest indices
    inc = np.arange(n, dtype=np.float32)
    assert oracle.topk(inc, 5)[0].tolist() == [999, 998, 997, 996, 995]
    rng = np.random.default_rng(7)
    r = rng.normal(size=n).astype(np.float32)
    assert oracle.topk(r, 1)[0][0] == int(np.argmax(r))
    full = oracle.topk(r, n)[0]
    np.testing.assert_array_equal(full, np.argsort(-r.astype(np.float64), kind="stable"))
    # -0 and +0 tie (lower index first); NaN outranks +inf; NaNs tie among themselves
    s = np.array([0.0, -0.0, np.inf, np.nan, -np.inf, np.nan, -0.0], dtype=np.float32)
    assert oracle.topk(s, 7)[0].tolist() == [3, 5, 2, 0, 1, 6, 4]


def test_topk_set_is_permutation_equivariant(oracle):
    rng = np.random.default_rng(8)
    v = rng.permutation(5000).astype(np.float32)  # distinct values
    perm = rng.permutation(5000)
    a = set(oracle.topk(v, 777)[0].tolist())
    b = set(oracle.topk(v[perm], 777)[0].tolist())
    assert a == {int(perm[j]) for j in b}
    with pytest.raises(ValueError):
        oracle.topk(v, 5001)


# --------------------------------------------------------------------------- #
# aggregation
# --------------------------------------------------------------------------- #
def test_aggregate_one_hot_uniform_identity_linearity(oracle):
    rng = np.random.default_rng(9)
    P, D = 5, 37  # P != D so a transposed access cannot pass
    reps = [rng.normal(size=D).astype(np.float32) for _ in range(P)]
    for i in range(P):
        w = np.zeros(P, np.float32)
        w[i] = 1.0
        out, out32, _ = oracle.aggregate(reps, w)
        np.testing.assert_array_equal(out32, reps[i])
    # equal step counts: Eq. 3 is the plain average of Section 4.3's balanced rule
    out, _, _ = oracle.aggregate(reps, np.full(P, 0.2, np.float32))
    np.testing.assert_allclose(out, np.float64(np.float32(0.2)) * np.sum(np.stack(reps).astype(np.float64), axis=0), rtol=1e-12, atol=1e-16)
    np.testing.assert_allclose(out, np.mean(np.stack(reps).astype(np.float64), axis=0), rtol=1e-6, atol=1e-7)
    # identical replicas and weights summing to 1 reproduce the replica
    w = np.array([0.5, 0.25, 0.125, 0.0625, 0.0625], np.float32)
    out, out32, mag = oracle.aggregate([reps[0]] * P, w)
    np.testing.assert_array_equal(out32, reps[0])
    np.testing.assert_allclose(mag, np.abs(reps[0].astype(np.float64)), rtol=1e-15)
    # library contraction, and linearity in w
    w1 = rng.random(P).astype(np.float32)
    w2 = rng.random(P).astype(np.float32)
    X = np.stack(reps).astype(np.float64)
    o1, _, m1 = oracle.aggregate(reps, w1)
    o2, _, _ = oracle.aggregate(reps, w2)
    np.testing.assert_allclose(o1, np.einsum("p,pd->d", w1.astype(np.float64), X), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(m1, np.einsum("p,pd->d", w1.astype(np.float64), np.abs(X)), rtol=1e-13)
    o12, _, _ = oracle.aggregate(reps, (w1.astype(np.float64) + w2.astype(np.float64)).astype(np.float32))
    np.testing.assert_allclose(o12, o1 + o2, rtol=1e-6, atol=1e-6)


def test_weights_from_steps_paper_setting(oracle):
    g = golden()
    tau = [int(g["tau_fast"])] * int(g["p_fast"]) + [int(g["tau_slow"])] * int(g["p_slow"])
    w = oracle.weights_from_steps(tau)
    assert sum(tau) == g["w_den"]
    np.testing.assert_array_equal(w[:8], np.float32(g["w_fast_num"] / g["w_den"]))
    np.testing.assert_array_equal(w[8:], np.float32(g["w_slow_num"] / g["w_den"]))
    assert abs(float(w.astype(np.float64).sum()) - 1.0) < 1e-6
    # the fast workers' share of the data, Section 4.2
    assert sum(tau[:8]) / sum(tau) == g["nf_num"] / g["nf_den"]
    # equal steps: uniform weights
    np.testing.assert_array_equal(oracle.weights_from_steps([7] * 4), np.float32(0.25))
    with pytest.raises(ValueError):
        oracle.weights_from_steps([0, 0])


def test_index_width_from_paper_example():
    g = golden()
    assert round(g["index_example_n"] * g["index_bytes"] / 1024, 1) == g["index_example_kib"]
    assert np.dtype(np.int32).itemsize == g["index_bytes"]
