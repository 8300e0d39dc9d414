"""Pins of the oracle's per-epoch data allocation (Section 4.2) to facts from outside the oracle.

The generator is pinned to its published known answers; the sizes to the paper's own setting; the
draws to what "uniformly at random without replacement" means: a valid subset of the candidates,
every subset equally likely, priorities that are uniform and independent between streams.
"""
import itertools
import math
import os

import numpy as np
import pytest

HERE = os.path.dirname(__file__)


def golden():
    d = {}
    for line in open(os.path.join(HERE, "golden", "paper_values.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            d[k.strip()] = float(v)
    return d


def test_philox_known_answers(oracle):
    n = 0
    for line in open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        w = [int(x, 16) for x in line]
        got = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in got] == w[6:10]
        n += 1
    assert n == 3


def test_priority_layout(oracle):
    # sample i uses word i mod 4 of the block with counter (i div 4, 0, stream_lo, stream_hi) and key
    # (seed_lo, seed_hi), top 30 bits: checked through the raw block function, whose values the known answers fix
    seed, stream = 0x299F31D0A4093822, 0x0370734413198A2E
    pr = oracle.priorities(23, seed, stream)
    for i in range(23):
        blk = oracle.philox4x32_10([i // 4, 0, stream & 0xFFFFFFFF, stream >> 32], [seed & 0xFFFFFFFF, seed >> 32])
        assert int(pr[i]) == int(blk[i % 4]) >> 2
    assert pr.max() < 2 ** 30


def test_allocation_sizes_paper_setting(oracle):
    g = golden()
    nf, ns, k = oracle.allocation_sizes(int(g["epoch_n"]), int(g["tau_fast"]), int(g["p_fast"]), int(g["tau_slow"]),
                                        int(g["p_slow"]), 1.0)
    assert (nf, ns) == (int(g["n_fast"]), int(g["n_slow"]))
    assert k == nf  # lambda = 1: the whole fast allocation is high-loss samples
    assert nf == int(g["epoch_n"]) * int(g["nf_num"]) // int(g["nf_den"])


@pytest.mark.parametrize("N,tf,pf,ts,ps,lam", [(100_000, 32, 8, 1, 2, 0.5), (1_281_167, 16, 4, 4, 4, 0.3), (7, 3, 1, 1, 1, 0.9),
                                                (1000, 5, 0, 2, 3, 0.5), (1000, 5, 2, 0, 3, 0.25), (0, 1, 1, 1, 1, 0.5)])
def test_allocation_sizes_properties(oracle, N, tf, pf, ts, ps, lam):
    nf, ns, k = oracle.allocation_sizes(N, tf, pf, ts, ps, lam)
    a, b = tf * pf, ts * ps
    assert nf + ns == N  # an epoch covers N samples
    assert nf * (a + b) <= N * a < (nf + 1) * (a + b)  # nf = floor(N a / (a + b)), in exact integers
    assert 0 <= k <= nf and k <= lam * nf < k + 1 + 1e-9


def test_worker_share_is_an_even_partition(oracle):
    for n, P in [(49612, 8), (388, 2), (5, 8), (0, 3), (1_000_003, 7)]:
        parts = [oracle.worker_share(n, P, p) for p in range(P)]
        assert parts[0][0] == 0 and parts[-1][1] == n
        assert all(parts[p][1] == parts[p + 1][0] for p in range(P - 1))
        sizes = [e - b for b, e in parts]
        assert max(sizes) - min(sizes) <= 1 and sum(sizes) == n


def test_draw_is_a_valid_subset_and_a_prefix_chain(oracle):
    N = 5000
    excl = np.arange(0, N, 7, dtype=np.int32)
    full = oracle.draw_uniform(N, N - excl.size, 11, 3, excl)
    assert np.array_equal(np.sort(full), np.setdiff1d(np.arange(N), excl))  # everything that is left, once each
    for m in (0, 1, 17, 2500):
        part = oracle.draw_uniform(N, m, 11, 3, excl)
        assert np.array_equal(part, full[:m])  # the first m of one fixed random order
    with pytest.raises(ValueError):
        oracle.draw_uniform(N, N - excl.size + 1, 11, 3, excl)
    # excluding samples removes them and leaves the order of the others alone
    plain = oracle.draw_uniform(N, N, 11, 3)
    assert np.array_equal(plain[~np.isin(plain, excl)], full)


def test_every_subset_equally_likely(oracle):
    # N = 6 candidates minus one excluded, m = 2: each of the C(5,2) = 10 subsets must come up 1/10 of the time,
    # and each of the 20 ordered pairs 1/20
    trials = 20000
    counts = {}
    for seed in range(trials):
        d = tuple(int(x) for x in oracle.draw_uniform(6, 2, seed, 5, [2]))
        counts[d] = counts.get(d, 0) + 1
    cand = [0, 1, 3, 4, 5]
    assert set(counts) == set(itertools.permutations(cand, 2))
    exp = trials / 20
    chi2 = sum((c - exp) ** 2 / exp for c in counts.values())
    assert chi2 < 50.0  # 19 degrees of freedom: P(chi2 > 50) ~ 1e-4
    sub = {}
    for (a, b), c in counts.items():
        sub[frozenset((a, b))] = sub.get(frozenset((a, b)), 0) + c
    chi2s = sum((c - trials / 10) ** 2 / (trials / 10) for c in sub.values())
    assert chi2s < 33.0  # 9 degrees of freedom


def test_priorities_uniform_and_streams_independent(oracle):
    n = 1 << 18
    a = oracle.priorities(n, 7, 0).astype(np.float64) / 2 ** 30
    b = oracle.priorities(n, 7, 1).astype(np.float64) / 2 ** 30
    c = oracle.priorities(n, 8, 0).astype(np.float64) / 2 ** 30
    for u in (a, b, c):
        assert abs(u.mean() - 0.5) < 5 * math.sqrt(1 / 12 / n)
        h, _ = np.histogram(u, bins=64, range=(0, 1))
        assert ((h - n / 64) ** 2 / (n / 64)).sum() < 130.0  # 63 degrees of freedom
    for u, v in ((a, b), (a, c), (a[:-1], a[1:])):
        assert abs(np.corrcoef(u, v)[0, 1]) < 5 / math.sqrt(n)
    # inclusion frequency of a 25 % draw, by position: no part of the index range is favoured
    m = n // 4
    d = oracle.draw_uniform(n, m, 7, 0)
    h, _ = np.histogram(d, bins=32, range=(0, n))
    p = m / n
    sd = math.sqrt(n / 32 * p * (1 - p))
    assert np.all(np.abs(h - m / 32) < 5 * sd)
    # two streams overlap like two independent draws: hypergeometric, mean m^2 / n
    d2 = oracle.draw_uniform(n, m, 7, 1)
    ov = np.intersect1d(d, d2).size
    assert abs(ov - m * m / n) < 5 * math.sqrt(m * p * (1 - p))


def test_fast_allocation_structure(oracle):
    rng = np.random.default_rng(5)
    N, k, fill = 3000, 700, 900
    losses = rng.gamma(2.0, 1.0, size=N).astype(np.float32)
    losses[rng.integers(0, N, 300)] = losses[rng.integers(0, N, 300)]  # ties
    out = oracle.fast_allocation(losses, k, fill, 3, 9)
    assert out.size == k + fill and np.unique(out).size == out.size
    order = np.argsort(-losses.astype(np.float64), kind="stable")  # library stable sort: ties by lower index
    assert np.array_equal(out[:k], order[:k])
    rest = out[k:]
    assert not np.isin(rest, out[:k]).any()
    # the fill is the draw from the unselected samples, whatever their loss
    assert np.array_equal(rest, oracle.draw_uniform(N, fill, 3, 9, out[:k]))
    # the fill does not look at the losses: its mean loss is that of the unselected, not of the selected
    unsel = np.setdiff1d(np.arange(N), out[:k])
    assert abs(losses[rest].mean() - losses[unsel].mean()) < 5 * losses[unsel].std() / math.sqrt(fill)
    # lambda = 1 (no fill) is the plain top-k; lambda -> 0 (no top-k) is a plain draw
    assert np.array_equal(oracle.fast_allocation(losses, k, 0, 3, 9), order[:k])
    assert np.array_equal(oracle.fast_allocation(losses, 0, fill, 3, 9), oracle.draw_uniform(N, fill, 3, 9))


def test_allocation_k_is_the_decimal_product_rounded_down(oracle):
    """k = floor(lambda N_F) of Section 4.2 for lambda given as a decimal fraction, checked in exact rational
    arithmetic: the double nearest to a decimal lambda may lie below it (0.29 * 100 = 28.999999999999996)."""
    from fractions import Fraction

    sizes = [100, 1000, 49_612, 50_000, 1_281_167, 999_983, 2_000_000_000]
    lams = [f"{i / 100:.2f}" for i in range(0, 101)] + [f"{i / 1000:.3f}" for i in range(1, 1000, 7)] + ["0.3333", "0.0001"]
    for n in sizes:
        for lam in lams:
            nf, ns, k = oracle.allocation_sizes(n, 1, 1, 0, 1, float(lam))  # all samples to the fast group: N_F = n
            assert nf == n and ns == 0
            assert k == (Fraction(lam) * n).__floor__(), (n, lam, k)
