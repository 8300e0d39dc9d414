"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *produces inputs* (logits, labels, replicas, weight draws,
step counts).  It holds none of the method's arithmetic: no cross-entropy, no
selection, no aggregation.  Both the CPU oracle's tests and the CUDA library's
tests draw their inputs from here, so that the two sides see identical bytes.

Generation is counter-based: every block of `_CHUNK` elements of a stream comes
from its own Philox key ``(seed, stream, replica, chunk)``, so a value depends
only on the seed and on its position, never on how many threads produced it or
on which sub-range was asked for.  All "N(a, b)" below mean mean a, standard
deviation b.

The five round configurations mirror one communication round of Algorithm 1 at
the scale of the models the paper trains (and larger): P worker replicas of a
flattened parameter vector (Eq. 3's x^i_t), aggregation weights that favour fast
workers, and a candidate pool of N samples whose per-sample loss drives the
top-k selection of Section 4.2.  They stand in for the paper's datasets and
trained models, which are not redistributed here.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

MASTER_SEED = 20250808

# stream ids
_S_BASE, _S_NOISE, _S_WEIGHT, _S_LOGIT, _S_LABEL, _S_MASK, _S_TIES = 1, 2, 3, 4, 5, 6, 7

# elements of one independently keyed block of a stream
_CHUNK = 1 << 20

IGNORE_INDEX = -100


@dataclass(frozen=True)
class RoundConfig:
    """One synthetic communication round: replicas + weights + candidate pool."""

    cfg_id: int
    name: str
    P: int  # worker replicas
    D: int  # parameters per replica (fp32)
    weight_mode: str  # "softmax": softmax of N(0,1) draws; "steps": tau_i ~ U{1..64}
    N: int  # pool samples
    T: int  # tokens per sample (1 = classification)
    C: int  # classes / vocabulary
    dtype: str  # "f32" or "bf16" logits
    sigma: float  # std of the logits
    bump: float  # added to the true-class logit
    mask_p: float  # probability that a token's label is IGNORE_INDEX
    k: int  # samples to select
    dup_frac: float = 0.0  # fraction of pool rows that are exact copies of other rows

    @property
    def seed(self) -> int:
        return MASTER_SEED + self.cfg_id

    @property
    def rows(self) -> int:
        return self.N * self.T

    @property
    def logit_bytes(self) -> int:
        return self.rows * self.C * (4 if self.dtype == "f32" else 2)


CONFIGS = {
    1: RoundConfig(1, "resnet20", 10, 272_474, "softmax", 50_000, 1, 10, "f32", 2.0, 1.5, 0.0, 12_500),
    2: RoundConfig(2, "resnet56", 10, 861_620, "softmax", 50_000, 1, 100, "f32", 2.0, 1.0, 0.0, 12_500),
    3: RoundConfig(3, "wrn28-10", 10, 36_479_194, "softmax", 50_000, 1, 100, "f32", 2.0, 1.0, 0.0, 5_000, 0.01),
    4: RoundConfig(4, "bert-base", 10, 109_482_240, "softmax", 1_024, 128, 30_522, "bf16", 3.0, 0.0, 0.10, 256),
    5: RoundConfig(5, "resnet50-stress", 16, 25_557_032, "steps", 1_281_167, 1, 1_000, "f32", 2.0, 2.0, 0.0, 320_000),
}


def scaled(cfg: RoundConfig, **kw) -> RoundConfig:
    """A copy of `cfg` with some sizes replaced (same seed, same streams)."""
    d = dict(cfg.__dict__)
    d.update(kw)
    return RoundConfig(**d)


def _workers() -> int:
    return max(1, min(32, os.cpu_count() or 1))


def _gen(seed: int, stream: int, sub: int, chunk: int) -> np.random.Generator:
    key = np.array([np.uint64(seed), (np.uint64(stream) << np.uint64(56)) | (np.uint64(sub) << np.uint64(40)) | np.uint64(chunk)],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _pmap(fn, n: int):
    if n <= 1:
        return [fn(i) for i in range(n)]
    with ThreadPoolExecutor(_workers()) as ex:
        return list(ex.map(fn, range(n)))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- #
# replicas and weights
# --------------------------------------------------------------------------- #
def _normal_range(seed: int, stream: int, sub: int, lo: int, hi: int, sigma: float, out: np.ndarray) -> None:
    """out[:] = sigma * N(0,1) for stream positions [lo, hi)."""
    c0, c1 = lo // _CHUNK, (hi - 1) // _CHUNK

    def one(i):
        c = c0 + i
        blk = _gen(seed, stream, sub, c).standard_normal(_CHUNK, dtype=np.float32)
        a, b = max(lo, c * _CHUNK), min(hi, (c + 1) * _CHUNK)
        np.multiply(blk[a - c * _CHUNK:b - c * _CHUNK], np.float32(sigma), out=out[a - lo:b - lo])

    if hi > lo:
        _pmap(one, c1 - c0 + 1)


def replica_slice(cfg: RoundConfig, i: int, lo: int = 0, hi: int | None = None, out: np.ndarray | None = None) -> np.ndarray:
    """Elements [lo, hi) of worker i's parameters: base ~ N(0, 0.05) + N(0, 1e-3)."""
    hi = cfg.D if hi is None else hi
    if out is None:
        out = np.empty(hi - lo, dtype=np.float32)
    noise = np.empty(hi - lo, dtype=np.float32)
    _normal_range(cfg.seed, _S_BASE, 0, lo, hi, 0.05, out)
    _normal_range(cfg.seed, _S_NOISE, i + 1, lo, hi, 1e-3, noise)
    out += noise
    return out


def step_counts(cfg: RoundConfig) -> np.ndarray:
    """Local step counts tau_i ~ U{1..64} (int32), the input of Eq. 3's weights."""
    return _gen(cfg.seed, _S_WEIGHT, 1, 0).integers(1, 65, size=cfg.P, dtype=np.int64).astype(np.int32)


def weight_draws(cfg: RoundConfig) -> np.ndarray:
    """Caller-supplied aggregation weights for the "softmax" configurations.

    A normalised positive vector built from seeded N(0,1) draws.  It is an
    *input* of the aggregation, which uses any weight vector as given.
    """
    z = _gen(cfg.seed, _S_WEIGHT, 0, 0).standard_normal(cfg.P)
    e = np.exp(z - z.max())
    return (e / e.sum()).astype(np.float32)


# --------------------------------------------------------------------------- #
# candidate pool
# --------------------------------------------------------------------------- #
def _rows_per_chunk(cfg: RoundConfig) -> int:
    return max(1, _CHUNK // cfg.C)


def _dup_map(cfg: RoundConfig) -> tuple[np.ndarray, np.ndarray]:
    """(dst, src) sample indices: sample dst is an exact copy of sample src."""
    n = int(round(cfg.dup_frac * cfg.N))
    if n == 0:
        return np.empty(0, np.int64), np.empty(0, np.int64)
    g = _gen(cfg.seed, _S_TIES, 0, 0)
    perm = g.permutation(cfg.N)
    dst, src = perm[:n], perm[n:2 * n]
    return dst.astype(np.int64), src.astype(np.int64)


def _raw_rows(cfg: RoundConfig, r0: int, r1: int):
    """Rows [r0, r1) of the flattened [N*T, C] pool before duplication."""
    rpc = _rows_per_chunk(cfg)
    c0, c1 = r0 // rpc, (r1 - 1) // rpc
    es = np.float32 if cfg.dtype == "f32" else np.uint16
    logits = np.empty((r1 - r0, cfg.C), dtype=es)
    labels = np.empty(r1 - r0, dtype=np.int64)

    def one(i):
        c = c0 + i
        blk = _gen(cfg.seed, _S_LOGIT, 0, c).standard_normal((rpc, cfg.C), dtype=np.float32)
        blk *= np.float32(cfg.sigma)
        lab = _gen(cfg.seed, _S_LABEL, 0, c).integers(0, cfg.C, size=rpc, dtype=np.int64)
        if cfg.bump != 0.0:
            blk[np.arange(rpc), lab] += np.float32(cfg.bump)
        if cfg.mask_p > 0.0:
            m = _gen(cfg.seed, _S_MASK, 0, c).random(rpc) < cfg.mask_p
            lab[m] = IGNORE_INDEX
        a, b = max(r0, c * rpc), min(r1, (c + 1) * rpc)
        sl = slice(a - c * rpc, b - c * rpc)
        logits[a - r0:b - r0] = blk[sl] if cfg.dtype == "f32" else f32_to_bf16_bits(blk[sl])
        labels[a - r0:b - r0] = lab[sl]

    if r1 > r0:
        _pmap(one, c1 - c0 + 1)
    return logits, labels


def pool_rows(cfg: RoundConfig, s0: int = 0, s1: int | None = None):
    """Samples [s0, s1) of the pool.

    Returns (logits [n, T, C] as float32 or as uint16 bf16 bit patterns,
    labels [n, T] int64).  Rows listed by the duplication map are replaced by
    exact copies of their source rows (logits and labels), which gives exactly
    tied losses for the selector's tie-break.
    """
    s1 = cfg.N if s1 is None else s1
    logits, labels = _raw_rows(cfg, s0 * cfg.T, s1 * cfg.T)
    logits = logits.reshape(s1 - s0, cfg.T, cfg.C)
    labels = labels.reshape(s1 - s0, cfg.T)
    dst, src = _dup_map(cfg)
    if dst.size:
        # dst and src are disjoint sets, so a source row is never itself a copy.
        sel = (dst >= s0) & (dst < s1)
        near = sel & (src >= s0) & (src < s1)
        logits[dst[near] - s0] = logits[src[near] - s0]
        labels[dst[near] - s0] = labels[src[near] - s0]
        for d, s in zip(dst[sel & ~near], src[sel & ~near]):
            lg, lb = _raw_rows(cfg, int(s) * cfg.T, (int(s) + 1) * cfg.T)
            logits[d - s0] = lg.reshape(cfg.T, cfg.C)
            labels[d - s0] = lb.reshape(cfg.T)
    return logits, labels


def pool_samples(cfg: RoundConfig, idx) -> tuple[np.ndarray, np.ndarray]:
    """The pool's samples at the given (arbitrary) indices, one by one."""
    lg, lb = [], []
    for i in idx:
        a, b = pool_rows(cfg, int(i), int(i) + 1)
        lg.append(a[0])
        lb.append(b[0])
    return np.stack(lg), np.stack(lb)


def loss_like_vector(seed: int, n: int, dup_frac: float = 0.0, specials: bool = False) -> np.ndarray:
    """A positive, heavy-tailed fp32 vector shaped like a per-sample loss table.

    Optional exact duplicates and special values (+-0, +-inf, NaN, denormals)
    for the selector's ordering rules.  Not a loss computation: just draws.
    """
    g = _gen(seed, _S_TIES, 1, 0)
    v = g.gamma(2.0, 1.2, size=n).astype(np.float32)
    nd = int(dup_frac * n)
    if nd and n > 1:
        dst = g.integers(0, n, size=nd)
        src = g.integers(0, n, size=nd)
        v[dst] = v[src]
    if specials and n >= 16:
        pos = g.permutation(n)[:12]
        sp = np.array([0.0, -0.0, np.inf, -np.inf, np.nan, -np.nan, 1e-45, -1e-45, 3.4e38, -3.4e38, np.inf, np.nan],
                      dtype=np.float32)
        sp[5] = np.frombuffer(np.uint32(0xFFC12345).tobytes(), dtype=np.float32)[0]
        v[pos] = sp
    return v
