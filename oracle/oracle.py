"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not the product).

Builds ``lsgd_oracle.cpp`` with g++ into ``liblsgd_oracle.so`` next to this file
and exposes its four functions on numpy arrays.  Only tests, the smoke check and
the benchmark's CPU-baseline leg may import this module.  It shares nothing with
the CUDA library and does not import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lsgd_oracle.cpp")
_LIB = os.path.join(_HERE, "liblsgd_oracle.so")
_lib = None

F32, BF16 = 0, 1
LOSS_DESC, INDEX_ASC = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle (g++ -O2, no fast-math) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fno-fast-math", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
        lib.oracle_score.argtypes = [vp, ctypes.c_int, vp, i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_topk.argtypes = [vp, i64, i64, ctypes.c_int, vp, vp]
        lib.oracle_aggregate.argtypes = [vp, vp, i32, i64, vp, vp, vp]
        lib.oracle_weights_from_steps.argtypes = [vp, i32, vp]
        u64, dbl = ctypes.c_uint64, ctypes.c_double
        lib.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        lib.oracle_allocation_sizes.argtypes = [i64, i32, i32, i32, i32, dbl, vp, vp, vp]
        lib.oracle_worker_share.argtypes = [i64, i32, i32, vp, vp]
        lib.oracle_draw_uniform.argtypes = [i64, i64, u64, u64, vp, i64, vp]
        lib.oracle_priorities.argtypes = [i64, u64, u64, vp]
        lib.oracle_fast_allocation.argtypes = [vp, i64, i64, i64, u64, u64, vp]
        lib.oracle_aggregate_round.argtypes = [vp, ctypes.c_int, vp, i32, i64, vp, vp, vp, vp, vp]
        lib.oracle_aggregate_round.restype = ctypes.c_int
        for f in (lib.oracle_score, lib.oracle_topk, lib.oracle_aggregate, lib.oracle_weights_from_steps,
                  lib.oracle_philox4x32_10, lib.oracle_allocation_sizes, lib.oracle_worker_share,
                  lib.oracle_draw_uniform, lib.oracle_priorities, lib.oracle_fast_allocation):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else None


def score(logits: np.ndarray, labels: np.ndarray, ignore_index: int = -100, return_tokens: bool = False):
    """Per-sample mean cross-entropy in double.

    logits: [N, T, C] or [N, C]; float32, or uint16 holding bf16 bit patterns.
    labels: [N, T] or [N] int64.  Returns (loss[N] float64, bad_label_count)
    and, if asked, the token losses [N, T] float64.
    """
    if logits.ndim == 2:
        logits = logits[:, None, :]
    N, T, C = logits.shape
    if logits.dtype == np.float32:
        dt = F32
    elif logits.dtype == np.uint16:
        dt = BF16
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    logits = np.ascontiguousarray(logits)
    labels = np.ascontiguousarray(labels, dtype=np.int64).reshape(N, T)
    out = np.empty(N, dtype=np.float64)
    tok = np.empty((N, T), dtype=np.float64) if return_tokens else None
    bad = np.zeros(1, dtype=np.int64)
    rc = _load().oracle_score(_ptr(logits), dt, _ptr(labels), N, T, C, ignore_index, _ptr(out), _ptr(tok), _ptr(bad))
    assert rc == 0
    return (out, int(bad[0]), tok) if return_tokens else (out, int(bad[0]))


def topk(losses: np.ndarray, k: int, order: int = LOSS_DESC):
    """(idx[k] int32, vals[k] float32): highest loss first, ties by lower index."""
    losses = np.ascontiguousarray(losses, dtype=np.float32)
    idx = np.empty(k, dtype=np.int32)
    vals = np.empty(k, dtype=np.float32)
    rc = _load().oracle_topk(_ptr(losses), losses.size, k, order, _ptr(idx), _ptr(vals))
    if rc != 0:
        raise ValueError("k out of range")
    return idx, vals


def aggregate(replicas, weights: np.ndarray):
    """Eq. 3 in double.  Returns (out float64 [D], out rounded to float32, sum_i |w_i x_i| float64)."""
    reps = [np.ascontiguousarray(r, dtype=np.float32) for r in replicas]
    P, D = len(reps), reps[0].size
    assert all(r.size == D for r in reps)
    w = np.ascontiguousarray(weights, dtype=np.float32)
    assert w.size == P
    ptrs = (ctypes.c_void_p * P)(*[r.ctypes.data for r in reps])
    out = np.empty(D, dtype=np.float64)
    out32 = np.empty(D, dtype=np.float32)
    mag = np.empty(D, dtype=np.float64)
    rc = _load().oracle_aggregate(ctypes.cast(ptrs, ctypes.c_void_p), _ptr(w), P, D, _ptr(out), _ptr(out32), _ptr(mag))
    assert rc == 0
    return out, out32, mag


def weights_from_steps(tau) -> np.ndarray:
    tau = np.ascontiguousarray(tau, dtype=np.int32)
    w = np.empty(tau.size, dtype=np.float32)
    rc = _load().oracle_weights_from_steps(_ptr(tau), tau.size, _ptr(w))
    if rc != 0:
        raise ValueError("step counts must sum to a positive number")
    return w


def philox4x32_10(ctr, key) -> np.ndarray:
    """One Philox4x32-10 block: ctr (4 x u32), key (2 x u32) -> 4 x u32."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.empty(4, dtype=np.uint32)
    assert c.size == 4 and k.size == 2
    _load().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def allocation_sizes(N: int, tau_fast: int, p_fast: int, tau_slow: int, p_slow: int, lam: float):
    """(N_F, N_S, k) of Section 4.2."""
    out = np.zeros(3, dtype=np.int64)
    rc = _load().oracle_allocation_sizes(N, tau_fast, p_fast, tau_slow, p_slow, lam, _ptr(out[0:1]), _ptr(out[1:2]),
                                         _ptr(out[2:3]))
    if rc != 0:
        raise ValueError("invalid allocation arguments")
    return int(out[0]), int(out[1]), int(out[2])


def worker_share(n: int, P: int, p: int):
    """[begin, end) of worker p's part of an n-entry list split evenly over P workers."""
    out = np.zeros(2, dtype=np.int64)
    rc = _load().oracle_worker_share(n, P, p, _ptr(out[0:1]), _ptr(out[1:2]))
    if rc != 0:
        raise ValueError("invalid split arguments")
    return int(out[0]), int(out[1])


def draw_uniform(N: int, m: int, seed: int, stream: int, exclude=None) -> np.ndarray:
    """m indices drawn uniformly without replacement from 0..N-1 minus `exclude`, in draw order."""
    ex = np.ascontiguousarray(exclude if exclude is not None else [], dtype=np.int32)
    out = np.empty(m, dtype=np.int32)
    rc = _load().oracle_draw_uniform(N, m, seed, stream, _ptr(ex), ex.size, _ptr(out))
    if rc != 0:
        raise ValueError("more draws than candidates")
    return out


def priorities(N: int, seed: int, stream: int) -> np.ndarray:
    out = np.empty(N, dtype=np.uint32)
    _load().oracle_priorities(N, seed, stream, _ptr(out))
    return out


def fast_allocation(losses: np.ndarray, k: int, n_fill: int, seed: int, stream: int) -> np.ndarray:
    """The fast workers' samples: k highest-loss first, then n_fill drawn from the rest."""
    losses = np.ascontiguousarray(losses, dtype=np.float32)
    out = np.empty(k + n_fill, dtype=np.int32)
    rc = _load().oracle_fast_allocation(_ptr(losses), losses.size, k, n_fill, seed, stream, _ptr(out))
    if rc != 0:
        raise ValueError("k + n_fill exceeds N")
    return out


def aggregate_round(replicas, weights: np.ndarray, base: np.ndarray | None = None):
    """One round's aggregation in double: Eq. 3, or base + sum_i w_i (x_i - base) when `base` is given.

    replicas: float32 arrays, or uint16 arrays holding bf16 bit patterns.  Returns (out float64, out rounded to
    float32, that rounded to bf16 bits, error scale float64).
    """
    dt = F32 if replicas[0].dtype == np.float32 else BF16
    want = np.float32 if dt == F32 else np.uint16
    reps = [np.ascontiguousarray(r, dtype=want) for r in replicas]
    P, D = len(reps), reps[0].size
    assert all(r.size == D and r.dtype == want for r in reps)
    w = np.ascontiguousarray(weights, dtype=np.float32)
    assert w.size == P
    b = np.ascontiguousarray(base, dtype=np.float32) if base is not None else None
    assert b is None or b.size == D
    ptrs = (ctypes.c_void_p * P)(*[r.ctypes.data for r in reps])
    out = np.empty(D, dtype=np.float64)
    out32 = np.empty(D, dtype=np.float32)
    out16 = np.empty(D, dtype=np.uint16)
    mag = np.empty(D, dtype=np.float64)
    rc = _load().oracle_aggregate_round(ctypes.cast(ptrs, ctypes.c_void_p), dt, _ptr(w), P, D, _ptr(b), _ptr(out),
                                        _ptr(out32), _ptr(out16), _ptr(mag))
    assert rc == 0
    return out, out32, out16, mag
