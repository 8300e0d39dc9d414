"""Thin Python binding of liblsgd (include/lsgd.h): argument marshalling only.

Every function has the name and the meaning of its C entry point.  Tensors are
torch CUDA tensors (torch is used for device memory and the current stream);
nothing is computed here and there is no fallback: if liblsgd.so cannot be
loaded, or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblsgd.so")

F32, BF16 = 0, 1
ORDER_LOSS_DESC, ORDER_INDEX_ASC = 0, 1
MAX_REPLICAS = 64
IGNORE_INDEX = -100

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)

EXPORTS = (
    "lsgd_version", "lsgd_status_string", "lsgd_score_workspace_bytes", "lsgd_topk_workspace_bytes",
    "lsgd_score_topk_workspace_bytes", "lsgd_score_losses", "lsgd_topk_select", "lsgd_score_topk",
    "lsgd_aggregate", "lsgd_weights_from_steps", "lsgd_read_device_status", "lsgd_topk_select_static",
    "lsgd_allocation_sizes", "lsgd_worker_share", "lsgd_draw_workspace_bytes", "lsgd_draw_uniform",
    "lsgd_fast_allocation_workspace_bytes", "lsgd_fast_allocation", "lsgd_aggregate_round",
)
STATIC_TOPK_MAX_N = 262144


class LsgdError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2508_08540_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t, ctypes.c_int
        L.lsgd_version.restype = ci
        L.lsgd_status_string.restype = ctypes.c_char_p
        L.lsgd_status_string.argtypes = [ci]
        for name, args in (("lsgd_score_workspace_bytes", [i64, i64, i64]), ("lsgd_topk_workspace_bytes", [i64, i64]),
                           ("lsgd_score_topk_workspace_bytes", [i64, i64, i64, i64])):
            getattr(L, name).restype = sz
            getattr(L, name).argtypes = args
        L.lsgd_score_losses.argtypes = [vp, ci, vp, i64, i64, i64, i64, vp, vp, sz, vp]
        L.lsgd_topk_select.argtypes = [vp, i64, i64, ci, vp, vp, vp, sz, vp]
        L.lsgd_topk_select_static.argtypes = [vp, i64, i64, ci, vp, vp, vp]
        L.lsgd_topk_select_static.restype = ci
        L.lsgd_score_topk.argtypes = [vp, ci, vp, i64, i64, i64, i64, i64, ci, vp, vp, vp, vp, sz, vp]
        L.lsgd_aggregate.argtypes = [vp, vp, i32, i64, vp, vp]
        L.lsgd_aggregate_round.argtypes = [vp, ci, vp, i32, i64, vp, vp, i32, vp]
        L.lsgd_aggregate_round.restype = ci
        u64 = ctypes.c_uint64
        L.lsgd_allocation_sizes.argtypes = [i64, i32, i32, i32, i32, ctypes.c_double, vp, vp, vp]
        L.lsgd_worker_share.argtypes = [i64, i32, i32, vp, vp]
        L.lsgd_draw_workspace_bytes.argtypes = [i64, i64]
        L.lsgd_draw_workspace_bytes.restype = sz
        L.lsgd_draw_uniform.argtypes = [i64, i64, u64, u64, vp, i64, vp, vp, sz, vp]
        L.lsgd_fast_allocation_workspace_bytes.argtypes = [i64, i64, i64]
        L.lsgd_fast_allocation_workspace_bytes.restype = sz
        L.lsgd_fast_allocation.argtypes = [vp, i64, i64, i64, u64, u64, vp, vp, sz, vp]
        L.lsgd_weights_from_steps.argtypes = [vp, i32, vp]
        L.lsgd_read_device_status.argtypes = [vp, vp, vp]
        for name in ("lsgd_score_losses", "lsgd_topk_select", "lsgd_score_topk", "lsgd_aggregate",
                     "lsgd_weights_from_steps", "lsgd_read_device_status", "lsgd_allocation_sizes", "lsgd_worker_share",
                     "lsgd_draw_uniform", "lsgd_fast_allocation"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().lsgd_status_string(int(status)).decode()


def version() -> int:
    return lib().lsgd_version()


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _p(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _check(fn: str, st: int) -> None:
    if st != OK:
        raise LsgdError(fn, st)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("logits must be float32 or bfloat16")


def _pool_shape(logits: torch.Tensor, labels: torch.Tensor):
    if logits.dim() == 2:
        N, C = logits.shape
        T = 1
    elif logits.dim() == 3:
        N, T, C = logits.shape
    else:
        raise ValueError("logits must be [N, C] or [N, T, C]")
    if not logits.is_contiguous() or not labels.is_contiguous():
        raise ValueError("logits and labels must be contiguous")
    if labels.dtype != torch.int64 or labels.numel() != N * T:
        raise ValueError("labels must be int64 with N*T entries")
    return N, T, C


def score_workspace_bytes(N: int, T: int, C: int) -> int:
    return lib().lsgd_score_workspace_bytes(N, T, C)


def topk_workspace_bytes(N: int, k: int) -> int:
    return lib().lsgd_topk_workspace_bytes(N, k)


def score_topk_workspace_bytes(N: int, T: int, C: int, k: int) -> int:
    return lib().lsgd_score_topk_workspace_bytes(N, T, C, k)


def workspace(nbytes: int, device=None) -> torch.Tensor:
    """A caller-owned scratch tensor of at least `nbytes` (torch allocations are 512-byte aligned)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device or "cuda")


def score_losses(logits, labels, losses=None, ws=None, ignore_index: int = IGNORE_INDEX):
    """lsgd_score_losses: per-sample mean cross-entropy.  Returns `losses` ([N] fp32)."""
    N, T, C = _pool_shape(logits, labels)
    if losses is None:
        losses = torch.empty(N, dtype=torch.float32, device=logits.device)
    if ws is None:
        ws = workspace(score_workspace_bytes(N, T, C), logits.device)
    st = lib().lsgd_score_losses(_p(logits), _dtype_code(logits), _p(labels), N, T, C, ignore_index, _p(losses), _p(ws),
                                 ws.numel(), _stream())
    _check("lsgd_score_losses", st)
    return losses


def topk_select(losses, k: int, order: int = ORDER_LOSS_DESC, out_idx=None, out_vals=None, ws=None, want_vals=True):
    """lsgd_topk_select: the k highest losses, ties by lower index.  Returns (idx int32 [k], vals fp32 [k] or None)."""
    N = losses.numel()
    if out_idx is None:
        out_idx = torch.empty(max(k, 0), dtype=torch.int32, device=losses.device)
    if out_vals is None and want_vals:
        out_vals = torch.empty(max(k, 0), dtype=torch.float32, device=losses.device)
    if ws is None:
        ws = workspace(topk_workspace_bytes(N, k), losses.device)
    st = lib().lsgd_topk_select(_p(losses), N, k, order, _p(out_idx), _p(out_vals), _p(ws), ws.numel(), _stream())
    _check("lsgd_topk_select", st)
    return out_idx, out_vals


def topk_select_static(losses, k: int, out_idx, out_vals=None, order: int = ORDER_LOSS_DESC):
    """lsgd_topk_select_static: the selector on the library's built-in scratch array.

    For callers that must not allocate: the outputs are passed in, no workspace
    exists, and nothing is allocated here either.  N <= STATIC_TOPK_MAX_N.
    Calls share one scratch array per device: keep them on one stream.
    """
    st = lib().lsgd_topk_select_static(_p(losses), losses.numel(), k, order, _p(out_idx), _p(out_vals), _stream())
    _check("lsgd_topk_select_static", st)
    return out_idx, out_vals


def score_topk(logits, labels, k: int, order: int = ORDER_LOSS_DESC, losses=None, out_idx=None, out_vals=None, ws=None,
               ignore_index: int = IGNORE_INDEX, want_vals=True):
    """lsgd_score_topk: scorer + selector in one enqueued sequence.  Returns (losses, idx, vals)."""
    N, T, C = _pool_shape(logits, labels)
    dev = logits.device
    if losses is None:
        losses = torch.empty(N, dtype=torch.float32, device=dev)
    if out_idx is None:
        out_idx = torch.empty(max(k, 0), dtype=torch.int32, device=dev)
    if out_vals is None and want_vals:
        out_vals = torch.empty(max(k, 0), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(score_topk_workspace_bytes(N, T, C, k), dev)
    st = lib().lsgd_score_topk(_p(logits), _dtype_code(logits), _p(labels), N, T, C, ignore_index, k, order, _p(losses),
                               _p(out_idx), _p(out_vals), _p(ws), ws.numel(), _stream())
    _check("lsgd_score_topk", st)
    return losses, out_idx, out_vals


def aggregate(replicas, weights, out=None):
    """lsgd_aggregate: out = sum_i weights[i] * replicas[i] (Eq. 3).  `weights`: P host floats."""
    P = len(replicas)
    D = replicas[0].numel() if P else 0
    for r in replicas:
        if r.dtype != torch.float32 or r.numel() != D or not r.is_contiguous():
            raise ValueError("replicas must be contiguous float32 tensors of one size")
    if out is None:
        out = torch.empty(D, dtype=torch.float32, device=replicas[0].device)
    ptrs = (ctypes.c_void_p * max(P, 1))(*[r.data_ptr() for r in replicas])
    w = (ctypes.c_float * max(P, 1))(*[float(x) for x in weights])
    if len(weights) != P:
        raise ValueError("one weight per replica")
    st = lib().lsgd_aggregate(ctypes.cast(ptrs, ctypes.c_void_p), ctypes.cast(w, ctypes.c_void_p), P, D, _p(out), _stream())
    _check("lsgd_aggregate", st)
    return out


def aggregate_round(replicas, weights, base=None, out=None, broadcast: bool = False, want_out: bool = True):
    """lsgd_aggregate_round: Eq. 3 (around `base` if given) over fp32 or bf16 replicas; optionally written back into them."""
    P = len(replicas)
    D = replicas[0].numel() if P else 0
    dt = _dtype_code(replicas[0]) if P else F32
    for r in replicas:
        if r.dtype != replicas[0].dtype or r.numel() != D or not r.is_contiguous():
            raise ValueError("replicas must be contiguous tensors of one dtype and size")
    if len(weights) != P:
        raise ValueError("one weight per replica")
    if base is not None and (base.dtype != torch.float32 or base.numel() != D or not base.is_contiguous()):
        raise ValueError("base must be a contiguous float32 tensor of D elements")
    if out is None and (want_out or not broadcast):
        out = torch.empty(D, dtype=torch.float32, device=replicas[0].device)
    ptrs = (ctypes.c_void_p * max(P, 1))(*[r.data_ptr() for r in replicas])
    w = (ctypes.c_float * max(P, 1))(*[float(x) for x in weights])
    st = lib().lsgd_aggregate_round(ctypes.cast(ptrs, ctypes.c_void_p), dt, ctypes.cast(w, ctypes.c_void_p), P, D, _p(base),
                                    _p(out), 1 if broadcast else 0, _stream())
    _check("lsgd_aggregate_round", st)
    return out


def allocation_sizes(N: int, tau_fast: int, p_fast: int, tau_slow: int, p_slow: int, lam: float):
    """lsgd_allocation_sizes: (N_F, N_S, k) of Section 4.2.  Host only."""
    nf, ns, k = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    st = lib().lsgd_allocation_sizes(N, tau_fast, p_fast, tau_slow, p_slow, lam, ctypes.byref(nf), ctypes.byref(ns),
                                     ctypes.byref(k))
    _check("lsgd_allocation_sizes", st)
    return nf.value, ns.value, k.value


def worker_share(n: int, P: int, p: int):
    """lsgd_worker_share: [begin, end) of worker p's part of an n-entry list.  Host only."""
    b, e = ctypes.c_int64(0), ctypes.c_int64(0)
    _check("lsgd_worker_share", lib().lsgd_worker_share(n, P, p, ctypes.byref(b), ctypes.byref(e)))
    return b.value, e.value


def draw_workspace_bytes(N: int, n_draw: int) -> int:
    return lib().lsgd_draw_workspace_bytes(N, n_draw)


def fast_allocation_workspace_bytes(N: int, k_high: int, n_fill: int) -> int:
    return lib().lsgd_fast_allocation_workspace_bytes(N, k_high, n_fill)


def draw_uniform(N: int, n_draw: int, seed: int, stream: int, exclude_idx=None, out_idx=None, ws=None, device=None):
    """lsgd_draw_uniform: n_draw of the N samples (minus exclude_idx), uniformly without replacement."""
    dev = exclude_idx.device if exclude_idx is not None else (device or "cuda")
    if out_idx is None:
        out_idx = torch.empty(max(n_draw, 0), dtype=torch.int32, device=dev)
    if ws is None:
        ws = workspace(draw_workspace_bytes(N, n_draw), dev)
    n_ex = exclude_idx.numel() if exclude_idx is not None else 0
    if exclude_idx is not None and (exclude_idx.dtype != torch.int32 or not exclude_idx.is_contiguous()):
        raise ValueError("exclude_idx must be a contiguous int32 tensor")
    st = lib().lsgd_draw_uniform(N, n_draw, seed, stream, _p(exclude_idx), n_ex, _p(out_idx), _p(ws), ws.numel(), _stream())
    _check("lsgd_draw_uniform", st)
    return out_idx


def fast_allocation(losses, k_high: int, n_fill: int, seed: int, stream: int, out_idx=None, ws=None):
    """lsgd_fast_allocation: the k_high highest-loss samples, then n_fill drawn from the rest."""
    N = losses.numel()
    if losses.dtype != torch.float32 or not losses.is_contiguous():
        raise ValueError("losses must be a contiguous float32 tensor")
    if out_idx is None:
        out_idx = torch.empty(max(k_high + n_fill, 0), dtype=torch.int32, device=losses.device)
    if ws is None:
        ws = workspace(fast_allocation_workspace_bytes(N, k_high, n_fill), losses.device)
    st = lib().lsgd_fast_allocation(_p(losses), N, k_high, n_fill, seed, stream, _p(out_idx), _p(ws), ws.numel(), _stream())
    _check("lsgd_fast_allocation", st)
    return out_idx


def weights_from_steps(tau) -> list[float]:
    """lsgd_weights_from_steps: w_i = tau_i / sum(tau) (Eq. 3), rounded to fp32.  Host only."""
    P = len(tau)
    t = (ctypes.c_int32 * max(P, 1))(*[int(x) for x in tau])
    w = (ctypes.c_float * max(P, 1))()
    st = lib().lsgd_weights_from_steps(ctypes.cast(t, ctypes.c_void_p), P, ctypes.cast(w, ctypes.c_void_p))
    _check("lsgd_weights_from_steps", st)
    return [w[i] for i in range(P)]


def read_device_status(ws) -> int:
    """lsgd_read_device_status: bad-label count of the last call that used `ws` (synchronises the stream)."""
    bad = ctypes.c_int32(0)
    st = lib().lsgd_read_device_status(_p(ws), ctypes.byref(bad), _stream())
    _check("lsgd_read_device_status", st)
    return bad.value
