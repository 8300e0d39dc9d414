#!/usr/bin/env python
"""Benchmark of the biased-local-SGD hot path on B200.

One "step" is one pass of the whole hot path over one synthetic round:
    lsgd_score_topk  (per-sample loss record + deterministic top-k, Section 4.2)
    lsgd_aggregate   (Eq. 3)
with the step-count weights of Eq. 3 computed once by lsgd_weights_from_steps
where the round uses them.  Inputs are resident in HBM for `value`; the `e2e`
leg repeats the step with host->device copies of all inputs from pinned memory
and device->host copies of the results inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead
(bounded samples of the same workload on the host cores).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2508_08540_b200 import workloads as wl  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


# --------------------------------------------------------------------------- #
# algorithmic bytes
# --------------------------------------------------------------------------- #
def score_topk_bytes(cfg, labels: np.ndarray) -> int:
    """Scorer: logits + loss of every unmasked row, every label; selector: the loss table read once, k indices and values."""
    es = 4 if cfg.dtype == "f32" else 2
    unmasked = int((labels != wl.IGNORE_INDEX).sum())
    rows = labels.size
    b = unmasked * (cfg.C * es + 4) + rows * 8
    b += 4 * cfg.N + 8 * cfg.k
    return b


def aggregate_bytes(cfg) -> int:
    return 4 * cfg.D * (cfg.P + 1)


# --------------------------------------------------------------------------- #
# clocks (read-only NVML sampling while the timed region runs)
# --------------------------------------------------------------------------- #
class ClockSampler:
    def __init__(self, index: int, period_s: float = 0.003):
        self.samples, self.reasons, self.sm_max = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.period = period_s

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake_slowdown": 0x80, "applications_clocks_setting": 0x2, "sync_boost": 0x10}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._t:
            self._t.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.sm_max, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- #
# CPU oracle timing (bounded samples)
# --------------------------------------------------------------------------- #
def oracle_sample(cfg, n_samples: int, d_elems: int):
    """Inputs for an oracle run on the first n_samples samples and the first d_elems parameters."""
    x, y = wl.pool_rows(cfg, 0, n_samples)
    reps = [wl.replica_slice(cfg, i, 0, d_elems) for i in range(cfg.P)]
    return x, y, reps


def round_weights_oracle(cfg, oracle):
    return oracle.weights_from_steps(wl.step_counts(cfg)) if cfg.weight_mode == "steps" else wl.weight_draws(cfg)


def time_oracle_step(oracle, cfg, x, y, reps, w):
    n = x.shape[0]
    k = max(1, min(n, round(cfg.k * n / cfg.N)))
    t0 = time.perf_counter()
    loss, _ = oracle.score(x, y)
    oracle.topk(loss.astype(np.float32), k, oracle.LOSS_DESC)
    t1 = time.perf_counter()
    oracle.aggregate(reps, w)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def calibrate_oracle(oracle, cfg, budget_s: float):
    """Sample sizes (samples, parameters) whose oracle run takes about budget_s (2/3 scoring, 1/3 aggregation)."""
    n0 = max(1, min(cfg.N, 4096 // max(1, cfg.T * cfg.C // 1000 + 1)))
    d0 = min(cfg.D, 1 << 18)
    x, y, reps = oracle_sample(cfg, n0, d0)
    w = round_weights_oracle(cfg, oracle)
    ts, ta = time_oracle_step(oracle, cfg, x, y, reps, w)
    n = int(max(1, min(cfg.N, n0 * (budget_s * 2 / 3) / max(ts, 1e-6))))
    d = int(max(1024, min(cfg.D, d0 * (budget_s / 3) / max(ta, 1e-6))))
    return n, d


def cpu_baseline(cfg, budget_s: float = 12.0):
    from oracle import oracle

    oracle.build()
    n, d = calibrate_oracle(oracle, cfg, budget_s)
    x, y, reps = oracle_sample(cfg, n, d)
    w = round_weights_oracle(cfg, oracle)
    ts, ta = time_oracle_step(oracle, cfg, x, y, reps, w)
    return {
        "value": n / ts, "unit": "samples/s", "cores": 1, "kind": "oracle",
        "sample": f"first {n} of {cfg.N} samples scored + top-k of them; aggregation of the first {d} of {cfg.D} parameters "
                  f"of all {cfg.P} replicas",
        "score_topk_s": ts, "aggregate_s": ta, "aggregate_gbs": 4 * d * (cfg.P + 1) / ta / 1e9,
        "host_cores_available": os.cpu_count(),
    }


def run_reference(args, cfg):
    """--impl reference: the CPU oracle, as it stands, on bounded samples of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle

    oracle.build()
    per_step = max(0.05, min(10.0, 90.0 / (args.steps + args.warmup)))
    n, d = calibrate_oracle(oracle, cfg, per_step)
    x, y, reps = oracle_sample(cfg, n, d)
    w = round_weights_oracle(cfg, oracle)
    for _ in range(args.warmup):
        time_oracle_step(oracle, cfg, x, y, reps, w)
    ts = ta = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a, b = time_oracle_step(oracle, cfg, x, y, reps, w)
        ts += a
        ta += b
    total = time.perf_counter() - t0
    value = n * args.steps / ts
    sample = (f"each step: first {n} of {cfg.N} samples scored + top-k of them, aggregation of the first {d} of {cfg.D} "
              f"parameters of all {cfg.P} replicas")
    line = {
        "impl": "reference", "metric": "score+top-k samples/s", "value": value, "unit": "samples/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg), "inputs": "host memory; CPU oracle",
        "aggregation": {"value": 4 * d * (cfg.P + 1) * args.steps / ta / 1e9, "unit": "GB/s"},
        "cpu_baseline": {"value": value, "unit": "samples/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of `values` over all ranks (identity without a process group).

    Every multi-GPU number is the slowest rank's: ranks run independent replicas of the round,
    so the job is as fast as its slowest member.
    """
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world: int, units_per_rank: float, steps: int, ms: float) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` per step, in `ms` (max over ranks)."""
    return world * units_per_rank * steps / (ms * 1e-3)


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernels, from ncu captures of
# scaled-down cases (128 of config 4's 1,024 sequences; 16,000,000 of its 109,482,240 parameters per replica), scaled
# to a full launch by the units processed.  Valid only for the kernels as captured: reset to None whenever
# score_stream_rows_kernel or aggregate_vec4_kernel changes, until the counters have been taken again.
NCU_TRAFFIC_BYTES = {
    ("score", 4): 7.27e9,      # 908.5 MB for 128 of 1,024 sequences
    ("aggregate", 4): 4.77e9,  # 697.3 MB for 16,000,000 of 109,482,240 parameters
}


def workload_config(cfg):
    return {
        "workload": f"config {cfg.cfg_id} ({cfg.name}-scale round): pool {cfg.N} x {cfg.T} x {cfg.C} {cfg.dtype} logits, "
                    f"k={cfg.k}; {cfg.P} replicas x {cfg.D} fp32 parameters",
        "N": cfg.N, "T": cfg.T, "C": cfg.C, "k": cfg.k, "P": cfg.P, "D": cfg.D, "order": "loss_desc",
        "l2": "inputs larger than L2 (no flush needed)" if cfg.logit_bytes > (1 << 28) else "L2 flushed between steps",
    }


# --------------------------------------------------------------------------- #
# GPU arm
# --------------------------------------------------------------------------- #
def run_gpu(args, cfg):
    import torch
    import torch.distributed as dist

    from paper_2508_08540_b200 import lsgd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    lsgd.lib()

    # ---- inputs: generated on the host into pinned memory, then made resident
    t_gen = time.perf_counter()
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    h_logits = torch.empty((cfg.N, cfg.T, cfg.C), dtype=tdt, pin_memory=True)
    h_labels = torch.empty((cfg.N, cfg.T), dtype=torch.int64, pin_memory=True)
    np_logits = h_logits.view(torch.int16).numpy().view(np.uint16) if cfg.dtype == "bf16" else h_logits.numpy()
    step = max(1, (1 << 28) // max(1, cfg.T * cfg.C * np_logits.itemsize))
    for s0 in range(0, cfg.N, step):
        s1 = min(cfg.N, s0 + step)
        x, y = wl.pool_rows(cfg, s0, s1)
        np_logits[s0:s1] = x
        h_labels.numpy()[s0:s1] = y
    h_reps = [torch.empty(cfg.D, dtype=torch.float32, pin_memory=True) for _ in range(cfg.P)]
    for i in range(cfg.P):
        wl.replica_slice(cfg, i, out=h_reps[i].numpy())
    if cfg.weight_mode == "steps":
        weights = lsgd.weights_from_steps(wl.step_counts(cfg).tolist())
    else:
        weights = wl.weight_draws(cfg).tolist()
    gen_s = time.perf_counter() - t_gen

    d_logits = h_logits.to(dev, non_blocking=True)
    d_labels = h_labels.to(dev, non_blocking=True)
    d_reps = [r.to(dev, non_blocking=True) for r in h_reps]
    losses = torch.empty(cfg.N, dtype=torch.float32, device=dev)
    idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    vals = torch.empty(cfg.k, dtype=torch.float32, device=dev)
    out = torch.empty(cfg.D, dtype=torch.float32, device=dev)
    ws = lsgd.workspace(lsgd.score_topk_workspace_bytes(cfg.N, cfg.T, cfg.C, cfg.k), dev)
    flush = None if cfg.logit_bytes > (1 << 28) else torch.empty(1 << 28, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    def step_resident(ev=None):
        if flush is not None:
            flush.fill_(1)
        if ev:
            ev[0].record()
        lsgd.score_topk(d_logits, d_labels, cfg.k, lsgd.ORDER_LOSS_DESC, losses=losses, out_idx=idx, out_vals=vals, ws=ws)
        if ev:
            ev[1].record()
        lsgd.aggregate(d_reps, weights, out=out)
        if ev:
            ev[2].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step_resident()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        barrier()
        start.record()
        for i in range(args.steps):
            step_resident(evs[i])
        end.record()
        barrier()
    total_ms = start.elapsed_time(end)
    st_ms = np.array([e[0].elapsed_time(e[1]) for e in evs])
    ag_ms = np.array([e[1].elapsed_time(e[2]) for e in evs])
    bad = lsgd.read_device_status(ws)
    # pools that fit in L2 were timed cold (flushed before every step); also give the warm figure
    warm = None
    if flush is not None:
        # the two calls captured once each into CUDA graphs and replayed: the device's time for a step whose inputs
        # may sit in L2, without the host's enqueue cost (which bounds eagerly launched steps shorter than ~60 us)
        side = torch.cuda.Stream()
        graphs = []
        with torch.cuda.stream(side):
            for call in (lambda: lsgd.score_topk(d_logits, d_labels, cfg.k, lsgd.ORDER_LOSS_DESC, losses=losses, out_idx=idx,
                                                 out_vals=vals, ws=ws),
                         lambda: lsgd.aggregate(d_reps, weights, out=out)):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    call()
                graphs.append(g)
        torch.cuda.synchronize()
        w_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(23)]
        for e in w_ev:
            e[0].record()
            graphs[0].replay()
            e[1].record()
            graphs[1].replay()
            e[2].record()
        torch.cuda.synchronize()
        warm = {"score_topk_ms": float(np.median([e[0].elapsed_time(e[1]) for e in w_ev[3:]])),
                "aggregate_ms": float(np.median([e[1].elapsed_time(e[2]) for e in w_ev[3:]])),
                "note": "the same two calls replayed from CUDA graphs without the L2 flush (inputs may be L2-resident); median of 20"}

    # ---- end to end: inputs from pinned host memory, results back to the host, every step
    e2e_steps = max(1, min(args.steps, 5 if cfg.logit_bytes > (1 << 30) else 20))
    h_idx = torch.empty(cfg.k, dtype=torch.int32, pin_memory=True)
    h_vals = torch.empty(cfg.k, dtype=torch.float32, pin_memory=True)
    h_out = torch.empty(cfg.D, dtype=torch.float32, pin_memory=True)
    h2d_st = h_logits.numel() * h_logits.element_size() + h_labels.numel() * 8
    d2h_st = cfg.k * 8
    h2d = h2d_st + cfg.P * cfg.D * 4
    d2h = d2h_st + cfg.D * 4

    def step_e2e(ev=None):
        if ev:
            ev[0].record()
        d_logits.copy_(h_logits, non_blocking=True)
        d_labels.copy_(h_labels, non_blocking=True)
        lsgd.score_topk(d_logits, d_labels, cfg.k, lsgd.ORDER_LOSS_DESC, losses=losses, out_idx=idx, out_vals=vals, ws=ws)
        h_idx.copy_(idx, non_blocking=True)
        h_vals.copy_(vals, non_blocking=True)
        if ev:
            ev[1].record()
        for d, h in zip(d_reps, h_reps):
            d.copy_(h, non_blocking=True)
        lsgd.aggregate(d_reps, weights, out=out)
        h_out.copy_(out, non_blocking=True)
        if ev:
            ev[2].record()

    e2e_ms = e2e_st_ms = float("nan")
    if not args.no_e2e:
        step_e2e()
        barrier()
        e_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(e2e_steps)]
        for i in range(e2e_steps):
            step_e2e(e_ev[i])
        barrier()
        e2e_st_ms = float(sum(e[0].elapsed_time(e[1]) for e in e_ev))
        e2e_ms = float(e_ev[0][0].elapsed_time(e_ev[-1][2]))

    # ---- the epoch's data allocation (Section 4.2) on the loss table just written: fast workers' list
    # (top-k + random fill) and the slow workers' independent draw, in the paper's 8-fast / 2-slow setting
    n_fast, n_slow, _ = lsgd.allocation_sizes(cfg.N, 32, 8, 1, 2, 1.0)
    k_high = min(cfg.k, n_fast)
    n_fill = n_fast - k_high
    a_idx = torch.empty(n_fast + n_slow, dtype=torch.int32, device=dev)
    a_ws = lsgd.workspace(max(lsgd.fast_allocation_workspace_bytes(cfg.N, k_high, n_fill),
                              lsgd.draw_workspace_bytes(cfg.N, n_slow)), dev)
    a_steps = 20
    a_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(a_steps)]
    for i in range(3 + a_steps):
        ev = a_ev[i - 3] if i >= 3 else None
        if ev:
            ev[0].record()
        lsgd.fast_allocation(losses, k_high, n_fill, cfg.seed, 2 * i, out_idx=a_idx[:n_fast], ws=a_ws)
        if ev:
            ev[1].record()
        lsgd.draw_uniform(cfg.N, n_slow, cfg.seed, 2 * i + 1, out_idx=a_idx[n_fast:], ws=a_ws)
        if ev:
            ev[2].record()
    torch.cuda.synchronize()
    fast_ms = float(np.median([e[0].elapsed_time(e[1]) for e in a_ev]))
    slow_ms = float(np.median([e[1].elapsed_time(e[2]) for e in a_ev]))

    # ---- the round's aggregation as the training loop uses it: around x_t, written back into the replicas,
    # fp32 and bf16 replicas (lsgd_aggregate_round); median of 10 calls each, outside the timed step
    round_legs = {}
    if not args.no_round:
        d_base = torch.empty(cfg.D, dtype=torch.float32, device=dev)
        d_base.copy_(d_reps[0])
        d_reps16 = [r.to(torch.bfloat16) for r in d_reps]
        for name, reps_, es, use_base, bcast in (("f32_delta_broadcast", d_reps, 4, True, True),
                                                 ("bf16_plain", d_reps16, 2, False, False),
                                                 ("bf16_delta_broadcast", d_reps16, 2, True, True)):
            r_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(10)]
            for i in range(13):
                if i >= 3:
                    r_ev[i - 3][0].record()
                lsgd.aggregate_round(reps_, weights, base=d_base if use_base else None, out=out, broadcast=bcast)
                if i >= 3:
                    r_ev[i - 3][1].record()
            torch.cuda.synchronize()
            ms = float(np.median([e[0].elapsed_time(e[1]) for e in r_ev]))
            nbytes = cfg.D * (cfg.P * es * (2 if bcast else 1) + (4 if use_base else 0) + 4)
            round_legs[name] = {"ms": ms, "algorithmic_bytes": nbytes, "gbs": nbytes / ms / 1e6}
        del d_reps16, d_base

    total_ms, st_sum, ag_sum, e2e_ms, e2e_st_ms = max_over_ranks(
        [total_ms, float(st_ms.sum()), float(ag_ms.sum()), e2e_ms, e2e_st_ms], dev)
    if rank == 0:
        peak, peak_src = measured_peak()
        st_bytes = score_topk_bytes(cfg, h_labels.numpy())
        ag_bytes = aggregate_bytes(cfg)
        st_gbs = st_bytes * args.steps / (st_sum * 1e-3) / 1e9
        ag_gbs = ag_bytes * args.steps / (ag_sum * 1e-3) / 1e9
        n_launch = launches_per_step(cfg)
        line = {
            "metric": "score+top-k samples/s", "value": job_throughput(world, cfg.N, args.steps, st_sum), "unit": "samples/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(cfg), "inputs": "resident in HBM",
            "score_topk": {"ms": st_sum / args.steps, "ms_median": float(np.median(st_ms)), "ms_best": float(st_ms.min()), "gbs": st_gbs,
                           "frac_of_measured_hbm": st_gbs / peak, "frac_of_nominal_8tbs": st_gbs / NOMINAL_HBM_GBS,
                           "algorithmic_bytes": st_bytes, "bad_labels": bad},
            "aggregation": {"value": world * ag_gbs, "unit": "GB/s", "ms": ag_sum / args.steps, "ms_median": float(np.median(ag_ms)), "ms_best": float(ag_ms.min()),
                            "frac_of_measured_hbm": ag_gbs / peak, "frac_of_nominal_8tbs": ag_gbs / NOMINAL_HBM_GBS,
                            "algorithmic_bytes": ag_bytes},
            "warm": warm,
            "round_samples_per_s": world * cfg.N * args.steps / (total_ms * 1e-3),
            "roofline": {"bound": "hbm", "kernel": "lsgd_score_topk (clearing kernel, scorer kernel, sequence mean, selector)",
                         "achieved": st_gbs, "peak": peak, "unit": "GB/s", "frac": st_gbs / peak,
                         "traffic": NCU_TRAFFIC_BYTES.get(("score", cfg.cfg_id)) if not (args.n_samples or args.d_params) else None,
                         "peak_source": peak_src},
            "roofline_aggregate": {"bound": "hbm", "kernel": "aggregate_vec4_kernel", "achieved": ag_gbs, "peak": peak,
                                   "unit": "GB/s", "frac": ag_gbs / peak,
                                   "traffic": NCU_TRAFFIC_BYTES.get(("aggregate", cfg.cfg_id)) if not (args.n_samples or args.d_params) else None,
                                   "peak_source": peak_src},
            "e2e": {"value": world * cfg.N * e2e_steps / (e2e_st_ms * 1e-3), "unit": "samples/s",
                    "ms_per_step": e2e_st_ms / e2e_steps, "steps": e2e_steps,
                    "h2d_bytes_per_step": h2d_st, "d2h_bytes_per_step": d2h_st,
                    "note": "score+top-k with logits and labels copied from pinned host memory and the k indices and "
                            "losses copied back, every step; bound by the host link",
                    "whole_step": {"ms_per_step": e2e_ms / e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                                   "note": "adds the replicas' upload, the aggregation and the download of its result"}},
            "allocation": {"n_fast": n_fast, "k_high": k_high, "n_fill": n_fill, "n_slow": n_slow,
                           "fast_allocation_ms": fast_ms, "slow_draw_ms": slow_ms,
                           "note": "Section 4.2 lists for 8 fast (tau 32) + 2 slow (tau 1) workers from the resident loss "
                                   "table; median of 20 calls, outside the timed step"},
            "aggregation_round": round_legs,
            "gpu_launches": n_launch * args.steps,
            "clocks": clocks.summary(),
            "input_generation_s": gen_s,
        }
        if world == 1 and not args.no_other_configs and not (args.n_samples or args.d_params):
            # the other four rounds, briefly, so that one run gives every configuration's figures from the same device
            line["other_configs"] = {str(c): other_config_leg(wl.CONFIGS[c], dev, min(args.steps, 20), peak)
                                     for c in sorted(wl.CONFIGS) if c != cfg.cfg_id}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def other_config_leg(cfg, dev, steps: int, peak: float) -> dict:
    """One of the other four rounds, timed briefly in the same process: the same two calls on that round's shapes,
    inputs resident, L2 flushed before every step where the pool fits in it.  Mean and median over `steps` steps."""
    import torch

    from paper_2508_08540_b200 import lsgd

    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    d_logits = torch.empty((cfg.N, cfg.T, cfg.C), dtype=tdt, device=dev)
    d_labels = torch.empty((cfg.N, cfg.T), dtype=torch.int64, device=dev)
    es = d_logits.element_size()
    slab = max(1, (1 << 28) // max(1, cfg.T * cfg.C * es))
    unmasked = 0
    for s0 in range(0, cfg.N, slab):
        s1 = min(cfg.N, s0 + slab)
        x, y = wl.pool_rows(cfg, s0, s1)
        unmasked += int((y != wl.IGNORE_INDEX).sum())
        hx = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) if cfg.dtype == "bf16" else torch.from_numpy(x)
        d_logits[s0:s1].copy_(hx.reshape(s1 - s0, cfg.T, cfg.C))
        d_labels[s0:s1].copy_(torch.from_numpy(y).reshape(s1 - s0, cfg.T))
    d_reps = []
    for i in range(cfg.P):
        h = np.empty(cfg.D, dtype=np.float32)
        wl.replica_slice(cfg, i, out=h)
        d_reps.append(torch.from_numpy(h).to(dev))
    weights = (lsgd.weights_from_steps(wl.step_counts(cfg).tolist()) if cfg.weight_mode == "steps"
               else wl.weight_draws(cfg).tolist())
    losses = torch.empty(cfg.N, dtype=torch.float32, device=dev)
    idx = torch.empty(cfg.k, dtype=torch.int32, device=dev)
    vals = torch.empty(cfg.k, dtype=torch.float32, device=dev)
    out = torch.empty(cfg.D, dtype=torch.float32, device=dev)
    ws = lsgd.workspace(lsgd.score_topk_workspace_bytes(cfg.N, cfg.T, cfg.C, cfg.k), dev)
    flush = None if cfg.logit_bytes > (1 << 28) else torch.empty(1 << 28, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    for i in range(3 + steps):
        ev = evs[i - 3] if i >= 3 else None
        if flush is not None:
            flush.fill_(1)
        if ev:
            ev[0].record()
        lsgd.score_topk(d_logits, d_labels, cfg.k, lsgd.ORDER_LOSS_DESC, losses=losses, out_idx=idx, out_vals=vals, ws=ws)
        if ev:
            ev[1].record()
        lsgd.aggregate(d_reps, weights, out=out)
        if ev:
            ev[2].record()
    torch.cuda.synchronize()
    st = np.array([e[0].elapsed_time(e[1]) for e in evs])
    ag = np.array([e[1].elapsed_time(e[2]) for e in evs])
    st_bytes = unmasked * (cfg.C * es + 4) + cfg.N * cfg.T * 8 + 4 * cfg.N + 8 * cfg.k
    ag_bytes = aggregate_bytes(cfg)
    st_gbs = st_bytes / (st.mean() * 1e-3) / 1e9
    ag_gbs = ag_bytes / (ag.mean() * 1e-3) / 1e9
    bad = lsgd.read_device_status(ws)
    del d_logits, d_labels, d_reps, losses, idx, vals, out, ws, flush
    torch.cuda.empty_cache()  # the next round's buffers are mapped afresh, not carved out of this round's
    return {"workload": workload_config(cfg)["workload"], "steps": steps, "l2": workload_config(cfg)["l2"],
            "bad_labels": bad,
            "score_topk": {"samples_per_s": cfg.N / (st.mean() * 1e-3), "ms": float(st.mean()), "ms_median": float(np.median(st)),
                           "gbs": st_gbs, "frac_of_measured_hbm": st_gbs / peak, "frac_of_nominal_8tbs": st_gbs / NOMINAL_HBM_GBS,
                           "algorithmic_bytes": st_bytes},
            "aggregation": {"ms": float(ag.mean()), "ms_median": float(np.median(ag)), "gbs": ag_gbs,
                            "frac_of_measured_hbm": ag_gbs / peak, "frac_of_nominal_8tbs": ag_gbs / NOMINAL_HBM_GBS,
                            "algorithmic_bytes": ag_bytes}}


def launches_per_step(cfg) -> int:
    """Kernels of liblsgd launched by one step, from the launch logic of the library."""
    n = 1                                           # the kernel that clears the head of the workspace
    n += 1 + (1 if cfg.T > 1 else 0)                # scorer (+ sequence mean)
    n += 1                                          # the selector is one kernel at every pool size
    n += 1                                          # aggregation
    return n


SWEEP_SHAPES = (  # rows, classes, dtype: one row shape per scorer kernel and regime, each pool larger than L2
    (20_000_000, 10, "f32"), (12_000_000, 32, "bf16"),
    (8_000_000, 48, "f32"), (5_000_000, 100, "f32"), (4_000_000, 200, "f32"), (2_000_000, 500, "f32"),
    (1_281_167, 1000, "f32"), (640_000, 2000, "f32"), (150_000, 8000, "f32"), (40_000, 30522, "f32"),
    (6_000_000, 100, "bf16"), (3_000_000, 300, "bf16"), (2_000_000, 1000, "bf16"), (1_000_000, 2000, "bf16"),
    (400_000, 4000, "bf16"), (300_000, 8000, "bf16"), (100_000, 16000, "bf16"), (131_072, 30522, "bf16"),
)


def run_scorer_sweep(args):
    """--sweep-scorer: lsgd_score_losses over a range of row lengths (seeded normal logits, sigma 2, uniform labels),
    and some of them again with confident rows."""
    import torch

    from paper_2508_08540_b200 import lsgd

    torch.cuda.set_device(0)
    peak, peak_src = measured_peak()
    out = []
    shapes = [(r, C, dt, 0.0) for r, C, dt in SWEEP_SHAPES]
    # the same pools from a model that is sure of its answer (true class + 14: p > 0.99, losses ~ 1e-3): the regime
    # in which the loss keeps its relative accuracy only through the max-excluded sum
    shapes += [(r, C, dt, 14.0) for r, C, dt in SWEEP_SHAPES if (C, dt) in ((100, "f32"), (1000, "f32"), (8000, "f32"),
                                                                           (300, "bf16"), (4000, "bf16"), (30522, "bf16"))]
    if args.sweep_filter:  # "C:dtype[:rows]": that row shape alone (profiling runs), optionally with fewer rows
        f = args.sweep_filter.split(":")
        shapes = [(int(f[2]) if len(f) > 2 else r, C, dt, b) for r, C, dt, b in shapes if C == int(f[0]) and dt == f[1] and b == 0.0]
    for rows, C, dt, bump in shapes:
        tdt = torch.float32 if dt == "f32" else torch.bfloat16
        g = torch.Generator(device="cuda").manual_seed(MASTER_SWEEP_SEED + C)
        x = torch.empty((rows, C), dtype=tdt, device="cuda")
        y = torch.randint(0, C, (rows,), device="cuda", generator=g)
        step = max(1, (1 << 28) // C)
        for r0 in range(0, rows, step):  # filled in slices: no fp32 copy of the whole pool
            r1 = min(rows, r0 + step)
            blk = torch.randn((r1 - r0, C), device="cuda", generator=g).mul_(2.0)
            if bump:
                blk[torch.arange(r1 - r0, device="cuda"), y[r0:r1]] += bump
            x[r0:r1] = blk.to(tdt)
            del blk
        losses = torch.empty(rows, dtype=torch.float32, device="cuda")
        ws = lsgd.workspace(lsgd.score_workspace_bytes(rows, 1, C), "cuda")
        for _ in range(3):
            lsgd.score_losses(x, y, losses=losses, ws=ws)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in ev:
            a.record()
            lsgd.score_losses(x, y, losses=losses, ws=ws)
            b.record()
        torch.cuda.synchronize()
        ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
        nbytes = rows * (C * x.element_size() + 12)
        out.append({"rows": rows, "C": C, "dtype": dt, "true_class_bump": bump, "row_bytes": C * x.element_size(), "ms": ms,
                    "gbs": nbytes / ms / 1e6, "frac_of_measured_hbm": nbytes / ms / 1e6 / peak})
        del x, y, losses, ws
        torch.cuda.empty_cache()  # every shape starts from freshly mapped memory
    print(json.dumps({"metric": "scorer GB/s by row shape", "unit": "GB/s", "peak": peak, "peak_source": peak_src,
                      "steps": args.steps, "data": "synthetic", "shapes": out}), flush=True)


MASTER_SWEEP_SEED = 20250808


def spawn_ranks(n: int, argv, timeout_s: float | None = None) -> int:
    """Starts `n` copies of the command `argv`, one per GPU of this node, with the environment a torchrun launch
    would give them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, a free MASTER_PORT), and waits for them.
    The children share this process's stdout (rank 0 prints the JSON line).  Returns the worst exit code.
    The ranks run independent replicas of the round; they only meet for barriers and the max over their timings."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env))
    worst = 0
    for pr in procs:
        try:
            rc = pr.wait(timeout=timeout_s)
        except subprocess.TimeoutExpired:
            pr.kill()
            rc = 124
        worst = max(worst, abs(rc))
    return worst


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4, choices=sorted(wl.CONFIGS))
    ap.add_argument("--impl", default="lsgd", choices=["lsgd", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep-scorer", action="store_true",
                    help="instead of the round: time lsgd_score_losses alone over a range of row lengths (1 GPU)")
    ap.add_argument("--sweep-filter", default="", help="with --sweep-scorer: only the row shape C:dtype[:rows]")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the brief legs over the other four rounds")
    ap.add_argument("--no-round", action="store_true", help="skip the lsgd_aggregate_round legs (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--n-samples", type=int, default=0, help="profiling: shrink the pool to this many samples")
    ap.add_argument("--d-params", type=int, default=0, help="profiling: shrink each replica to this many parameters")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.config]
    if args.n_samples or args.d_params:
        n = args.n_samples or cfg.N
        cfg = wl.scaled(cfg, name=cfg.name + "-scaled", N=n, k=max(1, cfg.k * n // cfg.N), D=args.d_params or cfg.D)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference" and not args.sweep_scorer:
        # started plainly with --gpus N: become the launcher of N ranks (under torchrun the environment is already set)
        sys.exit(spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    if args.sweep_scorer:
        args.steps = min(args.steps, 20)
        run_scorer_sweep(args)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()
