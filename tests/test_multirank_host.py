"""Host-side logic of the multi-rank benchmark on CPU (gloo, world size 2): the path has no
data-path collective (ranks run independent replicas of the round), only the max-over-ranks of
the timings and the whole-job throughput."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + rank, 5.0 - rank, 7.0]
    got = bench.max_over_ranks(mine)
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = got


def test_max_over_ranks_and_throughput_gloo():
    import bench

    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29731, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0, 7.0]
    # without a process group it is the identity
    assert bench.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]
    # two ranks, 1024 samples each per step, 10 steps in 20 ms -> 1,024,000 samples/s for the job
    assert bench.job_throughput(2, 1024, 10, 20.0) == 1_024_000.0


def test_bench_accounting_helpers():
    import numpy as np

    import bench
    from paper_2508_08540_b200 import workloads as wl

    cfg = wl.CONFIGS[1]
    labels = np.zeros((cfg.N, 1), np.int64)
    labels[:100] = wl.IGNORE_INDEX
    b = bench.score_topk_bytes(cfg, labels)
    assert b == (cfg.N - 100) * (cfg.C * 4 + 4) + cfg.N * 8 + 4 * cfg.N + 8 * cfg.k
    assert bench.aggregate_bytes(cfg) == 4 * cfg.D * (cfg.P + 1)
    assert bench.launches_per_step(wl.CONFIGS[4]) == 1 + 1 + 1 + 1 + 1  # clear, scorer, sequence mean, selector, Eq. 3
    assert bench.launches_per_step(wl.CONFIGS[5]) == 1 + 1 + 1 + 1
    assert bench.launches_per_step(wl.CONFIGS[1]) == 1 + 1 + 1 + 1


_RANK_STUB = """
import json, os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo", rank=rank, world_size=world)
ms = bench.max_over_ranks([3.0 + rank, 9.0 - rank])          # a stand-in for the timed step: each rank reports its own times
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "scaling": "weak", "ms": ms, "value": bench.job_throughput(world, 1024, 10, ms[0])}), flush=True)
dist.destroy_process_group()
"""


def test_spawn_ranks_starts_one_process_per_rank_gloo(capfd):
    """`bench.py --gpus N` started without torchrun becomes the launcher: the ranks it starts find each other
    (gloo here), take the maximum over their timings, and rank 0 alone prints the line."""
    import json

    import bench

    rc = bench.spawn_ranks(2, [sys.executable, "-c", _RANK_STUB % ROOT], timeout_s=240)
    assert rc == 0
    out = [l for l in capfd.readouterr().out.splitlines() if l.startswith("{")]
    assert len(out) == 1
    line = json.loads(out[0])
    assert line["n_gpus"] == 2 and line["scaling"] == "weak" and line["ms"] == [4.0, 9.0]
    assert line["value"] == 2 * 1024 * 10 / 4.0e-3
    # a failing rank is reported
    assert bench.spawn_ranks(2, [sys.executable, "-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"]) == 3
