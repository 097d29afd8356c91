"""The multi-rank part of bench.py on CPU: two gloo ranks, the job's time is the slowest rank's,
the job's throughput counts every rank's parameters (weak scaling, no data-path collective)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r measured (10 + 5 r) ms for the device-only loop and (100 - 7 r) ms end to end
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - 7.0 * rank], torch.device("cpu"), world)
    value = bench.whole_job_gparams(world, 1_000_000_000, ms / 5)       # 5 steps
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{ms} {e2e} {value}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        ms, e2e, value = (float(x) for x in open(tmp_path / f"rank{r}.txt").read().split())
        assert ms == 15.0 and e2e == 100.0                  # maxima over the ranks, on every rank
        assert value == pytest.approx(2 * 1e9 / 3e-3 / 1e9)   # 2 ranks x 1e9 params per 3 ms step


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], torch.device("cpu"), 1) == [3.0, 4.0]
    assert bench.whole_job_gparams(1, 2_000_000_000, 10.0) == pytest.approx(200.0)
