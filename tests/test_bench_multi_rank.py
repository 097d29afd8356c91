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


def _agree_main(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2505_00347_b200 import shard, synth
    sizes = synth.gpt125m_sizes()
    parts = shard.partition(sizes, 128, world)               # every rank computes the whole partition by itself
    mine = parts[rank]
    # what a rank would pass to the library: piece sizes, stream ids, element offsets
    desc = torch.tensor([[p.tensor, p.elem_offset, p.numel] for p in mine], dtype=torch.int64)
    blocks = torch.tensor([sum(-(-p.numel // 128) for p in mine)], dtype=torch.int64)
    gathered = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(gathered, blocks)
    # the ranks exchange a digest of the full partition: they must have computed the same one
    digest = torch.tensor([hash(tuple((p.tensor, p.elem_offset, p.numel) for r in parts for p in r)) % (1 << 62)])
    digests = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(digests, digest)
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{int(blocks)} {[int(x) for x in gathered]} {len(set(int(x) for x in digests))} "
                f"{int(desc[:, 2].sum())} {int((desc[:, 1] % 128).abs().sum())}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_partition(tmp_path):
    """The block-aligned partition of the GPT-style set: each rank computes it alone, the ranks agree on
    it, their block counts differ by at most one and add up, offsets sit on block boundaries."""
    from paper_2505_00347_b200 import synth
    world, port = 2, _free_port()
    mp.spawn(_agree_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    total_blocks = sum(-(-n // 128) for n in synth.gpt125m_sizes())
    import ast
    import re
    elems = 0
    rows = [open(tmp_path / f"rank{r}.txt").read() for r in range(world)]
    for r, row in enumerate(rows):
        m = re.match(r"(\d+) (\[.*?\]) (\d+) (\d+) (\d+)$", row)
        blocks, gathered, ndigests, numel, misaligned = int(m[1]), ast.literal_eval(m[2]), int(m[3]), int(m[4]), int(m[5])
        assert gathered[r] == blocks and sum(gathered) == total_blocks and max(gathered) - min(gathered) <= 1
        assert ndigests == 1 and misaligned == 0
        elems += numel
    assert elems == sum(synth.gpt125m_sizes())


def test_gpus_flag_starts_the_ranks_itself(tmp_path):
    """`bench.py --gpus 2` with no launcher in the environment re-runs itself as two ranks.  The CPU
    arm needs no GPU: rank 0 alone times the oracle and prints the one JSON line, the other rank
    exits 0 without work."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "1", "--cpu-sample", "65536"],
                       capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["value"] > 0


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], torch.device("cpu"), 1) == [3.0, 4.0]
    assert bench.whole_job_gparams(1, 2_000_000_000, 10.0) == pytest.approx(200.0)
