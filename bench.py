#!/usr/bin/env python
"""Benchmark of the fused SOLO optimizer step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl ours|reference]

With --gpus N > 1 and no launcher in the environment the command starts N ranks itself (one per
GPU, torch.distributed.run on 127.0.0.1); under a launcher it uses the ranks it is given.  Blocks
are independent, so the ranks share nothing on the data path: each steps its own shard (same shapes,
its own random streams) and the job's throughput is all ranks' parameters over the slowest rank's
time (weak scaling).

A step is one pass of the whole hot path (one solo_multi_step launch) over the workload's
tensor set.  Default workload: the LLaMA-7B-shaped set (6.74 B parameters, 2-bit first and 3-bit
second moments, block 128), the configuration the headline metric is quoted on; it fits one
B200 (45 GB).  Prints ONE JSON line on rank 0.

--impl reference times the CPU oracle (a deliberately plain program) on the host cores on a
bounded sample of the same workload; it is a reported baseline, not a target.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2505_00347_b200 import synth  # noqa: E402

METRIC = "fused optimizer-step Gparams/s and achieved HBM GB/s vs 8 TB/s (1 B200)"
UNIT = "Gparams/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per parameter of the step kernel from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum over the parameters of the captured launch, taken on
# the first three tensors of the 7B-shaped set and scaled by the element count; see profiles/).
# Reported for that workload and kernel only (the LLaMA-7B-shaped set, 2-bit / 3-bit, block 128, default
# kernel policy); null for anything else.
NCU_TRAFFIC_BYTES_PER_PARAM = 11.11


def algorithmic_bytes_per_param(bits_m: int, bits_v: int, block: int, param_bytes: int = 4) -> float:
    """What the method must move per parameter: parameter read + write, bf16 gradient, packed
    codes of both moments read + write, three fp32 per block read + write."""
    return 2 * param_bytes + 2 + 2 * (bits_m + bits_v) / 8 + 24 / block


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln)

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # samples taken under load: the upper half of the observed clocks
        sm_sorted = sorted(sm)
        med = float(np.median(sm_sorted[len(sm_sorted) // 2:])) if sm else None
        return {"sm_mhz": med, "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def build_workload(cfg: int, device, args):
    w = synth.workload(cfg)
    over = {}
    if args.max_tensors:
        over["sizes"] = w.sizes[: args.max_tensors]
    if args.bits_m:
        over["bits_m"] = args.bits_m
    if args.bits_v:
        over["bits_v"] = args.bits_v
    if args.block:
        over["block"] = args.block
    if over:
        w = synth.workload(cfg, **over)
    pdtype = torch.bfloat16 if args.param_bf16 else torch.float32
    params = [synth.make_param(w, i, device=device, dtype=pdtype) for i in range(len(w.sizes))]
    grads = [synth.make_grad(w, i, 1, device=device) for i in range(len(w.sizes))]
    return w, params, grads


def run_ours(args, rank, world):
    from paper_2505_00347_b200 import binding as B
    import __graft_entry__ as ge
    if rank == 0:
        ge.build()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    w, params, grads = build_workload(args.workload, device, args)
    B.set_kernel_policy(args.policy)
    state = B.State(list(w.sizes), w.bits_m, w.bits_v, w.block)
    if world > 1:
        # every rank steps its own shard of a job `world` times as large: same shapes, its own random streams
        state.set_origin([rank * len(w.sizes) + t for t in range(len(w.sizes))], None)
    ts = B.TensorSet(params, grads, state)
    h = B.hyper(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=1234,
                fixed_alpha=args.fixed_alpha, v_codebook=args.v_codebook, round_m=args.round_m,
                param_dtype=1 if args.param_bf16 else 0, param_round=1 if args.param_bf16 == 2 else 0)
    n = w.numel
    step_no = 0

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step_no += 1
        B.solo_multi_step(ts, h, step_no)
    sync_all()
    stream = torch.cuda.current_stream()
    clocks = ClockSampler(local)
    if rank == 0:
        clocks.start()
        time.sleep(0.3)
    launches0 = B.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps - 1)]   # between the steps
    e0.record(stream)
    for i in range(args.steps):
        step_no += 1
        B.solo_multi_step(ts, h, step_no)
        if i < args.steps - 1:
            marks[i].record(stream)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)
    edges = [e0] + marks + [e1]
    per_step = sorted(edges[i].elapsed_time(edges[i + 1]) for i in range(args.steps))
    launches = B.launch_count() - launches0
    clk = clocks.stop() if rank == 0 else None
    assert state.status() == 0

    # end to end through the host-buffer entry point: every step the gradients are read from pinned
    # host memory and the updated parameters are written back to it (chunked, three streams)
    pbytes = 2 if args.param_bf16 else 4
    e2e_ms, h2d, d2h, e2e_buffers = None, 2 * n, pbytes * n, None
    if not args.no_e2e:
        # one pinned buffer per tensor when this rank has the host to itself; with several ranks on the
        # host, or when that much page-locked memory is refused, all tensors share one buffer
        distinct = world == 1
        if distinct:
            try:
                hgs = [torch.empty(g.numel(), dtype=torch.bfloat16, pin_memory=True) for g in grads]
                hps = [torch.empty(p.numel(), dtype=p.dtype, pin_memory=True) for p in params]
                e2e_buffers = "one pinned host buffer per tensor"
            except RuntimeError:
                hgs = hps = None
                distinct = False
        if not distinct:
            big = max(w.sizes)
            hg = torch.empty(big, dtype=torch.bfloat16, pin_memory=True)
            hp = torch.empty(big, dtype=params[0].dtype, pin_memory=True)
            hgs = [hg[: g.numel()] for g in grads]
            hps = [hp[: p.numel()] for p in params]
            e2e_buffers = "all tensors share one pinned host buffer (same bytes moved)"
        for hgt, g in zip(hgs, grads):
            hgt.copy_(g)
        sync_all()
        k = max(1, min(args.steps, args.e2e_steps))
        step_no += 1
        B.solo_multi_step_host(params, hgs, hps, state, h, step_no)       # allocates the staging slots
        sync_all()
        e0.record(stream)
        for _ in range(k):
            step_no += 1
            B.solo_multi_step_host(params, hgs, hps, state, h, step_no)
        e1.record(stream)
        sync_all()
        e2e_ms = e0.elapsed_time(e1) / k

    ms, e2e_max = max_over_ranks([ms, e2e_ms or 0.0], device, world)
    if rank != 0:
        return None
    ms_per_step = ms / args.steps
    value = whole_job_gparams(world, n, ms_per_step)
    abytes = algorithmic_bytes_per_param(w.bits_m, w.bits_v, w.block, pbytes)
    achieved = n * abytes / (ms_per_step * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    out = {
        "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4),
        "step_ms": {"median": round(per_step[len(per_step) // 2], 4), "best": round(per_step[0], 4),
                    "worst": round(per_step[-1], 4), "note": "this rank's steps, CUDA events between launches"},
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: {len(w.sizes)} tensors, {n} params, m {w.bits_m}-bit / v {w.bits_v}-bit, "
                               f"block {w.block}, {'bf16' if args.param_bf16 else 'fp32'} params"
                               f"{' (stochastic rounding)' if args.param_bf16 == 2 else ''}, bf16 grads, "
                               "one solo_multi_step call per step"
                               + (f", fixed base {args.fixed_alpha}" if args.fixed_alpha else "")
                               + (f", baseline v codebook {args.v_codebook}" if args.v_codebook else "")
                               + (", first moment rounded stochastically (Eq. 5)" if args.round_m else ""),
                   "l2": "working set (params+grads+state) far larger than the 126 MB L2; no flush needed"
                         if n * abytes > 1e9 else "working set fits L2: launch-bound point, not a bandwidth point",
                   "bytes_per_param": round(abytes, 4),
                   "kernel_launches_per_step": round(launches / args.steps, 2)},
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind} copy bandwidth",
                     "frac_of_nominal_8TBs": round(achieved / NOMINAL_HBM_GBS, 4),
                     "traffic": (round(NCU_TRAFFIC_BYTES_PER_PARAM * n)
                                 if (NCU_TRAFFIC_BYTES_PER_PARAM is not None and args.policy == 0 and
                                     not args.param_bf16 and not args.v_codebook and not args.fixed_alpha and not args.round_m and
                                     w.cfg == 3 and (w.bits_m, w.bits_v, w.block) == (2, 3, 128)) else None)},
        "gpu_launches": int(launches),
        "clocks": clk,
    }
    if e2e_ms is not None:
        out["e2e"] = {"value": round(world * n / (e2e_max * 1e-3) / 1e9, 3), "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "call": "solo_multi_step_host", "buffers": e2e_buffers}
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, args.cpu_sample)
    return out


def max_over_ranks(values, device, world: int) -> list:
    """Element-wise maximum of `values` over all ranks (the slowest rank defines the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_gparams(world: int, params_per_rank: int, ms_per_step: float) -> float:
    """Every rank steps its own replica of the workload (no data-path collective): the job's
    throughput is all ranks' parameters over the slowest rank's time."""
    return world * params_per_rank / (ms_per_step * 1e-3) / 1e9


def cpu_baseline(w, sample_elems: int, steps: int = 1) -> dict:
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    import oracle
    n = min(sample_elems, max(w.sizes))
    sub = synth.workload(w.cfg, sizes=(n,))
    p = synth.make_param(sub, 0).numpy().copy()
    g = synth.bf16_bits(synth.make_grad(sub, 0, 1))
    st = oracle.State(n, w.bits_m, w.bits_v, w.block)
    h = oracle.hyper(lr=w.lr, beta1=w.beta1, beta2=w.beta2, weight_decay=w.weight_decay, seed=1234)
    threads = oracle.hardware_threads()
    oracle.step(p, g, st, h, 1, nthreads=threads)       # warm: page in, first non-zero state
    t0 = time.perf_counter()
    for t in range(steps):
        oracle.step(p, g, st, h, 2 + t, nthreads=threads)
    dt = (time.perf_counter() - t0) / steps
    return {"value": round(n / dt / 1e9, 5), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n} elements of the first tensor's shape, {steps} step(s) from a warm state"}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    w = synth.workload(args.workload)
    vals = []
    base = None
    for _ in range(args.warmup + args.steps):
        base = cpu_baseline(w, args.cpu_sample)
        vals.append(base["value"])
    vals = vals[args.warmup:] or vals
    v = float(np.mean(vals))
    base["value"] = round(v, 5)
    n = min(args.cpu_sample, max(w.sizes))
    return {"impl": "reference", "metric": METRIC, "value": round(v, 5), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(n / v / 1e6, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": f"{w.name}: CPU oracle on a {n}-element sample per step"},
            "cpu_baseline": base,
            "e2e": {"value": round(v, 5), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def spawn_ranks(n: int) -> int:
    """Re-runs this command as `n` ranks on this node, one per GPU, and returns the launcher's exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3)
    ap.add_argument("--max-tensors", type=int, default=0, help="use only the first tensors (small captures)")
    ap.add_argument("--bits-m", type=int, default=0, help="override the workload's first-moment width")
    ap.add_argument("--bits-v", type=int, default=0, help="override the workload's second-moment width")
    ap.add_argument("--block", type=int, default=0, help="override the workload's block size")
    ap.add_argument("--fixed-alpha", type=float, default=0.0,
                    help="fixed base of the logarithmic codebook (no quantile step); 0 = the paper's quantile rule")
    ap.add_argument("--v-codebook", type=int, default=0, choices=[0, 1, 2, 3],
                    help="second-moment quantizer: 0 SOLO (default), 1 unsigned DE, 2 linear, 3 linear without zero")
    ap.add_argument("--round-m", type=int, default=0, choices=[0, 1],
                    help="first moment: 0 nearest level (Eq. 1, default), 1 stochastic rounding (Eq. 5)")
    ap.add_argument("--param-bf16", type=int, default=0, choices=[0, 1, 2],
                    help="bf16 parameters: 1 nearest-even, 2 stochastic rounding (default 0: fp32)")
    ap.add_argument("--cpu-sample", type=int, default=1 << 27)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--policy", type=int, default=0, help="kernel policy: 0 fastest that applies, 1 general, 2 without / 3 always with the sixteen-per-thread kernel")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher yet: start one rank per GPU (this same command under torch.distributed.run)
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if world != max(args.gpus, 1) and rank == 0:
        print(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); reporting {world}",
              file=sys.stderr)
    if args.impl == "reference":
        out = run_reference(args, rank, world)
    else:
        if world > 1:
            import torch.distributed as dist
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl")
        out = run_ours(args, rank, world)
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
