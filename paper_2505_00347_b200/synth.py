"""Seeded synthetic workloads: tensor-set shapes and parameter / gradient generators.

The paper's real gradients need its datasets and trained weights; these inputs
stand in for them.  Shapes are plain architecture arithmetic, values follow the
distributions listed per workload below.  This module holds none of the
optimizer's arithmetic and imports neither the CUDA library nor the CPU oracle;
both are fed from it.

Everything is generated with ``torch.Generator`` objects seeded from
(workload, tensor index, step), on whatever device is asked for.  CPU and CUDA
generators give different streams for the same seed, so a comparison always
copies the generated tensors to the other side instead of regenerating them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

BLOCK_DEFAULT = 128  # block size used throughout the paper's experiments (Sec. 3.4)


@dataclass(frozen=True)
class Workload:
    """A named tensor set with its optimizer configuration."""

    name: str
    cfg: int                 # workload number, part of every seed
    sizes: tuple[int, ...]   # numel per tensor
    bits_m: int
    bits_v: int
    block: int
    lr: float
    weight_decay: float
    beta1: float
    beta2: float
    steps: int
    grad_kind: str           # "normal", "normal_scaled", "student_t3", "ragged_mix"

    @property
    def numel(self) -> int:
        return sum(self.sizes)


def gpt125m_sizes() -> tuple[int, ...]:
    """GPT-style 125M set: 12 layers, d=768, 4x MLP, vocab 50257, 1024 positions."""
    d, v, ctx, layers = 768, 50257, 1024, 12
    s = [v * d, ctx * d]
    for _ in range(layers):
        s += [d, d, d * 3 * d, 3 * d, d * d, d, d, d, d * 4 * d, 4 * d, 4 * d * d, d]
    s += [d, d]
    return tuple(s)


def llama7b_sizes() -> tuple[int, ...]:
    """LLaMA-7B-shaped set: 32 layers, d=4096, MLP 11008, vocab 32000, RMSNorm vectors."""
    d, f, v, layers = 4096, 11008, 32000, 32
    s = [v * d]
    for _ in range(layers):
        s += [d * d] * 4 + [d * f, d * f, f * d, d, d]
    s += [d, v * d]
    return tuple(s)


RAGGED_FORCED = (1, 2, 63, 64, 65, 127, 128, 129, 2047, 2049)


def ragged_sizes(count: int = 4096, max_numel: int = 4 << 20, seed: int = 4000) -> tuple[int, ...]:
    """`count` sizes drawn LogUniform(1, max_numel), with a few forced edge sizes."""
    rng = np.random.default_rng(seed)
    s = np.rint(np.exp(rng.uniform(0.0, math.log(max_numel), count))).astype(np.int64)
    s = np.clip(s, 1, max_numel)
    s[: len(RAGGED_FORCED)] = RAGGED_FORCED
    return tuple(int(x) for x in s)


def workload(cfg: int, **over) -> Workload:
    """The five benchmark workloads, by number."""
    if cfg == 1:
        w = Workload("single_1Mi", 1, (1 << 20,), 4, 4, 128, 1e-3, 0.01, 0.8, 0.999, 10, "normal")
    elif cfg == 2:
        w = Workload("gpt125m", 2, gpt125m_sizes(), 3, 3, 128, 1e-3, 0.01, 0.6, 0.999, 100,
                     "normal_scaled")
    elif cfg == 3:
        w = Workload("llama7b", 3, llama7b_sizes(), 2, 3, 128, 2e-5, 0.0, 0.5, 0.999, 10,
                     "student_t3")
    elif cfg == 4:
        w = Workload("ragged4096", 4, ragged_sizes(), 2, 3, 128, 1e-3, 0.01, 0.5, 0.999, 3,
                     "ragged_mix")
    elif cfg == 5:
        w = Workload("sweep_268M", 5, (1 << 28,), 4, 4, 128, 1e-3, 0.01, 0.8, 0.999, 3, "normal")
    else:
        raise ValueError(f"unknown workload {cfg}")
    if over:
        w = Workload(**{**w.__dict__, **over})
    return w


def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    seed = 0x9E3779B97F4A7C15
    for k in key:
        seed = (seed * 6364136223846793005 + int(k) + 1442695040888963407) % (1 << 63)
    g.manual_seed(seed)
    return g


def make_param(w: Workload, tensor: int, device="cpu", dtype=torch.float32) -> torch.Tensor:
    """Parameters ~ N(0, 0.02), seed from (workload, tensor)."""
    n = w.sizes[tensor]
    g = _gen(device, 1000 * w.cfg + tensor, 0)
    p = torch.empty(n, device=device, dtype=torch.float32).normal_(0.0, 0.02, generator=g)
    return p.to(dtype)


def tensor_grad_scale(w: Workload, tensor: int) -> float:
    """Per-tensor gradient scale ~ LogUniform(1e-4, 1e-2) for the GPT-style set, else 1."""
    if w.grad_kind != "normal_scaled":
        return 1.0
    rng = np.random.default_rng(1000 * w.cfg + tensor)
    return float(math.exp(rng.uniform(math.log(1e-4), math.log(1e-2))))


def make_grad(w: Workload, tensor: int, step: int, device="cpu") -> torch.Tensor:
    """bf16 gradient of one tensor at one step, seed from (workload, tensor, step)."""
    n = w.sizes[tensor]
    g = _gen(device, 1000 * w.cfg + tensor, step)
    f32 = torch.float32
    if w.grad_kind == "normal":
        x = torch.empty(n, device=device, dtype=f32).normal_(0.0, 1e-3, generator=g)
    elif w.grad_kind == "normal_scaled":
        x = torch.empty(n, device=device, dtype=f32).normal_(0.0, 1e-3, generator=g)
        x *= tensor_grad_scale(w, tensor)
    elif w.grad_kind == "student_t3":
        # t(3) = Z / sqrt(chi2_3 / 3): heavy tails, scaled to 1e-3
        x = torch.empty(n, device=device, dtype=f32).normal_(generator=g)
        chi = torch.zeros(n, device=device, dtype=f32)
        for _ in range(3):
            chi += torch.empty(n, device=device, dtype=f32).normal_(generator=g).square_()
        x *= torch.rsqrt(chi / 3.0).mul_(1e-3)
        del chi
    elif w.grad_kind == "ragged_mix":
        # per 128-element block: exact zeros (30 %), N(0,1e-6) or N(0,1) (35 % each);
        # every 20th tensor additionally has 30 % of its elements set to exactly zero
        nb = (n + 127) // 128
        kind = torch.rand(nb, device=device, generator=g)
        sigma = torch.where(kind < 0.30, 0.0, torch.where(kind < 0.65, 1e-6, 1.0)).to(f32)
        x = torch.empty(nb * 128, device=device, dtype=f32).normal_(generator=g)
        x = (x.view(nb, 128) * sigma[:, None]).reshape(-1)[:n].contiguous()
        if tensor % 20 == 7:
            x[torch.rand(n, device=device, generator=g) < 0.30] = 0.0
    else:
        raise ValueError(w.grad_kind)
    return x.to(torch.bfloat16)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_bf16(a: np.ndarray, device="cpu") -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 tensor."""
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)


def make_state(sizes, bits_m: int, bits_v: int, block: int, seed: int, device="cpu") -> dict:
    """A random packed optimizer state for a tensor list, as torch tensors on `device` in the
    library's layout (tensors one after the other, each starting on a new block).  Code bytes
    are uniform random (every bit pattern is a valid code string; the padding codes of a short
    last block are random too and must be ignored by a reader), scales are log-uniform, bases
    uniform in (0.2, 0.98); about 3 % of the blocks are the zero state."""
    g = _gen(device, seed, 77)
    nb = sum(-(-int(n) // block) for n in sizes)
    out = {}
    zero = torch.rand(nb, device=device, generator=g) < 0.03
    for key, b in (("m", bits_m), ("v", bits_v)):
        slot = block * b // 8
        codes = torch.randint(0, 256, (nb, slot), device=device, dtype=torch.uint8, generator=g)
        codes[zero] = 0
        out["codes_" + key] = codes.reshape(-1)

    def loguniform(lo, hi):
        u = torch.rand(nb, device=device, generator=g)
        return torch.exp(u * (math.log(hi) - math.log(lo)) + math.log(lo)).float()

    out["scale_m"] = loguniform(1e-8, 1e-1).masked_fill_(zero, 0.0)
    out["scale_v"] = loguniform(1e-14, 1e-2).masked_fill_(zero, 0.0)
    out["alpha"] = (torch.rand(nb, device=device, generator=g) * 0.78 + 0.2).float().masked_fill_(zero, 0.5)
    return out
