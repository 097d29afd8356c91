"""The synthetic workload generators: shapes, determinism, and the packing helper against
the oracle's bit-level accessors."""
import numpy as np
import torch

import oracle
import parity
from paper_2505_00347_b200 import synth


def test_tensor_set_shapes():
    g = synth.gpt125m_sizes()
    assert len(g) == 148 and sum(g) == 124_439_808
    l = synth.llama7b_sizes()
    assert len(l) == 291 and sum(l) == 6_738_415_616
    r = synth.ragged_sizes()
    assert len(r) == 4096 and r[:10] == synth.RAGGED_FORCED and max(r) <= 4 << 20 and min(r) == 1
    assert synth.ragged_sizes() == r
    for cfg in range(1, 6):
        w = synth.workload(cfg)
        assert w.cfg == cfg and w.block == 128


def test_generators_are_seeded():
    w = synth.workload(2, sizes=(1000, 300))
    a, b = synth.make_grad(w, 1, 3), synth.make_grad(w, 1, 3)
    assert torch.equal(a, b) and a.dtype == torch.bfloat16
    assert not torch.equal(a, synth.make_grad(w, 1, 4))
    assert torch.equal(synth.make_param(w, 0), synth.make_param(w, 0))
    assert 1e-4 <= synth.tensor_grad_scale(w, 0) <= 1e-2
    w4 = synth.workload(4, sizes=(128 * 200,))
    g = synth.make_grad(w4, 0, 1).float().view(200, 128)
    zero_blocks = (g == 0).all(1).float().mean()
    assert 0.15 < zero_blocks < 0.45
    w3 = synth.workload(3, sizes=(200_000,))
    t = synth.make_grad(w3, 0, 1).float()
    assert t.abs().max() > 8 * t.std() * 0.5 and abs(t.mean()) < 1e-4   # heavy tails
    bits = synth.bf16_bits(a)
    assert torch.equal(synth.bits_to_bf16(bits), a)


def test_pack_helper_matches_oracle_layout():
    for b in (2, 3, 4, 8):
        for block in (64, 128):
            rng = np.random.default_rng(b + block)
            codes = rng.integers(0, 1 << b, size=(3, block), dtype=np.uint8)
            packed = parity.pack_codes(codes, b)
            slot = block * b // 8
            for j in range(3):
                for e in range(block):
                    assert oracle.get_code(packed[j * slot:], e, b) == codes[j, e]
            assert np.array_equal(parity.unpack_codes(packed, b, block), codes)
    st = synth.make_state((130, 64, 1), 2, 3, 64, seed=1)
    assert st["codes_m"].numel() == (3 + 1 + 1) * 16 and st["codes_v"].numel() == 5 * 24
    assert st["alpha"].numel() == 5 and st["codes_m"].dtype == torch.uint8
    assert torch.all((st["alpha"] > 0) & (st["alpha"] < 1)) and torch.all(st["scale_v"] >= 0)
    again = synth.make_state((130, 64, 1), 2, 3, 64, seed=1)
    assert all(torch.equal(st[k], again[k]) for k in st)


def test_partition_is_block_aligned_and_complete():
    from paper_2505_00347_b200 import shard
    sizes = (1, 129, 2048 * 3 + 5, 64, 128 * 7, 2047, 300)
    for block in (64, 128, 2048):
        nblk = [-(-n // block) for n in sizes]
        for world in (1, 2, 3, 5, 8, 64):
            parts = shard.partition(sizes, block, world)
            assert len(parts) == world
            counts = [sum(-(-p.numel // block) for p in r) for r in parts]
            assert sum(counts) == sum(nblk) and max(counts) - min(counts) <= 1
            seen = {t: [] for t in range(len(sizes))}
            for r in parts:
                for p in r:
                    assert p.elem_offset % block == 0 and p.numel > 0
                    seen[p.tensor].append((p.elem_offset, p.numel))
            for t, n in enumerate(sizes):      # the pieces of a tensor tile it exactly, in order
                pos = 0
                for off, m in seen[t]:
                    assert off == pos and (m % block == 0 or off + m == n)
                    pos += m
                assert pos == n
