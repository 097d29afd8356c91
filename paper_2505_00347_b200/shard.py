"""Block-aligned partition of a tensor list over workers (host logic only; no arithmetic of the method).

Every quantization block is independent (own scale, own base, random draws addressed by the element
index), so the fused step shards without any exchange inside it: the blocks of all tensors, laid
end to end, are cut into `world` contiguous ranges of (nearly) equal block count, and each worker
steps the pieces that fall into its range with a state of its own.  A piece is described by the
tensor it belongs to, the index of its first element within that tensor (a multiple of the block
size) and its element count; only the last piece of a tensor can end off a block boundary.  What a
worker passes to solo_state_set_origin are the first two.  Whatever parameter exchange follows the
step (an all-gather of the updated pieces) is outside this library.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class Piece:
    tensor: int        # index of the tensor in the full list (its Philox stream)
    elem_offset: int   # first element of the piece within the tensor, a multiple of the block size
    numel: int         # elements of the piece


def partition(sizes, block: int, world: int) -> list[list[Piece]]:
    """Pieces per rank: the flattened block space cut into `world` contiguous ranges whose block
    counts differ by at most one.  Deterministic, so every rank can compute it by itself."""
    if world < 1 or block < 1:
        raise ValueError("world and block must be positive")
    sizes = [int(n) for n in sizes]
    nblk = [-(-n // block) for n in sizes]
    total = sum(nblk)
    base, extra = divmod(total, world)
    out, t, j = [], 0, 0                       # j: next unassigned block of tensor t
    for r in range(world):
        want = base + (1 if r < extra else 0)
        mine = []
        while want > 0:
            take = min(want, nblk[t] - j)
            lo = j * block
            hi = min(sizes[t], (j + take) * block)
            mine.append(Piece(t, lo, hi - lo))
            want -= take
            j += take
            if j == nblk[t]:
                t, j = t + 1, 0
        out.append(mine)
    return out
