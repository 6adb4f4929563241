"""Batch sharding for multi-GPU runs of the carve path.

Images are independent (no step of Sec. 3.3 reads another image), so N ranks simply carve
disjoint sets of images: no collective is on the data path.  The only communication a run
needs is a barrier and a max-reduction of the measured time.
"""
from __future__ import annotations

from typing import List, Tuple


def image_range(rank: int, world: int, images_per_rank: int) -> range:
    """Weak scaling: rank r owns images [r * B, (r + 1) * B)."""
    if not (0 <= rank < world) or images_per_rank < 1:
        raise ValueError("bad rank / world / images_per_rank")
    return range(rank * images_per_rank, (rank + 1) * images_per_rank)


def split_batch(total_images: int, world: int) -> List[Tuple[int, int]]:
    """Strong scaling: contiguous [begin, end) per rank, sizes differing by at most one."""
    if total_images < 0 or world < 1:
        raise ValueError("bad total_images / world")
    base, extra = divmod(total_images, world)
    out, begin = [], 0
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append((begin, begin + n))
        begin += n
    return out


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks of the default process group (the value itself when
    torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
