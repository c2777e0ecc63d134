"""Batch sharding of the seven-nested-loop CNN across GPUs (one process per GPU).

Output elements are independent and b is a free index of Eq. 1, so ranks split the images: each
rank convolves its own ``[Wi][Hi][C][B_r]`` Image slice with the replicated Filter and owns the
``[K][H][W][B_r]`` slice of Out.  The forward has no collective (the paper's parallel sketch,
Section 8, partitions outputs only; splitting b costs nothing but a Filter copy per rank).
Only host-side arithmetic lives here; ``torch.distributed`` is used for barriers and for the
max-over-ranks of timings.
"""
from __future__ import annotations

import numpy as np


def shard_batch(B: int, world: int, rank: int, multiple: int = 32):
    """Contiguous image range [b0, b0+n) of ``rank``.  Shard sizes are multiples of ``multiple``
    (one swizzled shared-memory row of the tensor-core kernel) whenever B allows; the remainder goes
    to the last ranks that still have room.  Every image belongs to exactly one rank."""
    if not (0 <= rank < world) or B <= 0 or multiple <= 0:
        raise ValueError("bad arguments")
    blocks, rem = divmod(B, multiple)
    base, extra = divmod(blocks, world)
    sizes = [(base + (1 if r < extra else 0)) * multiple for r in range(world)]
    sizes[-1] += rem                     # ragged tail (not a multiple): last rank
    b0 = sum(sizes[:rank])
    return b0, sizes[rank]


def slice_batch(array_b_last: np.ndarray, b0: int, n: int) -> np.ndarray:
    """Contiguous copy of images [b0, b0+n) of an array whose last subscript is b."""
    return np.ascontiguousarray(array_b_last[..., b0:b0 + n])


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Max of a per-rank scalar (timings are reported as the slowest rank's)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank: float, seconds_max: float, world: int) -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return world * units_per_rank / seconds_max
