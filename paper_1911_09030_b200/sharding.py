"""Host-side partitioning of a job over ranks (one process per GPU).

Algorithm 3 (Local AdaAlter) is coordinate-wise, and the synthetic gradient noise is keyed on
the GLOBAL coordinate index, so a job can be cut by coordinate range with no data-path
communication at all: rank r creates its context with `j_base = start(r)` and the results are
bit-identical to the single-process job.  The only collectives a multi-rank run needs are the
barrier and the max-over-ranks reduction of the timings.
"""
from __future__ import annotations

from typing import List, Tuple

ALIGN = 4  # la_config.j_base must be a multiple of 4 (coordinate pairs, 16-byte rows)


def coordinate_shard(N: int, rank: int, world: int, align: int = ALIGN) -> Tuple[int, int]:
    """[start, stop) of rank's coordinates when N coordinates are cut into `world` contiguous
    ranges whose starts are multiples of `align` (strong scaling: total work fixed)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = (N + align - 1) // align
    lo = (units * rank) // world * align
    hi = (units * (rank + 1)) // world * align
    return min(lo, N), min(hi, N)


def all_shards(N: int, world: int, align: int = ALIGN) -> List[Tuple[int, int]]:
    return [coordinate_shard(N, r, world, align) for r in range(world)]


def weak_scaling_base(N: int, rank: int, align: int = ALIGN) -> int:
    """Global index of rank's first coordinate when every rank runs a full copy of an
    N-coordinate configuration on its own, disjoint coordinate range (weak scaling)."""
    return rank * ((N + align - 1) // align * align)


def max_over_ranks(value: float, dist=None) -> float:
    """Max of a per-rank scalar (e.g. a device-timed duration); identity without a process group."""
    if dist is None or not dist.is_available() or not dist.is_initialized():
        return float(value)
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])
