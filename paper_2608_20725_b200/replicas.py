"""Host-side helpers for running the layer on several GPUs of one node.

Output image n depends on input image n only (paper Eq. 1), so the batch splits
across ranks with no exchange: every rank holds the filter and a contiguous slab
of the batch; there is no data-path collective.  The only communication is the
max-over-ranks of the measured device time.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def batch_slice(n_images: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous slab [begin, end) of the batch owned by `rank`; sizes differ by at most one."""
    if not (0 <= rank < world) or n_images < 0:
        raise ValueError("bad rank/world/batch")
    base, extra = divmod(n_images, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values: Sequence[float], device="cpu") -> List[float]:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Aggregate rate (units per second) of `world` ranks that each processed `units_per_rank`
    units in at most `ms_max` milliseconds (weak scaling)."""
    return world * units_per_rank / (ms_max * 1e-3)
