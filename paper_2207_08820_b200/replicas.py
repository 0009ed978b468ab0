"""Host logic for running the path on several GPUs of one node: independent replicas, one process per GPU.

Images are independent and the weights are a few hundred kilobytes, so the batch is sharded across ranks and the
data path has no collective.  The only exchanges are for measurement: a barrier around the timed region and a
max-over-ranks of the per-rank device times.  The same code runs with the gloo backend on CPU in the tests.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_range(total: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the units (images, matrix rows) that `rank` owns when `total` units are split as evenly
    as possible over `world` ranks (the first total % world ranks get one more)."""
    if world < 1 or not 0 <= rank < world or total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(seed: int, rank: int) -> int:
    """Seed of the synthetic input of a rank: every replica draws its own batch."""
    return seed + rank


def max_over_ranks(times_ms: Sequence[float], device: torch.device) -> List[float]:
    """Element-wise maximum of per-rank timings (identity when no process group is initialised)."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank: int, world: int, step_ms: float) -> float:
    """Whole-job units per second when every rank processes `units_per_rank` units per step (weak scaling)."""
    return units_per_rank * world / (step_ms * 1e-3)
