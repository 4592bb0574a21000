"""Host-side helpers for running the scoring path on several GPUs.

Units, matrices and blocks are independent, so the path shards with no exchange of data between
ranks: every rank scores its own contiguous range of decoder blocks.  The only cross-rank
values are scalars on the control path -- the plan's total bits (an int64 sum) and the step time
(a max) -- reduced with torch.distributed on whatever backend the process group uses (NCCL on
GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def block_range(n_blocks: int, rank: int, world: int) -> range:
    """Contiguous, disjoint, exhaustive split of n_blocks global block indices."""
    if not (0 <= rank < world):
        raise ValueError("rank %d of %d" % (rank, world))
    lo = rank * n_blocks // world
    hi = (rank + 1) * n_blocks // world
    return range(lo, hi)


def _device_for_backend():
    return torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")


def sum_int64(value: int) -> int:
    """Sum of an integer over all ranks (exact)."""
    if not (dist.is_available() and dist.is_initialized()):
        return int(value)
    t = torch.tensor([int(value)], dtype=torch.int64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def max_float(value: float) -> float:
    """Maximum of a float over all ranks (the slowest rank's time)."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_device_for_backend())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def average_bits(total_centibits: int, n_weights: int) -> float:
    """b_bar = sum B_i / sum n_i over all ranks (Eq. 6), from per-rank totals."""
    return sum_int64(total_centibits) / (100.0 * sum_int64(n_weights))
