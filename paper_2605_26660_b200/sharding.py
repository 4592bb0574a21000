"""Host-side helpers for running the scoring path on several GPUs.

Units, matrices and blocks are independent, so the path shards with no exchange of data between
ranks: every rank scores its own contiguous range of decoder blocks.  The only cross-rank
values are scalars on the control path -- the plan's total bits (an int64 sum) and the step time
(a max) -- reduced with torch.distributed on whatever backend the process group uses (NCCL on
GPUs, gloo in the CPU tests).  The one call that looks at all units at once is the heuristic
allocator's rule: for it the ranks exchange their units' scores and counts (a few bytes per unit,
`gather_units`), every rank runs the rule on the same gathered arrays and keeps its own slice.
A calibration input can also be split by tokens: `combine_act_stats` merges the per-rank statistics.
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


def gather_units(*arrays: torch.Tensor):
    """All-gathers per-unit 1-D tensors of the same length (scores, weight counts, ...) in rank order.

    Ranks may hold different numbers of units.  Returns (gathered tensors, begin, end): every rank gets the
    same concatenation, and [begin, end) is where this rank's units sit in it.  Without a process group the
    inputs come back unchanged."""
    n = int(arrays[0].numel())
    for a in arrays:
        if a.dim() != 1 or a.numel() != n:
            raise ValueError("gather_units wants 1-D tensors of one length")
    if not (dist.is_available() and dist.is_initialized()):
        return list(arrays), 0, n
    world, rank = dist.get_world_size(), dist.get_rank()
    counts = torch.zeros(world, dtype=torch.int64, device=arrays[0].device)
    counts[rank] = n
    dist.all_reduce(counts, op=dist.ReduceOp.SUM)
    counts = [int(c) for c in counts.tolist()]
    width = max(counts)
    out = []
    for a in arrays:
        padded = torch.zeros(width, dtype=a.dtype, device=a.device)
        padded[:n] = a
        parts = [torch.empty_like(padded) for _ in range(world)]
        dist.all_gather(parts, padded)
        out.append(torch.cat([p[:c] for p, c in zip(parts, counts)]))
    begin = sum(counts[:rank])
    return out, begin, begin + n


def gather_rows(table: torch.Tensor) -> torch.Tensor:
    """All-gathers a per-unit table [n, k] (e.g. the error table err[u][6] of this rank's units) by rows, in rank
    order; every rank gets the table of the whole model.  Ranks may hold different numbers of units."""
    if table.dim() != 2:
        raise ValueError("gather_rows wants a 2-D tensor")
    cols, _, _ = gather_units(*[table[:, j].contiguous() for j in range(table.shape[1])])
    return torch.stack(cols, dim=1)


def allocate_across_ranks(allocate, saliency, n_weights, n_groups, n_protected=None):
    """The heuristic allocator's rule over the units of all ranks.  `allocate(saliency, n_weights, n_groups,
    n_protected)` is the rule on whole-model arrays (e.g. a closure over windq_greedy_allocate with the
    target and headroom) and returns a dict with `actions` and `total_centibits`; every rank calls it on the
    same gathered arrays, so all ranks hold the same plan.  Returns (this rank's actions, total centibits of
    the model)."""
    has_p = n_protected is not None
    arrays = [saliency, n_weights, n_groups] + ([n_protected] if has_p else [])
    gathered, begin, end = gather_units(*arrays)
    res = allocate(gathered[0], gathered[1], gathered[2], gathered[3] if has_p else None)
    return res["actions"][begin:end], int(res["total_centibits"])


def combine_act_stats(s_local: torch.Tensor, tokens_local: int) -> torch.Tensor:
    """Activation statistics of a calibration input whose tokens are split over the ranks.

    Every rank calls windq_act_stats on its own slice of tokens (s_local[j] = mean of x_tj^2 over its
    tokens_local tokens); the statistic of the whole input is the token-weighted mean of the slices,
    s[j] = sum_r tokens_r * s_r[j] / sum_r tokens_r, formed in float64 and all-reduced (one sum of C + 1
    numbers).  Returns fp32 [C] on every rank.  Without a process group the input comes back unchanged."""
    if not (dist.is_available() and dist.is_initialized()):
        return s_local
    acc = torch.empty(s_local.numel() + 1, dtype=torch.float64, device=s_local.device)
    acc[:-1] = s_local.to(torch.float64) * float(tokens_local)
    acc[-1] = float(tokens_local)
    dist.all_reduce(acc, op=dist.ReduceOp.SUM)
    return (acc[:-1] / acc[-1]).to(torch.float32)
