"""Multi-process plumbing, one process per GPU.  EDEN's senders are independent and the
receiver's only cross-client step is a sum, so the single-GPU library scales out in two
ways: as independent replicas (every rank has its own round of clients; only timings are
reduced), or with one round's senders split over the ranks, each rank decoding its share
into a partial mean (eden_mean_partial) and one sum all-reduce of d floats finishing the
mean of Section 2.2.2 on every rank."""
from __future__ import annotations

import os
from typing import List, Sequence

import torch
import torch.distributed as dist


def rank_info():
    """(rank, world size, local rank) from the torchrun environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(values: Sequence[float], device="cpu") -> List[float]:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_gbs(world: int, bytes_per_rank: int, ms_per_step: float) -> float:
    """Aggregate GB/s of `world` replicas that each move bytes_per_rank per step, the step
    time being the slowest rank's."""
    return world * bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def shard_clients(n_total: int, rank: int, world: int) -> range:
    """The contiguous block of client indices rank `rank` of `world` handles: sizes differ
    by at most one, earlier ranks take the larger blocks."""
    base, extra = divmod(n_total, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def sum_partial_means(partial: torch.Tensor, group=None) -> torch.Tensor:
    """In-place sum all-reduce of this rank's partial mean over the ranks (identity without
    a process group): afterwards every rank holds the mean over all senders."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(partial, op=dist.ReduceOp.SUM, group=group)
    return partial


def sharded_mean(ctx, codes, scales, bits, seeds, d: int, n_total: int, recv_masks=None, out=None, group=None):
    """Receiver with the round's n_total senders split over the ranks: `codes`, `scales`,
    `bits`, `seeds`, `recv_masks` are this rank's share (see shard_clients).  Returns the
    mean over all senders (on every rank)."""
    partial = ctx.mean_partial(codes, scales, bits, seeds, d, n_total, recv_masks, out)
    return sum_partial_means(partial, group)
