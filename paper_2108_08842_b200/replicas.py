"""Multi-process plumbing for running independent replicas of the hot path, one process
per GPU.  EDEN's senders are independent and the receiver's only cross-client step is a
sum, so the single-GPU library scales out as replicas: every rank works on its own
clients and nothing crosses ranks on the data path.  Only timings are reduced."""
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
