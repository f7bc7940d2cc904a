"""Multi-GPU plumbing: independent replicas, one process per GPU.

The hot path lives on one GPU (all N nodes are buffers of that GPU), so several GPUs run several
independent copies of the workload, each on its own batch, with no data-path collective.  The only
exchange is the timing: the slowest rank's time bounds the job.
"""
from __future__ import annotations

from typing import List

import torch


def rank_node_ids(rank: int, n_nodes: int) -> List[int]:
    """Node indices (they enter the input seeds) of replica `rank`: disjoint between ranks."""
    return [rank * n_nodes + n for n in range(n_nodes)]


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The maximum of `value` over all ranks (the value itself without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(bytes_per_rank: float, ms_per_step_local: float, world: int, dist=None, device="cpu"):
    """(whole-job GB/s, ms per step) with the step time taken as the max over ranks."""
    ms = max_over_ranks(ms_per_step_local, dist, device)
    return world * bytes_per_rank / (ms * 1e-3) / 1e9, ms
