"""Replica bookkeeping for multi-GPU runs.

The layer runs on one GPU with every expert resident; several GPUs run independent replicas on their own
batches ("weak" scaling). Nothing crosses GPUs on the data path: the only exchange is the timing summary
below (a max-reduction over ranks), so it is the whole multi-process surface of the benchmark.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity for a single process)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(tokens_per_replica: int, steps: int, total_ms_max: float, world: int) -> float:
    """Whole-job tokens/s: every replica processes its own batch each step; the slowest rank sets the time."""
    return world * tokens_per_replica * steps / (total_ms_max / 1e3)
