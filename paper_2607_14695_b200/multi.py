"""Host-side logic for running the benchmark on several GPUs of one node.

The hot path shards only by stream and has no exchange step, so N GPUs run N independent replicas of the
batch: no data-path collective. The only communication is the barrier around the timed region and the
max-over-ranks of the device time, from which the whole-job throughput follows."""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replica_throughput(steps_per_rank: int, world: int, slowest_ms: float) -> float:
    """Steps per second of the whole job: every rank did steps_per_rank steps of its own replica in slowest_ms."""
    return world * steps_per_rank / (slowest_ms * 1e-3)
