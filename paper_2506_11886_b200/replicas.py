"""Multi-GPU plumbing of the benchmark: the decode path does not shard (one GPU holds one
replica of the per-layer cache and runs the whole step), so N GPUs run N independent replicas.
The only cross-rank traffic is the timing protocol: a barrier on both sides of the timed region
and the maximum of the per-rank device times.  Works with any torch.distributed backend
(nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> tuple[int, int]:
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier() -> None:
    if world()[1] > 1:
        dist.barrier()


def max_over_ranks(value_ms: float, device="cpu") -> float:
    """Slowest rank's time: the time of the whole job."""
    if world()[1] == 1:
        return float(value_ms)
    t = torch.tensor([float(value_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_us_per_step(ms_total_max: float, steps: int, n_replicas: int) -> float:
    """Whole-job microseconds per decode step: N replicas finish N steps in the time of one."""
    return ms_total_max * 1e3 / steps / n_replicas
