"""Multi-GPU plumbing of the benchmark: the path shards by independent sequences, so N ranks
run N replicas with no data-path collective.  The only exchanges are a barrier around the
timed region and the maximum over ranks of the device-measured times; whole-job throughput is
the units all ranks processed divided by that maximum.  Backend-agnostic (NCCL on GPUs, gloo in
the CPU tests)."""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own synthetic sequences."""
    return int(base_seed) + 1000 * int(rank)


def max_over_ranks(values_ms: Sequence[float], device: torch.device) -> list:
    """Element-wise maximum over all ranks of locally measured durations."""
    t = torch.tensor(list(values_ms), device=device, dtype=torch.float64)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_us_per_token(dec_ms_max: float, world: int, batch: int, steps: int) -> float:
    """Latency-type metric of N replicas: the slowest rank's decode time over the tokens all
    ranks decoded in it (weak scaling: per-rank work fixed)."""
    tokens = int(world) * int(batch) * int(steps)
    return dec_ms_max * 1e3 / tokens if tokens else float("nan")


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
