"""Multi-process plumbing for running independent replicas of the hot path, one per GPU.

The one-GPU path has no exchange step, so N GPUs run N independent batches ("replicas only"):
no collective touches the data.  What the ranks do share is bookkeeping: a barrier around the
timed region and the maximum over ranks of each measured duration.  Works on any
torch.distributed backend (NCCL on GPUs, gloo on CPU for tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import inputs


def replica_problem(index: int, rank: int):
    """Workload `index` for replica `rank`: rank 0 gets the named configuration, the others the
    same recipe and shape with their own seed."""
    if rank == 0:
        return inputs.config(index)
    seed = inputs.BASE_SEED + index + 100 * rank
    if index == 3:
        return inputs.simclr_batch(4096, 128, "bf16", seed=seed)
    B = {0: 64, 1: 128, 2: 4096, 4: 65536}[index]
    return inputs.dpr_batch(B, 768, "f32" if index == 0 else "bf16", seed=seed)


def max_over_ranks(values, device="cpu") -> list[float]:
    """Element-wise maximum of a list of floats over all ranks (identity without a group)."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_rate(units_per_replica: float, world: int, ms_per_step_max: float) -> float:
    """Aggregate rate of `world` replicas that each process `units_per_replica` per step, timed
    as the slowest rank."""
    return world * units_per_replica / (ms_per_step_max * 1e-3)
