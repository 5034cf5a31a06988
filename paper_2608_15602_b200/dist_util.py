"""Host-side helpers for the multi-process benchmark: the path has no exchange step, so N ranks run
N independent replicas and only the timing is combined (max over ranks) -- no collective on the data
path.  Works with any torch.distributed backend (nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replica_throughput(bytes_per_step_per_rank: int, ms_per_step_max: float, world: int) -> float:
    """Whole-job GB/s of `world` replicas that each move bytes_per_step_per_rank per step, the step
    time being the slowest rank's."""
    return world * bytes_per_step_per_rank / (ms_per_step_max * 1e-3) / 1e9
