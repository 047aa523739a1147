"""Host-side logic of the multi-GPU run: (batch, head) units are independent, so every rank runs its own
replica of the workload and the only communication is the reduction of the ranks' timings."""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import inputs


def replica_workload(w: inputs.Workload, rank: int) -> inputs.Workload:
    """The workload instance of `rank`: same shapes, its own seed (independent data per replica)."""
    return inputs.with_seed(w, w.seed + 1000 * rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank's time counts)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def aggregate_value(flops_per_rank: float, world: int, step_ms: float) -> float:
    """Whole-job TFLOP/s: all ranks' FLOPs divided by the slowest rank's step time."""
    return world * flops_per_rank / (step_ms * 1e-3) / 1e12
