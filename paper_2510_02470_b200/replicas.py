"""Multi-GPU runs are independent replicas (the selection path is one sequential sketch followed by a pass whose
consensus needs every row, so nothing is sharded and there is no data-path collective). The only exchange between
ranks is for reporting: the step time of the whole job is the slowest rank's, and the whole-job throughput counts
the rows of all replicas against it."""
from typing import Optional

import torch


def max_over_ranks(x: float, device: Optional[torch.device] = None) -> float:
    """The largest ``x`` over all ranks of the default process group (``x`` itself without one)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rows_per_s(rows_per_replica: int, world: int, slowest_step_ms: float) -> float:
    """Rows of all ``world`` replicas per second of the slowest replica's step (weak scaling: per-GPU work is fixed)."""
    return world * rows_per_replica / (slowest_step_ms * 1e-3)
