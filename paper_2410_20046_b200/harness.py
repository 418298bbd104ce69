"""Host-side helpers of the multi-process benchmark: which synthetic batch a rank takes and
how per-rank timings are merged.  No device code and no arithmetic of the method."""
from __future__ import annotations


def batch_id(b: int, rank: int, world: int, n_batches: int) -> int:
    """Seed index of pre-staged batch `b` on `rank`: ranks take disjoint batches, so the
    job as a whole processes `world` times the samples of one replica per step."""
    assert 0 <= rank < world and 0 <= b < n_batches
    return rank * n_batches + b


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of one float over the default process group (identity when
    torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_step: float, world: int, steps: int, max_ms: float) -> float:
    """Whole-job units per second: every rank's units over the slowest rank's time."""
    return units_per_rank_step * world * steps / (max_ms * 1e-3)
