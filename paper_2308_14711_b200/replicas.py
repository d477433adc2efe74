"""Host-side logic of running N independent replicas of the layer (one process per GPU).

Tokens are independent and the parameters are replicated, so there is no collective on the data path:
each rank runs the same workload on its own tokens.  The only communication is for timing: a barrier
before and after the timed region and the maximum of the ranks' elapsed times.
"""
from __future__ import annotations

from typing import Optional


def max_over_ranks(value: float, dist=None, device: Optional[str] = None) -> float:
    """Maximum of `value` over all ranks of the default process group (identity without a group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(tokens_per_step_per_rank: int, steps: int, world_size: int, elapsed_ms_max: float) -> float:
    """Tokens per second of the whole job: every rank processed steps * tokens in at most elapsed_ms_max."""
    return world_size * tokens_per_step_per_rank * steps / (elapsed_ms_max * 1e-3)


def token_shard(total_tokens: int, rank: int, world_size: int):
    """[begin, end) of the tokens rank `rank` takes when one batch is split evenly over the ranks."""
    base, rem = divmod(total_tokens, world_size)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
