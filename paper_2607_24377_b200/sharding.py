"""Multi-GPU plumbing for the forward pass.

Attention heads (and, within a head, query rows) are independent in Algorithm 2, so the path
shards with no data-path collective: each rank runs the library on its own heads (or on its own
batch).  The KV axis must not be split across ranks: the quantized tiles depend on the
running-max history.  The only cross-rank operation is the timing reduction of the benchmark.
"""
from __future__ import annotations


def shard_heads(n_heads: int, rank: int, world: int) -> range:
    """Contiguous, balanced slice of the B*H head index space owned by `rank`."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_heads, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms_per_step_local: float, world: int, device=None) -> tuple[float, float]:
    """(whole-job units per second, ms per step) with the step time taken as the max over ranks."""
    ms = max_over_ranks(ms_per_step_local, device)
    return world * units_per_rank / (ms * 1e-3), ms
