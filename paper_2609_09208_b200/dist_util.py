"""Process-group plumbing for multi-GPU runs (one process per GPU, torch.distributed).

The decode path partitions into independent units (sequence x KV head): ranks share no data, so
there is no collective on the data path.  The only communication is the barrier around the timed
region and the reduction of the timing itself (maximum over ranks) and of the work counters (sum).
"""
from __future__ import annotations

import os


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def init_from_env(backend: str):
    """Initialise the default process group from torchrun's environment; no-op for one process."""
    import torch.distributed as dist
    rank, world, _ = env_rank_world()
    if world == 1 or dist.is_initialized():
        return rank, world
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def _reduce(x: float, op, device):
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device="cpu") -> float:
    import torch.distributed as dist
    return _reduce(x, dist.ReduceOp.SUM, device)


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of `n_units` independent units for `rank` (sizes differ by <= 1)."""
    lo = n_units * rank // world
    hi = n_units * (rank + 1) // world
    return range(lo, hi)


def aggregate_throughput(units_this_rank: float, elapsed_ms_this_rank: float, device="cpu"):
    """Whole-job throughput: all ranks' units divided by the slowest rank's time."""
    total_units = sum_over_ranks(units_this_rank, device)
    worst_ms = max_over_ranks(elapsed_ms_this_rank, device)
    return total_units / (worst_ms * 1e-3), worst_ms
