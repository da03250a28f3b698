"""Host-side sharding of an env population over ranks (one process per GPU).

Envs never interact and every random draw is keyed by the global env index, so rank r simply owns
the global range [r * n_per_rank, (r+1) * n_per_rank): no collective touches the data path.  The
only communication is the timing protocol of the bench: a barrier and a max / sum over ranks.
"""
from __future__ import annotations

import os


def env_range(rank: int, world: int, n_per_rank: int):
    """(env_offset, n_envs) of one rank under weak scaling (fixed work per rank)."""
    if not (0 <= rank < world) or n_per_rank < 1:
        raise ValueError("bad rank/world/n_per_rank")
    if world * n_per_rank > 1 << 32:
        raise ValueError("global population exceeds the 32-bit env index of the RNG counter")
    return rank * n_per_rank, n_per_rank


def dist_env():
    """(rank, local_rank, world) from the torchrun environment; (0, 0, 1) when not launched by it."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init_process_group(backend: str):
    """Join the job described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT.  Returns torch.distributed or None."""
    rank, _, world = dist_env()
    if world == 1:
        return None
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if not dist.is_initialized():
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return dist


def reduce_timing(dist, elapsed_ms: float, units: float, device=None):
    """Max of the per-rank time and sum of the per-rank units (what `value` is computed from)."""
    if dist is None:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
