"""Multi-GPU plumbing: the forward pass shards by (batch, KV head) with no exchange on the data path, so the
only distributed pieces are the split of independent units over ranks and the reduction of the timing."""
from __future__ import annotations

import torch

__all__ = ["shard_range", "combine_timing"]


def shard_range(n_units: int, world: int, rank: int) -> range:
    """Contiguous, balanced share of `n_units` independent units for `rank` of `world` (sizes differ by <= 1)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def combine_timing(ms_local: float, units_local: float, device="cpu"):
    """(max over ranks of the per-step time, sum over ranks of the units processed).

    Uses the default process group when one is initialised (NCCL on GPUs, gloo in the CPU tests); with a
    single process it returns its inputs."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
