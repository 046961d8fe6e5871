"""Multi-GPU plumbing: environments are independent (paper Section 3.2), so ranks take disjoint
contiguous ranges of seeded environment ids and exchange nothing on the data path.  The only
communication is a barrier and the max-over-ranks of the timings."""
from __future__ import annotations

import torch
import torch.distributed as dist


def env_offset(rank: int, envs_per_rank: int) -> int:
    """First seeded environment id of `rank` (weak scaling: every rank renders envs_per_rank)."""
    return rank * envs_per_rank


def split_envs(total_envs: int, rank: int, world: int):
    """Contiguous [begin, end) range of `rank` when a fixed batch is divided (strong scaling)."""
    base, rem = divmod(total_envs, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def max_over_ranks(values, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]
