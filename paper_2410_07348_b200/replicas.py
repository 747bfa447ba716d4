"""Multi-GPU form of the layer: token-sharded replicas.

Tokens are independent through a MoE++ layer and through a stack of layers, and every zero-computation
expert is replicated on every GPU by design (arXiv 2410.07348, Section 3.4), so N GPUs that each hold all
weights run N independent token batches with no data-path collective.  The only cross-rank traffic is
the timing protocol below: a barrier before and after the timed region and a max over ranks of the
device-side duration.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def token_shard(T: int, rank: int, world: int):
    """Contiguous [begin, end) slice of T tokens owned by `rank`; sizes differ by at most one."""
    base, extra = divmod(T, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def whole_job_rate(units_this_rank: float, ms_this_rank: float, device="cpu"):
    """(units summed over ranks) / (slowest rank's time): returns (units_per_second, max_ms)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_this_rank / (ms_this_rank * 1e-3), ms_this_rank
    t = torch.tensor([ms_this_rank], dtype=torch.float64, device=device)
    u = torch.tensor([units_this_rank], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / (float(t.item()) * 1e-3), float(t.item())
