"""Host-side plumbing for running the path on several GPUs of one node.

The path is independent per token (dense rows and MoE tokens never interact), so it shards by tokens with no
data-path collective: every rank holds a replica of the weights and its own slice of the tokens.  The only
communication is the timing protocol (barrier, max over ranks), which works on any torch.distributed backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_tokens(m_total: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced token shard of `rank`: (first token, number of tokens); shards tile [0, m_total)."""
    base, rem = divmod(m_total, world)
    start = rank * base + min(rank, rem)
    return start, base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar (elapsed time) over the default process group; identity without one."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Aggregate throughput when every rank processed `units_per_rank` within the slowest rank's time."""
    return units_per_rank * world / max_seconds
