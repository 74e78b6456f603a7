"""Token-row sharding across ranks.

Every step of the layer is row-local (the rotation, the per-token scales, the GEMM rows), so a batch
of M tokens is split by rows, the prepared layer is replicated, and no collective touches the data
path.  The only communication is the max-over-ranks of the measured time."""
from __future__ import annotations

import torch
import torch.distributed as dist


def row_shard(M: int, rank: int, world: int) -> tuple[int, int]:
    """Half-open row range [lo, hi) of `rank`; shards differ by at most one row and cover [0, M)."""
    if not (0 <= rank < world) or M < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(M, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """MAX all-reduce of a scalar (the timing rule for multi-GPU numbers)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, ms: float, world: int) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` in `ms` (already the max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)
