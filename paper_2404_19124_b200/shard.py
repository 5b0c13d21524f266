"""Host-side plumbing for running the draft + verify path on several GPUs.

Sequences are independent (the candidate tree, its pruning and the verification reductions are
all per sequence, Sec. 3.1), so a batch is split into contiguous slices of sequences, one per
rank, with the speculator weights replicated.  No data crosses ranks on the path; only timings
(max over ranks) and, if the caller wants them in one place, the small result tensors do.
"""
from __future__ import annotations

from typing import List, Tuple


def split_sequences(total: int, world: int) -> List[Tuple[int, int]]:
    """(start, count) of every rank's contiguous slice; the first `total % world` ranks get one more."""
    if total < 0 or world < 1:
        raise ValueError("need total >= 0 and world >= 1")
    base, extra = divmod(total, world)
    out, start = [], 0
    for r in range(world):
        cnt = base + (1 if r < extra else 0)
        out.append((start, cnt))
        start += cnt
    return out


def max_over_ranks(x: float, dist=None, device="cpu") -> float:
    """Slowest rank's value (a step is finished when the last rank is)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: int, world: int, seconds_slowest: float) -> float:
    """Units processed by all ranks per second of the slowest rank's time."""
    return units_per_rank * world / seconds_slowest


def gather_rows(local, counts: List[int], dist, dst: int = 0):
    """Concatenates per-rank tensors (different leading sizes) on rank `dst`; returns None elsewhere."""
    import torch
    world = dist.get_world_size()
    rank = dist.get_rank()
    bufs = None
    if rank == dst:
        bufs = [torch.empty((c,) + tuple(local.shape[1:]), dtype=local.dtype) for c in counts]
    # gloo / nccl gather needs equal sizes, so pad to the largest slice
    m = max(counts)
    pad = torch.zeros((m,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    recv = [torch.empty_like(pad) for _ in range(world)] if rank == dst else None
    dist.gather(pad, recv, dst=dst)
    if rank != dst:
        return None
    return torch.cat([recv[r][: counts[r]].cpu() for r in range(world)], dim=0)
