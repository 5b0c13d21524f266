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


# ---- vocabulary-parallel heads ---------------------------------------------------------------
# For small batches a draft is the time to read the vocabulary-sized head matrices once per level
# (Sec. 3.1: that is where the speculator's parameters are).  Splitting those rows over the GPUs of
# one node divides that time; what has to cross the links per level is each rank's top-k list and one
# log-sum-exp per tree node, a few kilobytes.

def split_vocab(V: int, world: int, multiple: int = 8) -> List[Tuple[int, int]]:
    """(first row, rows) of every rank's slice of the vocabulary: contiguous, disjoint, covering [0, V);
    all but the last slice are a multiple of `multiple` rows (whole 16-byte groups of bf16 rows are not
    required, but equal tile shapes on every rank are convenient)."""
    if V < world or world < 1:
        raise ValueError("need V >= world >= 1")
    per = -(-V // world)
    per = -(-per // multiple) * multiple
    out, start = [], 0
    for r in range(world):
        cnt = max(0, min(per, V - start))
        if cnt == 0:
            raise ValueError(f"vocabulary of {V} rows leaves rank {r} of {world} without rows")
        out.append((start, cnt))
        start += cnt
    return out


_send_buffers = {}   # (device, bytes) -> uint8 tensor: the copy of this rank's slot that is sent, kept between calls


def all_gather_slots(region, rank: int, dist, group=None) -> None:
    """`region`: uint8 tensor [world, slot_bytes] of which row `rank` is filled; afterwards every row is.
    Any backend (NCCL on the GPU the region lives on, gloo for CPU tensors).  The slot that is sent is copied
    into a buffer that is allocated once per (device, size) and reused, so a draft allocates nothing per level."""
    import torch
    world, nbytes = region.shape[0], region.shape[1]
    key = (str(region.device), int(nbytes))
    mine = _send_buffers.get(key)
    if mine is None:
        mine = torch.empty(nbytes, dtype=torch.uint8, device=region.device)
        _send_buffers[key] = mine
    mine.copy_(region[rank])
    dist.all_gather([region[g] for g in range(world)], mine, group=group)


def draft_vocab_parallel(binding, h, ctx_state, last_tok, topk, K, workspace=None, cand_tok=None, cand_logp=None,
                         exchange=None, stream=None):
    """One draft on a handle that holds a vocabulary shard (binding.spec_create(..., vocab_shard=...)).
    `exchange(level, region)` must fill the other ranks' rows of `region` ([n_ranks, slot_bytes] uint8 view
    of the workspace); the default all-gathers over torch.distributed's default group.  Every rank
    returns the same (cand_tok, cand_logp, workspace)."""
    import torch
    B = ctx_state.shape[0]
    n = h.n_heads
    if workspace is None:
        workspace = torch.empty(binding.spec_draft_workspace_bytes(h, B, topk, K), dtype=torch.uint8, device=h.device)
    if cand_tok is None:
        cand_tok = torch.empty((B, K, n), dtype=torch.int32, device=h.device)
    if cand_logp is None:
        cand_logp = torch.empty((B, K), dtype=torch.float32, device=h.device)
    if exchange is None:
        import torch.distributed as dist

        def exchange(level, region):
            all_gather_slots(region, h.vp_rank, dist)
    for level in range(n):
        binding.spec_draft_vp_local(h, level, ctx_state, last_tok, topk, K, workspace, stream=stream)
        off, slot = binding.spec_draft_vp_exchange(h, B, topk, K, level)
        exchange(level, workspace[off: off + slot * h.vp_ranks].view(h.vp_ranks, slot))
        last = level == n - 1
        binding.spec_draft_vp_merge(h, level, B, topk, K, workspace, cand_tok if last else None,
                                    cand_logp if last else None, stream=stream)
    return cand_tok, cand_logp, workspace
