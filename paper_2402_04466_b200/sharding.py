"""Stream-to-rank sharding for multi-GPU runs (host logic only).

Streams are independent problems (own frames, own recurrent state, shared read-only weights),
so they are dealt round-robin to the ranks and never exchange data on the GPU; the only
cross-rank traffic is the host-side gather of the small per-frame result records and the
max-over-ranks reduction of step times.
"""
from __future__ import annotations

from typing import Dict, List, Sequence


def assign_streams(n_streams: int, world_size: int) -> List[List[int]]:
    """streams[r] = global stream ids handled by rank r (stream s lives on rank s mod world_size)."""
    if n_streams < 0 or world_size < 1:
        raise ValueError("n_streams >= 0 and world_size >= 1 required")
    return [[s for s in range(n_streams) if s % world_size == r] for r in range(world_size)]


def owner_of(stream: int, world_size: int) -> int:
    return stream % world_size


def gather_results(local: Dict[int, dict], world_size: int, group=None) -> Dict[int, dict]:
    """All ranks receive {global stream id: result record} for every stream of the tick."""
    if world_size == 1:
        return dict(local)
    import torch.distributed as dist
    parts: List[Dict[int, dict]] = [None] * world_size  # type: ignore[list-item]
    dist.all_gather_object(parts, local, group=group)
    merged: Dict[int, dict] = {}
    for rank, part in enumerate(parts):
        for sid, rec in part.items():
            if owner_of(sid, world_size) != rank:
                raise RuntimeError(f"rank {rank} reported stream {sid} that it does not own")
            if sid in merged:
                raise RuntimeError(f"stream {sid} reported twice")
            merged[sid] = rec
    return merged


def max_over_ranks(values: Sequence[float], world_size: int, device=None, group=None) -> List[float]:
    """Element-wise maximum over ranks of a short list of timings."""
    if world_size == 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return [float(v) for v in t.cpu()]
