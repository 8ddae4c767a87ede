"""Sharding of independent videos over ranks (one process per GPU).

The merging path has no exchange step between videos: a rank merges its own videos and only
the row counts travel (one all-gather) so that every rank knows where its rows start in the
global packed output.  No feature data crosses ranks.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def videos_of_rank(n_videos: int, world: int, rank: int) -> range:
    """Contiguous block of video indices of a rank (sizes differ by at most one)."""
    base, extra = divmod(n_videos, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def global_row_offsets(local_counts: Sequence[int], n_videos: int) -> Tuple[List[int], int]:
    """All-gathers the per-video row counts and returns (first global row of each of THIS rank's
    videos, total rows).  Works on any backend; the tensors live on the CPU for gloo and on the
    current CUDA device for nccl."""
    world, rank = dist.get_world_size(), dist.get_rank()
    device = "cuda" if dist.get_backend() == "nccl" else "cpu"
    longest = -(-n_videos // world)
    mine = torch.zeros(longest, dtype=torch.int64, device=device)
    mine[:len(local_counts)] = torch.tensor(list(local_counts), dtype=torch.int64, device=device)
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    counts = []
    for r in range(world):
        counts.extend(gathered[r][:len(videos_of_rank(n_videos, world, r))].tolist())
    offsets = [0]
    for c in counts:
        offsets.append(offsets[-1] + int(c))
    own = videos_of_rank(n_videos, world, rank)
    return [offsets[v] for v in own], offsets[-1]
