"""One long video over several GPUs, cut into segments of consecutive frames (Section 3.3: the
temporal chains run over frames, so they may cross a cut).

Every rank holds its own frames with the last frame of the rank before it in front (the halo).
It merges halo + segment with the ordinary kernels, then the ranks are finished from the last
to the first: a rank takes in what the next rank merged into the nodes of its last frame, hands
what it merged into its halo's nodes to the rank before, and writes the rows it owns.  Per cut,
one message of at most H*W rows of D floats travels.  The arithmetic runs in the library's
kernels; this module only allocates, calls and moves messages.
"""
from dataclasses import dataclass
from typing import List, Optional

import torch

from . import binding


class LocalLink:
    """Ranks emulated one after the other in one process (last rank first): a mailbox."""

    def __init__(self, world: int):
        self.world = world
        self.box = {}
        self.counts = [0] * world

    def for_rank(self, rank: int) -> "LocalLink":
        return _RankView(self, rank)


class _RankView:
    def __init__(self, shared: LocalLink, rank: int):
        self.shared, self.rank, self.world = shared, rank, shared.world

    def send_prev(self, tensors: List[torch.Tensor]) -> None:
        self.shared.box[self.rank - 1] = [t.clone() for t in tensors]

    def recv_next(self, like: List[torch.Tensor]) -> List[torch.Tensor]:
        return self.shared.box.pop(self.rank)

    def rows_before(self, owned: int) -> int:
        # the emulation runs the last rank first, so the caller supplies the counts beforehand
        return sum(self.shared.counts[:self.rank])


class DistLink:
    """Ranks of a torch.distributed group, rank r holding segment r."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def _peer(self, r: int) -> int:
        return r if self.group is None else self.dist.get_global_rank(self.group, r)

    def send_prev(self, tensors: List[torch.Tensor]) -> None:
        for t in tensors:
            self.dist.send(t.contiguous(), self._peer(self.rank - 1), group=self.group)

    def recv_next(self, like: List[torch.Tensor]) -> List[torch.Tensor]:
        out = [torch.empty_like(t) for t in like]
        for t in out:
            self.dist.recv(t, self._peer(self.rank + 1), group=self.group)
        return out

    def rows_before(self, owned: int) -> int:
        mine = torch.tensor([owned], dtype=torch.int64, device="cuda" if self.dist.get_backend(self.group) == "nccl"
                            else "cpu")
        every = [torch.zeros_like(mine) for _ in range(self.world)]
        self.dist.all_gather(every, mine, group=self.group)
        return int(sum(int(c) for c in every[:self.rank]))


@dataclass
class SegmentOutput:
    out_feats: torch.Tensor      # [capacity, D]; the first owned_count rows are this rank's rows
    out_pos: torch.Tensor        # [capacity] ids in the whole video
    owned_count: int
    rows_before: int             # rows owned by earlier ranks: this rank's offset in the packed result
    device_status: torch.Tensor


def message_like(H: int, W: int, D: int, device) -> List[torch.Tensor]:
    """Shapes of one message: number of entries, their cells, weights V and sums S."""
    return [torch.zeros(1, dtype=torch.int32, device=device), torch.zeros(H * W, dtype=torch.int32, device=device),
            torch.zeros(H * W, dtype=torch.float32, device=device),
            torch.zeros((H * W, D), dtype=torch.float32, device=device)]


class SegmentMerge:
    """One rank's part.  ``local`` is ``[T_r (+1), H, W, D]``: the halo first when ``has_halo``."""

    def __init__(self, local: torch.Tensor, has_halo: bool, first_frame: int, tau_s: float, tau_t: float, lv1: int = 4,
                 out_dtype: torch.dtype = torch.bfloat16, pos: int = binding.POS_SURVIVED, wt: int = binding.W_NODE,
                 match: int = binding.MATCH_TOPLEFT):
        if local.dim() != 4 or not local.is_cuda or not local.is_contiguous():
            raise ValueError("local must be a contiguous CUDA tensor [T, H, W, D]")
        if has_halo and local.shape[0] < 2:
            raise ValueError("a segment holds at least one frame besides its halo")
        self.local, self.has_halo, self.first_frame = local, has_halo, first_frame
        self.pos, self.out_dtype = pos, out_dtype
        T, H, W, D = local.shape
        self.T, self.H, self.W, self.D = T, H, W, D
        shape = (1, T, H, W, D)
        self.plan = binding.MergePlan(shape, local.dtype, tau_s, tau_t, lv1, torch.float32, binding.POS_SURVIVED, wt,
                                      None, True, local.device, match)
        self.halo_plan = None
        if has_halo:
            self.halo_plan = binding.MergePlan((1, 1, H, W, D), local.dtype, tau_s, 2.0, lv1, torch.float32,
                                               binding.POS_SURVIVED, wt, None, True, local.device, match)

    def merge_local(self) -> int:
        """The segment's own merge; returns the number of rows this rank owns (synchronises)."""
        self.res = self.plan.run(self.local.unsqueeze(0))
        self.weights = binding.sttm_row_weights(self.plan)
        n_h = 0
        if self.has_halo:
            self.halo = self.halo_plan.run(self.local[:1].unsqueeze(0))
            self.halo_w = binding.sttm_row_weights(self.halo_plan)
            n_h = int(self.halo.out_count[0].item())
        self.count = int(self.res.out_count[0].item())
        self.owned = self.count - n_h
        return self.owned

    def finish(self, link) -> SegmentOutput:
        """Takes in the next rank's message, sends this rank's, writes the owned rows."""
        dev, HW, D = self.local.device, self.H * self.W, self.D
        rows = max(self.count, 1)
        extra = torch.zeros((rows, D), dtype=torch.float32, device=dev)
        extra_w = torch.zeros((rows,), dtype=torch.float32, device=dev)
        status = self.res.device_status
        before = link.rows_before(self.owned)
        if link.rank + 1 < link.world:
            n_dev, anchors, v, s = link.recv_next(message_like(self.H, self.W, D, dev))
            map_last = self.res.merge_map[0, (self.T - 1) * HW:]
            binding.sttm_segment_fold(map_last, anchors, v, s, n_dev, extra, extra_w, status)
        if self.has_halo:
            msg = message_like(self.H, self.W, D, dev)
            msg[0].copy_(self.halo.out_count)
            msg[1][:].copy_(self.halo.out_pos[:HW])
            binding.sttm_segment_emit(self.res.out_feats, self.weights, extra, extra_w, self.halo.out_feats, self.halo_w,
                                      self.halo.out_count, msg[2], msg[3])
            link.send_prev(msg)
        out_feats = torch.empty((rows, D), dtype=self.out_dtype, device=dev)
        out_pos = torch.empty((rows,), dtype=torch.int32, device=dev)
        owned = torch.zeros(1, dtype=torch.int32, device=dev)
        shift = before if self.pos == binding.POS_REASSIGNED else (self.first_frame - (1 if self.has_halo else 0)) * HW
        binding.sttm_segment_finish(self.res.out_feats, self.res.out_pos, self.weights, extra, extra_w,
                                    self.res.out_count, self.halo.out_count if self.has_halo else None, shift,
                                    self.pos, out_feats, out_pos, owned)
        return SegmentOutput(out_feats, out_pos, self.owned, before, status)


def cut_frames(T: int, world: int) -> List[int]:
    """First frame of every segment (and T at the end): as even as the frame count allows."""
    if world < 1 or T < world:
        raise ValueError("every rank needs at least one frame")
    return [r * T // world for r in range(world + 1)]
