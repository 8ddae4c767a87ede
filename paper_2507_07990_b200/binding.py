"""Thin ctypes binding of libsttm.so: argument marshalling only.

Every step of the path runs in the CUDA library; torch is used for device memory and
for the current stream.  There is no fallback: if the library is missing the calls
raise.  Function names follow include/sttm.h.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence, Union

import numpy as np
import torch

from . import build as _build

BF16, F32 = 0, 1
POS_SURVIVED, POS_REASSIGNED = 0, 1
W_NODE, W_AREA = 0, 1
MATCH_TOPLEFT, MATCH_BEST = 0, 1
STATUS_NAMES = ["ok", "bad argument", "unsupported shape", "workspace too small",
                "output capacity exceeded", "root search did not converge", "CUDA error",
                "a wait inside a kernel ran out"]

EXPORTS = ["sttm_default_params", "sttm_workspace_bytes", "sttm_sims_per_frame", "sttm_spatial",
           "sttm_temporal", "sttm_merge_ex", "sttm_merge", "sttm_merge_host", "sttm_release_cache",
           "sttm_last_launch_count", "sttm_status_string", "sttm_stage_count", "sttm_stage_name",
           "sttm_set_stage_events", "sttm_set_tuning", "sttm_set_ring_split", "sttm_last_path", "sttm_last_gram_stage",
           "sttm_fused_launch_shape", "sttm_spatial_static", "sttm_merged_positions",
           "sttm_merged_positions_workspace", "sttm_merge_budget", "sttm_budget_workspace_bytes",
           "sttm_row_weights", "sttm_segment_fold", "sttm_segment_emit", "sttm_segment_finish",
           "sttm_status_from_bits", "sttm_merge_status"]


class SttmParams(C.Structure):
    _fields_ = [("B", C.c_int), ("T", C.c_int), ("H", C.c_int), ("W", C.c_int), ("D", C.c_int),
                ("in_dtype", C.c_int), ("out_dtype", C.c_int), ("lv1", C.c_int),
                ("tau_s", C.c_float), ("tau_t", C.c_float),
                ("tau_s_per_video", C.POINTER(C.c_float)), ("tau_t_per_video", C.POINTER(C.c_float)),
                ("pos", C.c_int), ("wt", C.c_int), ("out_capacity_rows", C.c_longlong), ("match", C.c_int)]


class SttmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else "status %d" % code
        super().__init__("%s failed: %s" % (where, name))


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen libsttm.so (built in-tree by ``build.build()``); raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError("libsttm.so is not built (%s); run `python -m paper_2507_07990_b200.build`" % path)
    lib = C.CDLL(path)
    vp, pp = C.c_void_p, C.POINTER(SttmParams)
    lib.sttm_default_params.argtypes = [pp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float]
    lib.sttm_default_params.restype = None
    lib.sttm_workspace_bytes.argtypes = [pp]
    lib.sttm_workspace_bytes.restype = C.c_size_t
    lib.sttm_sims_per_frame.argtypes = [C.c_int, C.c_int, C.c_int]
    lib.sttm_sims_per_frame.restype = C.c_int
    lib.sttm_spatial.argtypes = [vp, pp, vp, C.c_size_t, vp, vp, vp, vp]
    lib.sttm_spatial.restype = C.c_int
    lib.sttm_spatial_static.argtypes = [vp, pp, vp, vp, vp, vp]
    lib.sttm_spatial_static.restype = C.c_int
    lib.sttm_temporal.argtypes = [vp, pp, vp, C.c_size_t, vp, vp, vp, vp, vp, vp]
    lib.sttm_temporal.restype = C.c_int
    lib.sttm_merge_ex.argtypes = [vp, pp, vp, C.c_size_t, vp, vp, vp, vp, vp, vp, vp]
    lib.sttm_merge_ex.restype = C.c_int
    lib.sttm_merge.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, vp, vp, vp, vp]
    lib.sttm_merge.restype = C.c_int
    lib.sttm_merge_host.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp]
    lib.sttm_merge_host.restype = C.c_int
    lib.sttm_release_cache.argtypes = []
    lib.sttm_release_cache.restype = None
    lib.sttm_last_launch_count.argtypes = []
    lib.sttm_last_launch_count.restype = C.c_int
    lib.sttm_stage_count.argtypes = []
    lib.sttm_stage_count.restype = C.c_int
    lib.sttm_stage_name.argtypes = [C.c_int]
    lib.sttm_stage_name.restype = C.c_char_p
    lib.sttm_set_stage_events.argtypes = [C.POINTER(C.c_void_p)]
    lib.sttm_set_stage_events.restype = None
    lib.sttm_set_tuning.argtypes = [C.c_int, C.c_int, C.c_int]
    lib.sttm_set_tuning.restype = None
    lib.sttm_budget_workspace_bytes.argtypes = [pp]
    lib.sttm_budget_workspace_bytes.restype = C.c_size_t
    lib.sttm_merge_budget.argtypes = [C.c_void_p, pp, C.POINTER(C.c_longlong), C.c_void_p, C.c_size_t, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.sttm_merge_budget.restype = C.c_int
    lib.sttm_merged_positions_workspace.argtypes = [C.c_longlong]
    lib.sttm_merged_positions_workspace.restype = C.c_size_t
    lib.sttm_merged_positions.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_longlong, C.c_void_p, C.c_size_t,
                                          C.c_void_p, C.c_longlong, C.c_void_p, C.c_void_p]
    lib.sttm_merged_positions.restype = C.c_int
    vp = C.c_void_p
    lib.sttm_row_weights.argtypes = [pp, vp, vp, vp, vp, vp]
    lib.sttm_row_weights.restype = C.c_int
    lib.sttm_segment_fold.argtypes = [vp, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp, vp, C.c_longlong, vp, vp]
    lib.sttm_segment_fold.restype = C.c_int
    lib.sttm_segment_emit.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.c_int, C.c_int, vp, vp, vp]
    lib.sttm_segment_emit.restype = C.c_int
    lib.sttm_segment_finish.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.c_int, C.c_longlong, C.c_longlong, C.c_int,
                                        C.c_int, vp, vp, vp, vp]
    lib.sttm_segment_finish.restype = C.c_int
    lib.sttm_set_ring_split.argtypes = [C.c_int, C.c_int]
    lib.sttm_set_ring_split.restype = None
    lib.sttm_status_from_bits.argtypes = [C.c_int32]
    lib.sttm_status_from_bits.restype = C.c_int
    lib.sttm_merge_status.argtypes = [C.POINTER(C.c_int32), vp]
    lib.sttm_merge_status.restype = C.c_int
    lib.sttm_last_path.argtypes = []
    lib.sttm_last_path.restype = C.c_int
    lib.sttm_last_gram_stage.argtypes = []
    lib.sttm_last_gram_stage.restype = C.c_int
    lib.sttm_fused_launch_shape.argtypes = [pp, C.POINTER(C.c_int)]
    lib.sttm_fused_launch_shape.restype = C.c_int
    lib.sttm_status_string.argtypes = [C.c_int]
    lib.sttm_status_string.restype = C.c_char_p
    if path == _build.LIB_PATH:
        _lib = lib
    return lib


def _check(code: int, where: str):
    if code != 0:
        raise SttmError(code, where)


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.bfloat16:
        return BF16
    if t == torch.float32:
        return F32
    raise TypeError("features must be bfloat16 or float32")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Problem:
    """Marshalled parameters plus the keep-alive references ctypes needs."""
    params: SttmParams
    keep: tuple


def make_params(shape: Sequence[int], in_dtype: torch.dtype, tau_s: Union[float, Sequence[float]],
                tau_t: Union[float, Sequence[float]], lv1: int = 4, out_dtype: torch.dtype = torch.bfloat16,
                pos: int = POS_SURVIVED, wt: int = W_NODE, capacity: Optional[int] = None,
                match: int = MATCH_TOPLEFT) -> Problem:
    B, T, H, W, D = shape
    p = SttmParams()
    p.B, p.T, p.H, p.W, p.D = B, T, H, W, D
    p.in_dtype, p.out_dtype, p.lv1 = _dtype_code(in_dtype), _dtype_code(out_dtype), lv1
    keep = []
    if isinstance(tau_s, (float, int)):
        p.tau_s = float(tau_s)
    else:
        arr = (C.c_float * B)(*[float(v) for v in tau_s])
        p.tau_s_per_video = C.cast(arr, C.POINTER(C.c_float))
        keep.append(arr)
    if isinstance(tau_t, (float, int)):
        p.tau_t = float(tau_t)
    else:
        arr = (C.c_float * B)(*[float(v) for v in tau_t])
        p.tau_t_per_video = C.cast(arr, C.POINTER(C.c_float))
        keep.append(arr)
    p.pos, p.wt, p.match = pos, wt, match
    p.out_capacity_rows = B * T * H * W if capacity is None else capacity
    return Problem(p, tuple(keep))


def sttm_workspace_bytes(problem: Problem) -> int:
    return int(load_library().sttm_workspace_bytes(C.byref(problem.params)))


def sttm_fused_launch_shape(problem: Problem) -> Optional[dict]:
    """Launch shape of the fused kernel for a problem, or None when it does not apply."""
    arr = (C.c_int * 12)()
    if not load_library().sttm_fused_launch_shape(C.byref(problem.params), arr):
        return None
    names = ["cluster_size", "channels_per_cta", "threads", "ring_slots", "smem_bytes", "frames_per_item", "items",
             "resident_clusters", "clusters", "mma_warps", "sum_ring_slots", "lead_frames"]
    return dict(zip(names, list(arr)))


def sttm_sims_per_frame(H: int, W: int, lv1: int = 4) -> int:
    return int(load_library().sttm_sims_per_frame(H, W, lv1))


def _as5d(feats: torch.Tensor) -> torch.Tensor:
    if feats.dim() == 4:
        feats = feats.unsqueeze(0)
    if feats.dim() != 5 or not feats.is_cuda or not feats.is_contiguous():
        raise ValueError("features must be a contiguous CUDA tensor [B, T, H, W, D] or [T, H, W, D]")
    return feats


def alloc_workspace(problem: Problem, device) -> torch.Tensor:
    n = sttm_workspace_bytes(problem)
    if n == 0:
        # let the library name the reason
        _check(load_library().sttm_spatial(None, C.byref(problem.params), None, 0, None, None, None, None),
               "sttm_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def sttm_spatial(feats: torch.Tensor, tau_s, lv1: int = 4, want_sims: bool = False, ws: Optional[torch.Tensor] = None):
    """Spatial stage alone.  Returns (cover_level int8 [B,T,H,W], frame_counts int32 [B,T],
    spatial_sims float32 [B,T,sims_per_frame] or None, workspace)."""
    feats = _as5d(feats)
    B, T, H, W, D = feats.shape
    prob = make_params(feats.shape, feats.dtype, tau_s, 2.0, lv1)
    ws = alloc_workspace(prob, feats.device) if ws is None else ws
    cover = torch.empty((B, T, H, W), dtype=torch.int8, device=feats.device)
    counts = torch.empty((B, T), dtype=torch.int32, device=feats.device)
    sims = None
    if want_sims:
        sims = torch.full((B, T, sttm_sims_per_frame(H, W, lv1)), float("nan"), dtype=torch.float32,
                          device=feats.device)
    _check(load_library().sttm_spatial(_ptr(feats), C.byref(prob.params), _ptr(ws), ws.numel(), _ptr(cover),
                                       _ptr(counts), _ptr(sims), _stream()), "sttm_spatial")
    return cover, counts, sims, ws


def sttm_spatial_static(feats: torch.Tensor, tau_s, cover: torch.Tensor, counts: torch.Tensor,
                        sims: Optional[torch.Tensor] = None, lv1: int = 4) -> None:
    """Spatial stage through the entry point that allocates nothing: the caller passes every
    output buffer (``cover`` int8 [B,T,H,W], ``counts`` int32 [B,T], optionally ``sims`` float32
    [B,T,sims_per_frame]); the stage's scratch is the fixed array inside the library.  Raises
    SttmError("workspace too small") when the problem needs more scratch than that array has."""
    feats = _as5d(feats)
    prob = make_params(feats.shape, feats.dtype, tau_s, 2.0, lv1)
    _check(load_library().sttm_spatial_static(_ptr(feats), C.byref(prob.params), _ptr(cover), _ptr(counts),
                                              _ptr(sims), _stream()), "sttm_spatial_static")


def sttm_temporal(feats: torch.Tensor, cover: torch.Tensor, tau_s, tau_t, ws: torch.Tensor, lv1: int = 4,
                  want_sims: bool = False, match: int = MATCH_TOPLEFT):
    """Temporal stage alone, on a workspace sttm_spatial has filled.  Returns (link, root,
    temporal_sims or None, device_status)."""
    feats = _as5d(feats)
    B, T, H, W, D = feats.shape
    prob = make_params(feats.shape, feats.dtype, tau_s, tau_t, lv1, match=match)
    link = torch.empty((B, T * H * W), dtype=torch.int32, device=feats.device)
    root = torch.empty((B, T * H * W), dtype=torch.int32, device=feats.device)
    tsim = torch.empty((B, T * H * W), dtype=torch.float32, device=feats.device) if want_sims else None
    status = torch.zeros(1, dtype=torch.int32, device=feats.device)
    _check(load_library().sttm_temporal(_ptr(feats), C.byref(prob.params), _ptr(ws), ws.numel(), _ptr(cover),
                                        _ptr(link), _ptr(root), _ptr(tsim), _ptr(status), _stream()),
           "sttm_temporal")
    return link, root, tsim, status


@dataclass
class MergeOutput:
    out_feats: torch.Tensor      # [capacity, D]
    out_pos: torch.Tensor        # [capacity] int32
    out_count: torch.Tensor      # [B] int32
    out_offsets: torch.Tensor    # [B+1] int64
    merge_map: Optional[torch.Tensor]
    device_status: torch.Tensor
    launches: int


class MergePlan:
    """Pre-allocated buffers for repeated sttm_merge_ex calls on one problem shape."""

    def __init__(self, shape, in_dtype, tau_s, tau_t, lv1=4, out_dtype=torch.bfloat16, pos=POS_SURVIVED,
                 wt=W_NODE, capacity=None, want_map=False, device="cuda", match=MATCH_TOPLEFT):
        self.problem = make_params(shape, in_dtype, tau_s, tau_t, lv1, out_dtype, pos, wt, capacity, match)
        p = self.problem.params
        B, T, H, W, D = shape
        self.ws = alloc_workspace(self.problem, device)
        cap = int(p.out_capacity_rows)
        self.out_feats = torch.empty((cap, D), dtype=out_dtype, device=device)
        self.out_pos = torch.empty((cap,), dtype=torch.int32, device=device)
        self.out_count = torch.empty((B,), dtype=torch.int32, device=device)
        self.out_offsets = torch.empty((B + 1,), dtype=torch.int64, device=device)
        self.merge_map = torch.empty((B, T * H * W), dtype=torch.int32, device=device) if want_map else None
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def run(self, feats: torch.Tensor) -> MergeOutput:
        lib = load_library()
        _check(lib.sttm_merge_ex(_ptr(feats), C.byref(self.problem.params), _ptr(self.ws), self.ws.numel(),
                                 _ptr(self.out_feats), _ptr(self.out_pos), _ptr(self.merge_map),
                                 _ptr(self.out_count), _ptr(self.out_offsets), _ptr(self.status), _stream()),
               "sttm_merge_ex")
        return MergeOutput(self.out_feats, self.out_pos, self.out_count, self.out_offsets, self.merge_map,
                           self.status, int(lib.sttm_last_launch_count()))


def sttm_merge_ex(feats: torch.Tensor, tau_s, tau_t, lv1: int = 4, out_dtype: torch.dtype = torch.bfloat16,
                  pos: int = POS_SURVIVED, wt: int = W_NODE, capacity: Optional[int] = None,
                  want_map: bool = True, match: int = MATCH_TOPLEFT) -> MergeOutput:
    """The whole path for ``[B, T, H, W, D]`` (or one video ``[T, H, W, D]``)."""
    feats = _as5d(feats)
    plan = MergePlan(tuple(feats.shape), feats.dtype, tau_s, tau_t, lv1, out_dtype, pos, wt, capacity, want_map,
                     feats.device, match)
    return plan.run(feats)


def sttm_row_weights(plan: MergePlan) -> torch.Tensor:
    """Weight of every row of the plan's last run (which must have kept its merge map)."""
    p = plan.problem.params
    rows = min(int(p.B * p.T * p.H * p.W), int(p.out_capacity_rows))
    weights = torch.empty((rows,), dtype=torch.float32, device=plan.ws.device)
    _check(load_library().sttm_row_weights(C.byref(p), _ptr(plan.ws), _ptr(plan.merge_map), _ptr(plan.out_offsets),
                                           _ptr(weights), _stream()), "sttm_row_weights")
    return weights


def sttm_segment_fold(map_last, anchors, v, s, n_dev, extra, extra_w, status) -> None:
    n_max, D = s.shape
    _check(load_library().sttm_segment_fold(_ptr(map_last), _ptr(anchors), _ptr(v), _ptr(s), _ptr(n_dev), n_max,
                                            map_last.numel(), D, _ptr(extra), _ptr(extra_w), extra_w.numel(),
                                            _ptr(status), _stream()), "sttm_segment_fold")


def sttm_segment_emit(feats, weights, extra, extra_w, halo_feats, halo_w, n_h_dev, v_out, s_out) -> None:
    n_max, D = s_out.shape
    _check(load_library().sttm_segment_emit(_ptr(feats), _ptr(weights), _ptr(extra), _ptr(extra_w), _ptr(halo_feats),
                                            _ptr(halo_w), _ptr(n_h_dev), n_max, D, _ptr(v_out), _ptr(s_out),
                                            _stream()), "sttm_segment_emit")


def sttm_segment_finish(feats, pos, weights, extra, extra_w, count_dev, n_h_dev, pos_shift, pos_mode, out_feats,
                        out_pos, owned_count) -> None:
    _check(load_library().sttm_segment_finish(_ptr(feats), _ptr(pos), _ptr(weights), _ptr(extra), _ptr(extra_w),
                                              _ptr(count_dev), _ptr(n_h_dev), feats.shape[1], extra_w.numel(),
                                              pos_shift, pos_mode, _dtype_code(out_feats.dtype), _ptr(out_feats),
                                              _ptr(out_pos), _ptr(owned_count), _stream()), "sttm_segment_finish")


class BudgetPlan:
    """Pre-allocated buffers for repeated sttm_merge_budget calls on one problem shape."""

    def __init__(self, shape, in_dtype, tau_s, budget_rows, lv1=4, out_dtype=torch.bfloat16, want_map=False,
                 device="cuda"):
        B, T, H, W, D = shape
        self.problem = make_params(shape, in_dtype, tau_s, 2.0, lv1, out_dtype)
        p = self.problem.params
        lib = load_library()
        need = int(lib.sttm_budget_workspace_bytes(C.byref(p)))
        if need == 0:
            raise SttmError(2, "sttm_budget_workspace_bytes")
        ws = torch.empty(need + 256, dtype=torch.uint8, device=device)
        self.ws = ws[(-ws.data_ptr()) % 256:]
        cap = int(p.out_capacity_rows)
        self.out_feats = torch.empty((cap, D), dtype=out_dtype, device=device)
        self.out_pos = torch.empty((cap,), dtype=torch.int32, device=device)
        self.out_count = torch.empty((B,), dtype=torch.int32, device=device)
        self.out_offsets = torch.empty((B + 1,), dtype=torch.int64, device=device)
        self.merge_map = torch.empty((B, T * H * W), dtype=torch.int32, device=device) if want_map else None
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.tau = torch.empty((B,), dtype=torch.float32, device=device)
        rows = budget_rows if hasattr(budget_rows, "__len__") else [budget_rows] * B
        self.budgets = (C.c_longlong * B)(*[int(v) for v in rows])

    def run(self, feats: torch.Tensor) -> MergeOutput:
        lib = load_library()
        _check(lib.sttm_merge_budget(_ptr(feats), C.byref(self.problem.params), self.budgets, _ptr(self.ws),
                                     self.ws.numel(), _ptr(self.out_feats), _ptr(self.out_pos), _ptr(self.merge_map),
                                     _ptr(self.out_count), _ptr(self.out_offsets), _ptr(self.tau), _ptr(self.status),
                                     _stream()), "sttm_merge_budget")
        return MergeOutput(self.out_feats, self.out_pos, self.out_count, self.out_offsets, self.merge_map,
                           self.status, int(lib.sttm_last_launch_count()))


def sttm_merge_budget(feats: torch.Tensor, tau_s: float, budget_rows, lv1: int = 4,
                      out_dtype: torch.dtype = torch.bfloat16, want_map: bool = True):
    """Budget mode: tau_s as given, tau_t chosen per video on the device so that video v keeps at
    most ``budget_rows[v]`` rows.  Returns (MergeOutput, tau_t [B] float32 on the device)."""
    feats = _as5d(feats)
    plan = BudgetPlan(tuple(feats.shape), feats.dtype, tau_s, budget_rows, lv1, out_dtype, want_map, feats.device)
    return plan.run(feats), plan.tau


def sttm_merged_positions(merge_map: torch.Tensor, out_offsets: torch.Tensor, rows: int):
    """Mean member index of every output row ("merged" positions of Section 3.4) from the merge map and
    the video offsets that sttm_merge_ex wrote.  Returns (float32 [rows], device_status)."""
    if merge_map.dim() != 2 or merge_map.dtype != torch.int32 or not merge_map.is_cuda or not merge_map.is_contiguous():
        raise ValueError("merge_map must be a contiguous int32 CUDA tensor [B, N]")
    B, N = merge_map.shape
    lib = load_library()
    ws = torch.empty(int(lib.sttm_merged_positions_workspace(rows)) + 256, dtype=torch.uint8, device=merge_map.device)
    ws = ws[(-ws.data_ptr()) % 256:]
    out = torch.empty((rows,), dtype=torch.float32, device=merge_map.device)
    status = torch.zeros(1, dtype=torch.int32, device=merge_map.device)
    _check(lib.sttm_merged_positions(_ptr(merge_map), _ptr(out_offsets), B, N, _ptr(ws), ws.numel(), _ptr(out), rows,
                                     _ptr(status), _stream()), "sttm_merged_positions")
    return out, status


def sttm_merge(feats: torch.Tensor, tau_s: float, tau_t: float):
    """One bf16 video with the default settings.  Returns (out_feats [N, D], out_pos [N], out_count [1])."""
    if feats.dim() != 4 or feats.dtype != torch.bfloat16 or not feats.is_cuda or not feats.is_contiguous():
        raise ValueError("sttm_merge takes one contiguous bf16 CUDA video [T, H, W, D]")
    T, H, W, D = feats.shape
    out = torch.empty((T * H * W, D), dtype=torch.bfloat16, device=feats.device)
    pos = torch.empty((T * H * W,), dtype=torch.int32, device=feats.device)
    cnt = torch.empty((1,), dtype=torch.int32, device=feats.device)
    _check(load_library().sttm_merge(_ptr(feats), T, H, W, D, float(tau_s), float(tau_t), _ptr(out), _ptr(pos),
                                     _ptr(cnt), _stream()), "sttm_merge")
    return out, pos, cnt


def sttm_merge_host(h_feats: torch.Tensor, tau_s, tau_t, lv1: int = 4, out_dtype: torch.dtype = torch.bfloat16,
                    pos: int = POS_SURVIVED, wt: int = W_NODE, h_out_feats: Optional[torch.Tensor] = None,
                    h_out_pos: Optional[torch.Tensor] = None, want_map: bool = False):
    """Host-buffer entry point: ``h_feats`` is a CPU tensor (pinned for speed)
    ``[B, T, H, W, D]``; outputs are CPU tensors.  Copies are part of the call."""
    if h_feats.dim() == 4:
        h_feats = h_feats.unsqueeze(0)
    if h_feats.is_cuda or not h_feats.is_contiguous():
        raise ValueError("sttm_merge_host takes a contiguous CPU tensor")
    B, T, H, W, D = h_feats.shape
    prob = make_params(h_feats.shape, h_feats.dtype, tau_s, tau_t, lv1, out_dtype, pos, wt)
    cap = int(prob.params.out_capacity_rows)
    if h_out_feats is None:
        h_out_feats = torch.empty((cap, D), dtype=out_dtype).pin_memory()
    if h_out_pos is None:
        h_out_pos = torch.empty((cap,), dtype=torch.int32).pin_memory()
    h_map = torch.empty((B, T * H * W), dtype=torch.int32) if want_map else None
    h_cnt = torch.zeros((B,), dtype=torch.int32)
    h_off = torch.zeros((B + 1,), dtype=torch.int64)
    h_status = torch.zeros((1,), dtype=torch.int32)
    _check(load_library().sttm_merge_host(_ptr(h_feats), C.byref(prob.params), _ptr(h_out_feats), _ptr(h_out_pos),
                                          _ptr(h_map), _ptr(h_cnt), _ptr(h_off), _ptr(h_status)),
           "sttm_merge_host")
    return MergeOutput(h_out_feats, h_out_pos, h_cnt, h_off, h_map, h_status, 0)


class StageTimer:
    """Records one CUDA event per stage boundary of sttm_merge_ex (on the stream the
    kernels run on) and reports the time each stage took."""

    def __init__(self):
        lib = load_library()
        self.names = [lib.sttm_stage_name(i).decode() for i in range(lib.sttm_stage_count())]
        self.events = [torch.cuda.Event(enable_timing=True) for _ in range(len(self.names) + 1)]
        for e in self.events:
            e.record()                      # forces creation of the underlying cudaEvent_t
        torch.cuda.synchronize()
        self._handles = (C.c_void_p * len(self.events))(*[C.c_void_p(e.cuda_event) for e in self.events])

    def __enter__(self):
        load_library().sttm_set_stage_events(self._handles)
        return self

    def __exit__(self, *exc):
        load_library().sttm_set_stage_events(None)

    def stage_ms(self):
        """Call after a synchronize: milliseconds of every stage of the last call."""
        return {n: self.events[i].elapsed_time(self.events[i + 1]) for i, n in enumerate(self.names)}
