"""Seeded synthetic videos for the STTM token-merging path.

This module only *draws inputs*: it holds none of the method's arithmetic (no pooling,
no similarity, no merging) and is the one piece of code that both the CUDA path and the
CPU oracle's tests consume.  The same byte buffer is handed to both sides.

Recipe ("block generator"): K random object vectors; every frame is a quadtree
subdivision of the token grid (padded to a power of two, blocks clipped to H x W) whose
leaf blocks each carry one object id; a token is its block's object vector plus fresh
Gaussian noise per token, per frame and per channel.  From frame to frame a leaf block
persists (same block, same object) with probability ``p_static``, otherwise it is
replaced by a fresh random subtree rooted at itself; when three or more of four sibling
leaves are replaced in the same frame their parent is replaced instead, which lets
blocks coarsen again and keeps long videos stationary.  The root block always splits
(a frame is never one single object); every other block splits with ``split_p``.

Contrast.  A leaf block also draws a contrast, one of ``VideoSpec.contrast`` with equal
probability, which multiplies its object vector (not the noise) for as long as the block
persists.  With one class (the default) every block has contrast 1 and all similarities
of same-object tokens fall into one narrow cluster, so a threshold can only switch
merging on or off.  With several classes the similarities form one cluster per class
and level (cosine of two noisy copies of a.o is a^2 / (a^2 + sigma^2) for leaves), the
clusters are separated by gaps far wider than the decision margin, and thresholds placed
between them decide which classes merge: that is what lets a workload land near a stated
token budget.

Random numbers come from numpy's counter-based Philox generator, keyed by
(seed, stream, frame), so a frame's noise does not depend on generation order.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field, asdict
from typing import List, Optional, Tuple

import numpy as np

__all__ = [
    "VideoSpec", "CONFIGS", "config_videos", "make_video", "frame_structure",
    "f32_to_bf16_bits", "bf16_bits_to_f32", "load_thresholds", "THRESHOLDS_PATH",
]

_STREAM_OBJECTS = 0
_STREAM_STRUCTURE = 1
_STREAM_NOISE = 2          # + frame index


def _rng(seed: int, stream: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ stream, sub]))


# ----------------------------------------------------------------------------------
# bf16 <-> f32 bit conversions (round to nearest even), plain integer arithmetic
# ----------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------
# block structure
# ----------------------------------------------------------------------------------
class _Node:
    """A block of the generator's quadtree: a leaf with an object id, or four children."""
    __slots__ = ("obj", "kids", "amp")

    def __init__(self, obj: int = -1, kids=None, amp: int = 0):
        self.obj = obj
        self.amp = amp          # index into VideoSpec.contrast
        self.kids = kids        # list of 4 (_Node or None) in (top-left, top-right, bottom-left, bottom-right) order


def _in_bounds(depth: int, bi: int, bj: int, side0: int, H: int, W: int) -> bool:
    s = side0 >> depth
    return bi * s < H and bj * s < W


def _fresh(rng, depth, bi, bj, spec, side0) -> "_Node":
    if depth < spec.depth_max and (depth == 0 or rng.random() < spec.split_p):
        kids = []
        for a in (0, 1):
            for b in (0, 1):
                ci, cj = 2 * bi + a, 2 * bj + b
                if _in_bounds(depth + 1, ci, cj, side0, spec.H, spec.W):
                    kids.append(_fresh(rng, depth + 1, ci, cj, spec, side0))
                else:
                    kids.append(None)
        return _Node(kids=kids)
    obj = int(rng.integers(spec.K))
    # (a single contrast class draws nothing, so such videos are what they were without the option)
    amp = int(rng.integers(len(spec.contrast))) if len(spec.contrast) > 1 else 0
    return _Node(obj=obj, amp=amp)


def _evolve(rng, node, depth, bi, bj, spec, side0) -> Tuple["_Node", bool]:
    """Next frame's version of ``node``; second value: was a leaf and got replaced."""
    if node.kids is None:
        if rng.random() < spec.p_static:
            return node, False
        return _fresh(rng, depth, bi, bj, spec, side0), True
    new_kids, replaced_leaves = [], 0
    for k, kid in enumerate(node.kids):
        if kid is None:
            new_kids.append(None)
            continue
        nk, rep = _evolve(rng, kid, depth + 1, 2 * bi + (k >> 1), 2 * bj + (k & 1), spec, side0)
        new_kids.append(nk)
        replaced_leaves += int(rep)
    if replaced_leaves >= 3:
        return _fresh(rng, depth, bi, bj, spec, side0), False
    return _Node(kids=new_kids), False


def _paint(node, depth, bi, bj, side0, obj_map, depth_map, amp_map):
    H, W = obj_map.shape
    s = side0 >> depth
    if node.kids is None:
        obj_map[bi * s:min((bi + 1) * s, H), bj * s:min((bj + 1) * s, W)] = node.obj
        depth_map[bi * s:min((bi + 1) * s, H), bj * s:min((bj + 1) * s, W)] = depth
        amp_map[bi * s:min((bi + 1) * s, H), bj * s:min((bj + 1) * s, W)] = node.amp
        return
    for k, kid in enumerate(node.kids):
        if kid is not None:
            _paint(kid, depth + 1, 2 * bi + (k >> 1), 2 * bj + (k & 1), side0, obj_map, depth_map, amp_map)


@dataclass
class VideoSpec:
    """One synthetic video.  ``unit`` is the normalisation of the object vectors:
    'rms' gives every object unit root-mean-square per channel (L2 norm sqrt(D)),
    'l2' gives unit L2 norm."""
    T: int
    H: int
    W: int
    D: int
    dtype: str = "bf16"            # 'bf16' or 'f32'
    depth_max: int = 3
    p_static: float = 0.8
    sigma: float = 0.05
    split_p: float = 0.5
    K: int = 16
    unit: str = "rms"
    contrast: Tuple[float, ...] = (1.0,)   # contrast classes of a leaf block, drawn with equal probability
    scale_unit_rms: bool = True    # multiply the tensor by one scalar so tokens have unit RMS
    seed: int = 20250707

    @property
    def tokens(self) -> int:
        return self.T * self.H * self.W


def frame_structure(spec: VideoSpec, want_contrast: bool = False):
    """Object-id map and block-depth map, both ``[T, H, W]`` (int16 / int8); with
    ``want_contrast`` also the map of contrast-class indices (int8)."""
    side0 = 1
    while side0 < max(spec.H, spec.W):
        side0 *= 2
    rng = _rng(spec.seed, _STREAM_STRUCTURE)
    obj = np.zeros((spec.T, spec.H, spec.W), dtype=np.int16)
    dep = np.zeros((spec.T, spec.H, spec.W), dtype=np.int8)
    amp = np.zeros((spec.T, spec.H, spec.W), dtype=np.int8)
    root = _fresh(rng, 0, 0, 0, spec, side0)
    for t in range(spec.T):
        if t > 0:
            root, _ = _evolve(rng, root, 0, 0, 0, spec, side0)
        _paint(root, 0, 0, 0, side0, obj[t], dep[t], amp[t])
    return (obj, dep, amp) if want_contrast else (obj, dep)


def _objects(spec: VideoSpec) -> np.ndarray:
    o = _rng(spec.seed, _STREAM_OBJECTS).standard_normal((spec.K, spec.D)).astype(np.float64)
    o /= np.sqrt((o * o).sum(axis=1, keepdims=True))
    if spec.unit == "rms":
        o *= np.sqrt(spec.D)
    elif spec.unit != "l2":
        raise ValueError("unit must be 'rms' or 'l2'")
    return o.astype(np.float32)


def make_video(spec: VideoSpec, out: Optional[np.ndarray] = None) -> np.ndarray:
    """Generate the video.  Returns ``[T, H, W, D]`` float32 (dtype 'f32') or the bf16
    bit patterns as uint16 (dtype 'bf16').  ``out`` may supply the destination buffer
    (e.g. pinned host memory viewed as a numpy array)."""
    objs = _objects(spec)
    obj_map, _, amp_map = frame_structure(spec, want_contrast=True)
    amps = np.asarray(spec.contrast, dtype=np.float32)
    if spec.scale_unit_rms:
        # expected mean square of a token (contrast classes are equally likely per block)
        mean_sq = float((objs.astype(np.float64) ** 2).mean()) * float((amps.astype(np.float64) ** 2).mean()) \
            + spec.sigma ** 2
        scale = np.float32(1.0 / np.sqrt(mean_sq))
    else:
        scale = np.float32(1.0)
    np_dtype = np.uint16 if spec.dtype == "bf16" else np.float32
    shape = (spec.T, spec.H, spec.W, spec.D)
    if out is None:
        out = np.empty(shape, dtype=np_dtype)
    assert out.shape == shape and out.dtype == np_dtype
    hw = spec.H * spec.W
    for t in range(spec.T):
        noise = _rng(spec.seed, _STREAM_NOISE, t).standard_normal((hw, spec.D), dtype=np.float32)
        noise *= np.float32(spec.sigma)
        if len(amps) > 1:
            noise += objs[obj_map[t].reshape(hw)] * amps[amp_map[t].reshape(hw)][:, None]
        else:
            noise += objs[obj_map[t].reshape(hw)]
        noise *= scale
        if spec.dtype == "bf16":
            out[t] = f32_to_bf16_bits(noise).reshape(spec.H, spec.W, spec.D)
        else:
            out[t] = noise.reshape(spec.H, spec.W, spec.D)
    return out


# ----------------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------------
BASE_SEED = 20250707
# contrast classes of the workloads that are run at a token budget
CONTRAST = (1.0, 0.5, 0.35, 0.25, 0.18, 0.12)

CONFIGS = {
    # name: shared fields; 'p_static' is a list with one entry per video
    "tiny":  dict(index=1, T=4, H=8, W=8, D=64, dtype="f32", depth_max=3, sigma=0.05,
                  p_static=[0.8], scale_unit_rms=False, budgets=[None], fixed_tau=(0.9, 0.9)),
    "llava": dict(index=2, contrast=CONTRAST, T=64, H=13, W=13, D=3584, dtype="bf16", depth_max=3, sigma=0.05,
                  p_static=[0.8], scale_unit_rms=True, budgets=[0.5, 0.3]),
    "qwen":  dict(index=3, contrast=CONTRAST, T=128, H=16, W=16, D=3584, dtype="bf16", depth_max=4, sigma=0.08,
                  p_static=[0.7], scale_unit_rms=True, budgets=[0.5]),
    "long":  dict(index=4, contrast=CONTRAST, T=1024, H=13, W=13, D=3584, dtype="bf16", depth_max=3, sigma=0.05,
                  p_static=[0.9], scale_unit_rms=True, budgets=[0.3]),
    "mixed": dict(index=5, contrast=CONTRAST, T=64, H=13, W=13, D=3584, dtype="bf16", depth_max=3, sigma=0.05,
                  p_static=[0.95, 0.9, 0.8, 0.7, 0.6, 0.5, 0.3, 0.1], scale_unit_rms=True,
                  budgets=[0.5, 0.3]),
}


def config_videos(name: str, seed_bump: int = 0) -> List[VideoSpec]:
    """The VideoSpec of every video of a named workload."""
    c = CONFIGS[name]
    specs = []
    for v, p in enumerate(c["p_static"]):
        specs.append(VideoSpec(T=c["T"], H=c["H"], W=c["W"], D=c["D"], dtype=c["dtype"],
                               depth_max=c["depth_max"], p_static=p, sigma=c["sigma"],
                               scale_unit_rms=c["scale_unit_rms"], contrast=tuple(c.get("contrast", (1.0,))),
                               seed=BASE_SEED + c["index"] + 100 * v + 1000 * seed_bump))
    return specs


THRESHOLDS_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "workload_thresholds.json")


def load_thresholds() -> dict:
    """Thresholds (tau_s, tau_t) per workload, video and budget.  The file is written by
    the calibration script that sits beside the CPU oracle; it is data, not code."""
    with open(THRESHOLDS_PATH) as f:
        return json.load(f)
