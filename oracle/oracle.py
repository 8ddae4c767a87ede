"""ctypes front end of the CPU oracle (oracle/sttm_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module.
It compiles the C file with gcc on first use (``build()``) and never touches the CUDA
library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sttm_oracle.c")
_HDR = os.path.join(_HERE, "sttm_oracle.h")
_LIB = os.path.join(_HERE, "_build", "libsttm_oracle.so")

BF16, F32, F64 = 0, 1, 2
W_NODE, W_AREA = 0, 1
POS_SURVIVED, POS_REASSIGNED = 0, 1
MATCH_TOPLEFT, MATCH_BEST, MATCH_TOPLEFT_ONLY = 0, 1, 2


class _Cfg(C.Structure):
    _fields_ = [("T", C.c_int), ("H", C.c_int), ("W", C.c_int), ("D", C.c_int),
                ("dtype", C.c_int), ("lv1", C.c_int),
                ("tau_s", C.c_double), ("tau_t", C.c_double),
                ("weight_mode", C.c_int), ("pos_mode", C.c_int), ("match_mode", C.c_int)]


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, strict IEEE arithmetic).  Returns the library path."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-fno-fast-math",
                               "-ffp-contract=off", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.oracle_levels.restype = C.c_int
        lib.oracle_levels.argtypes = [C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        lib.oracle_sims_per_frame.restype = C.c_int
        lib.oracle_sims_per_frame.argtypes = [C.c_int, C.c_int, C.c_int]
        lib.oracle_merge.restype = C.c_int64
        lib.oracle_merge.argtypes = [C.c_void_p, C.POINTER(_Cfg)] + [C.c_void_p] * 8 + [C.c_int64] \
            + [C.c_void_p] * 3 + [C.c_int64, C.c_void_p]
        _lib = lib
    return _lib


def levels(H: int, W: int, lv1: int = 4):
    """[(H_l, W_l)] for l = 0 (token grid) .. L-1 (coarsest map)."""
    Hl = (C.c_int * 24)()
    Wl = (C.c_int * 24)()
    L = _load().oracle_levels(H, W, lv1, Hl, Wl)
    return [(Hl[l], Wl[l]) for l in range(L)]


@dataclass
class OracleResult:
    count: int
    spatial_sims: Optional[np.ndarray]   # [T, sims_per_frame] float64
    cover_level: np.ndarray              # [T, H, W] int8
    link: np.ndarray                     # [T*H*W] int32
    root: np.ndarray                     # [T*H*W] int32
    merge_map: np.ndarray                # [T*H*W] int32
    out_feats: Optional[np.ndarray]      # [count, D] float64
    out_pos: np.ndarray                  # [count] int32
    out_members: np.ndarray              # [count] int32
    tsim_v: Optional[np.ndarray]
    tsim_u: Optional[np.ndarray]
    tsim: Optional[np.ndarray]
    comparisons_spatial: int
    comparisons_temporal: int


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    raise TypeError("features must be uint16 (bf16 bits), float32 or float64")


def merge(feats: np.ndarray, tau_s: float, tau_t: float, lv1: int = 4,
          weight_mode: int = W_NODE, pos_mode: int = POS_SURVIVED, match_mode: int = MATCH_TOPLEFT,
          want_feats: bool = True, want_sims: bool = False, want_pairs: bool = False) -> OracleResult:
    """Run the whole path on one video ``[T, H, W, D]``."""
    lib = _load()
    feats = np.ascontiguousarray(feats)
    T, H, W, D = feats.shape
    N = T * H * W
    cfg = _Cfg(T, H, W, D, _dtype_code(feats), lv1, float(tau_s), float(tau_t),
               weight_mode, pos_mode, match_mode)
    nsim = lib.oracle_sims_per_frame(H, W, lv1)
    sims = np.zeros((T, nsim), dtype=np.float64) if want_sims else None
    cover = np.zeros((T, H, W), dtype=np.int8)
    link = np.zeros(N, dtype=np.int32)
    root = np.zeros(N, dtype=np.int32)
    mmap = np.zeros(N, dtype=np.int32)
    pos = np.zeros(N, dtype=np.int32)
    members = np.zeros(N, dtype=np.int32)
    counters = np.zeros(3, dtype=np.int64)
    pair_cap = 0
    tv = tu = ts = None
    if want_pairs:
        pair_cap = 2 * N        # each kept node of frames t and t-1 is in at most this many pairs
        tv = np.zeros(pair_cap, dtype=np.int32)
        tu = np.zeros(pair_cap, dtype=np.int32)
        ts = np.zeros(pair_cap, dtype=np.float64)

    def p(a):
        return a.ctypes.data_as(C.c_void_p) if a is not None else None

    out = None
    cap = N
    if want_feats:
        # first pass without features to learn the row count, so that the feature buffer is exact
        cnt = lib.oracle_merge(p(feats), C.byref(cfg), None, None, None, None, None, None, None, None,
                               0, None, None, None, 0, None)
        if cnt < 0:
            raise ValueError("oracle_merge rejected its arguments")
        out = np.zeros((max(int(cnt), 1), D), dtype=np.float64)
        cap = int(cnt)
    count = lib.oracle_merge(p(feats), C.byref(cfg), p(sims), p(cover), p(link), p(root), p(mmap),
                             p(out), p(pos), p(members), cap, p(tv), p(tu), p(ts), pair_cap, p(counters))
    if count < 0:
        raise ValueError("oracle_merge rejected its arguments")
    count = int(count)
    npairs = int(counters[2])
    if want_pairs:
        assert npairs <= pair_cap
        tv, tu, ts = tv[:npairs], tu[:npairs], ts[:npairs]
    return OracleResult(count, sims, cover, link, root, mmap,
                        out[:count] if out is not None else None, pos[:count], members[:count],
                        tv, tu, ts, int(counters[0]), int(counters[1]))


def merged_positions(merge_map: np.ndarray, count: int) -> np.ndarray:
    """Section 3.4, "merged" position strategy, read as: the position of an output row is the mean
    of the indices (t*H*W + y*W + x) of the cells merged into it.  ``merge_map`` holds the row of
    every cell of one video.  Plain definition: integer sums, one division in double precision,
    one rounding to float32."""
    merge_map = np.asarray(merge_map).reshape(-1)
    sums = np.zeros(count, dtype=np.int64)
    cnts = np.zeros(count, dtype=np.int64)
    for i, r in enumerate(merge_map.tolist()):
        sums[r] += i
        cnts[r] += 1
    return (sums.astype(np.float64) / cnts.astype(np.float64)).astype(np.float32)


def best_candidate_cosines(feats: np.ndarray, tau_s: float, lv1: int = 4):
    """(number of kept nodes, descending array with, for every kept node that has candidates in
    the frame before it, the largest cosine to them) under the cover maps that ``tau_s`` gives."""
    base = merge(feats, tau_s, 2.0, lv1=lv1, want_feats=False, want_pairs=True)
    best = {}
    for v, sim in zip(base.tsim_v.tolist(), base.tsim.tolist()):
        best[v] = max(best.get(v, -2.0), sim)
    return base.count, np.sort(np.array(list(best.values()), dtype=np.float64))[::-1]


def budget_tau_t(feats: np.ndarray, tau_s: float, budget_rows: int, lv1: int = 4):
    """Budget mode (the adaptive threshold the paper names as future work): with the cover maps
    fixed by ``tau_s``, a kept node is merged into the frame before iff the largest cosine to its
    candidates exceeds tau_t, so the row count is nodes - #{best cosine > tau_t}.  Returns
    (tau_t, gap): the middle of the gap between the k-th and the (k+1)-th largest best cosine,
    k = nodes - budget, and the width of that gap; (2.0, inf) when no temporal merging is needed,
    (-2.0, 0) when the budget cannot be met.  Plain definition on top of ``merge``."""
    nodes, m = best_candidate_cosines(feats, tau_s, lv1)
    k = nodes - int(budget_rows)
    if k <= 0:
        return 2.0, float("inf")
    if k > len(m):
        return -2.0, 0.0
    mk = m[k - 1]
    mk1 = m[k] if k < len(m) else mk - 2e-3
    return 0.5 * (mk + mk1), float(mk - mk1)
