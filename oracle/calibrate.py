"""Choose (tau_S, tau_T) for every synthetic workload and write them to the package's
``workload_thresholds.json``.  TEST INFRASTRUCTURE: calls only the CPU oracle and the
seeded input generator; run by hand (``python -m oracle.calibrate``), its output is
committed as data.

The paper tunes its thresholds by hand so that a token budget is approximately met
(Section 4.1, implementation details).  Parity testing additionally needs every
similarity that takes part in a decision to stay clear of its threshold, so a threshold
can only sit in a gap of the similarity distribution.  The rule used here:

* candidate tau_S = midpoints of gaps >= GAP between consecutive sorted parent-child
  similarities (all frames, all levels); candidate tau_T = the same over the temporal
  candidate similarities that the chosen tau_S produces.  Both stages stay switched on:
  only candidates below the largest similarity are considered.
* the tau_S candidates considered are the lowest one whose spatial-only count still
  reaches budget * N, its lower neighbour and the TOP_S distinct spatial-only counts
  above it; for each of them the two tau_T candidates whose output counts bracket
  budget * N.  Pairs whose count is within NEAR * N of budget * N, from either side,
  meet the budget "approximately" as in the paper (its own runs land at 45.5 % / 27.6 %
  for the 50 % / 30 % budgets); among them the pair whose spatial-only fraction is
  nearest sqrt(budget) wins (the paper's stages remove about equal shares, Table 6).
  If no pair is that near, the nearest count wins.
* the workload with fixed thresholds (tiny) keeps them; its seed is bumped until every
  similarity is at least MARGIN away from them.
"""
from __future__ import annotations

import json
import sys
import time

import numpy as np

from paper_2507_07990_b200 import inputs
from oracle import oracle

GAP = 2.2e-4        # minimal width of a gap that may hold a threshold
MARGIN = 1.0e-4     # every decision similarity is at least this far from its threshold
TOP_S = 8
NEAR = 0.03         # a count within this fraction of all tokens of the budget meets it "approximately"


def gap_midpoints(values: np.ndarray, gap: float = GAP):
    s = np.sort(np.asarray(values, dtype=np.float64).ravel())
    d = np.diff(s)
    return [float((s[i] + s[i + 1]) / 2) for i in np.nonzero(d >= gap)[0]]


def margin_of(result: oracle.OracleResult, tau_s: float, tau_t: float) -> float:
    """Smallest distance between a threshold and a similarity the oracle evaluated."""
    m = float(np.min(np.abs(result.spatial_sims - tau_s)))
    if result.tsim is not None and len(result.tsim):
        m = min(m, float(np.min(np.abs(result.tsim - tau_t))))
    return m


def calibrate_video(video: np.ndarray, budget: float, lv1: int = 4, log=print):
    N = video.shape[0] * video.shape[1] * video.shape[2]
    target = budget * N
    base = oracle.merge(video, 2.0, 2.0, lv1=lv1, want_sims=True, want_feats=False)
    s_cands = sorted(gap_midpoints(base.spatial_sims), reverse=True)       # descending tau_S
    if not s_cands:
        raise RuntimeError("no threshold candidates")
    spatial = {}

    def spatial_at(k):
        if k not in spatial:
            spatial[k] = oracle.merge(video, s_cands[k], 2.0, lv1=lv1, want_feats=False, want_pairs=True)
        return spatial[k]

    # The spatial-only count does not grow when tau_S falls.  Temporal merging only removes rows,
    # so a rung is of use when its spatial-only count is at least about the target: find the last
    # such candidate by bisection and walk up from there over TOP_S distinct spatial-only counts.
    lo, hi, last = 0, len(s_cands) - 1, 0
    while lo <= hi:
        mid = (lo + hi) // 2
        if spatial_at(mid).count >= target:
            last, lo = mid, mid + 1
        else:
            hi = mid - 1
    rungs, seen_counts = [], set()
    for k in range(min(last + 1, len(s_cands) - 1), -1, -1):
        r = spatial_at(k)
        if r.count in seen_counts:
            continue
        seen_counts.add(r.count)
        rungs.append((s_cands[k], r))
        if len(rungs) == TOP_S + 1:
            break
    best = None
    for ts, r in rungs:
        if r.tsim is None or len(r.tsim) == 0:
            continue
        # (stay below the largest similarity: the temporal stage stays switched on)
        t_cands = sorted(gap_midpoints(r.tsim))
        if not t_cands:
            continue
        counts = {}

        def count_at(k):
            if k not in counts:
                counts[k] = oracle.merge(video, ts, t_cands[k], lv1=lv1, want_feats=False).count
            return counts[k]

        # the output count does not decrease when tau_T grows: bisect for the largest count that
        # fits, then compare it with its upper neighbour
        lo, hi, fit = 0, len(t_cands) - 1, None
        while lo <= hi:
            mid = (lo + hi) // 2
            if count_at(mid) <= target:
                fit, lo = mid, mid + 1
            else:
                hi = mid - 1
        near = [k for k in ((fit,) if fit is not None else ()) + ((fit + 1,) if fit is not None else (0,))
                if 0 <= k < len(t_cands)]
        for k in near:
            cand = (count_at(k), ts, t_cands[k])
            log("    tau_s %.6f (spatial-only %.4f): tau_t %.6f -> %.4f" % (ts, r.count / N, cand[2], cand[0] / N))
            # Pairs that land within NEAR of the budget (from either side) count as meeting it, and
            # among them the one whose spatial-only fraction is nearest sqrt(budget) wins: the
            # paper's runs at the 30 % budget keep 57-60 % with the spatial stage alone and
            # 54-57 % with the temporal stage alone (Table 6).  Otherwise: the nearest count.
            off = abs(cand[0] - target)
            if off <= NEAR * N:
                key = (0, abs(r.count / N - budget ** 0.5), off)
            else:
                key = (1, off, cand[0] > target)
            if best is None or key < best[0]:
                best = (key, cand)
    if best is None:
        raise RuntimeError("no threshold candidates")
    count, ts, tt = best[1]
    final = oracle.merge(video, ts, tt, lv1=lv1, want_sims=True, want_pairs=True, want_feats=False)
    m = margin_of(final, ts, tt)
    assert final.count == count
    if m < MARGIN:
        raise RuntimeError("margin %.3e below %.1e" % (m, MARGIN))
    return dict(tau_s=ts, tau_t=tt, count=int(count), tokens=int(N), fraction=count / N, margin=m)


def main(argv):
    names = argv[1:] or list(inputs.CONFIGS)
    try:
        table = inputs.load_thresholds()
    except FileNotFoundError:
        table = {}
    for name in names:
        cfg = inputs.CONFIGS[name]
        entry = {"seed_bump": 0, "videos": []}
        t0 = time.time()
        if "fixed_tau" in cfg:
            ts, tt = cfg["fixed_tau"]
            bump = 0
            while True:
                spec = inputs.config_videos(name, bump)[0]
                video = inputs.make_video(spec)
                per_lv1 = {}
                for lv1 in (4, 2):
                    r = oracle.merge(video, ts, tt, lv1=lv1, want_sims=True, want_pairs=True, want_feats=False)
                    per_lv1[lv1] = (r.count, margin_of(r, ts, tt))
                if min(m for _, m in per_lv1.values()) >= MARGIN:
                    break
                bump += 1
            entry["seed_bump"] = bump
            entry["videos"].append({"fixed": dict(tau_s=ts, tau_t=tt, count=per_lv1[4][0],
                                                  count_lv1_2=per_lv1[2][0], tokens=spec.tokens,
                                                  fraction=per_lv1[4][0] / spec.tokens,
                                                  margin=min(m for _, m in per_lv1.values()))})
            print(name, "seed bump", bump, entry["videos"][0])
        else:
            for v, spec in enumerate(inputs.config_videos(name)):
                video = inputs.make_video(spec)
                per_budget = {}
                for b in cfg["budgets"]:
                    print("%s video %d budget %.2f" % (name, v, b))
                    per_budget["%.2f" % b] = calibrate_video(video, b)
                    print("  ->", per_budget["%.2f" % b])
                entry["videos"].append(per_budget)
        entry["seconds"] = round(time.time() - t0, 1)
        table[name] = entry
        with open(inputs.THRESHOLDS_PATH, "w") as f:
            json.dump(table, f, indent=1, sort_keys=True)
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
