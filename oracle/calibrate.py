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
* among the TOP_S highest tau_S candidates that give distinct spatial-only counts, and
  for each of them all tau_T candidates, take the pair whose output count is the
  largest that does not exceed budget * N; if no pair fits the budget, the pair with
  the smallest count.
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
TOP_S = 4


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
    s_cands = sorted(gap_midpoints(base.spatial_sims), reverse=True)
    rungs, seen_counts = [], set()
    for ts in s_cands:
        r = oracle.merge(video, ts, 2.0, lv1=lv1, want_feats=False, want_pairs=True)
        if r.count in seen_counts:
            continue
        seen_counts.add(r.count)
        rungs.append((ts, r))
        if len(rungs) == TOP_S:
            break
    best = None
    for ts, r in rungs:
        t_cands = sorted(gap_midpoints(r.tsim))
        # the output count does not decrease when tau_T grows: bisect for the largest fit
        lo, hi, fit = 0, len(t_cands) - 1, None
        counts = {}

        def count_at(k):
            if k not in counts:
                counts[k] = oracle.merge(video, ts, t_cands[k], lv1=lv1, want_feats=False).count
            return counts[k]

        while lo <= hi:
            mid = (lo + hi) // 2
            if count_at(mid) <= target:
                fit, lo = mid, mid + 1
            else:
                hi = mid - 1
        if fit is None and t_cands:
            fit = 0
        if fit is None:
            continue
        cand = (count_at(fit), ts, t_cands[fit])
        log("    tau_s %.6f (spatial-only %.4f): tau_t %.6f -> %.4f" % (ts, r.count / N, cand[2], cand[0] / N))
        fits = cand[0] <= target
        if best is None:
            best = cand
        else:
            best_fits = best[0] <= target
            if (fits and not best_fits) or (fits and best_fits and cand[0] > best[0]) \
                    or (not fits and not best_fits and cand[0] < best[0]):
                best = cand
    if best is None:
        raise RuntimeError("no threshold candidates")
    count, ts, tt = best
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
