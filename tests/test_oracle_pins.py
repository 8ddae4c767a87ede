"""Pins of the CPU oracle against things other than itself: hand-worked closed forms,
an independently written brute force, library average pooling, special cases with a
textbook answer, the paper's comparison counts, and invariants of the method."""
import dataclasses
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2507_07990_b200 import inputs
from tests import helpers
from tests.bruteforce import sttm_bruteforce, level_sizes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quad_2x2.json")
OFF = 2.0   # a threshold no cosine can exceed: the stage never merges


def small_video(seed, T, H, W, D=8, K=4, sigma=0.3, p_static=0.6, depth_max=3):
    spec = inputs.VideoSpec(T=T, H=H, W=W, D=D, dtype="f32", depth_max=depth_max, p_static=p_static,
                            sigma=sigma, K=K, scale_unit_rms=False, seed=seed)
    return inputs.make_video(spec).astype(np.float64)


# ---------------------------------------------------------------- level sizes (Section 3.2)
@pytest.mark.parametrize("H,W,lv1,expect", [
    (13, 13, 4, [(13, 13), (7, 7), (4, 4)]),
    (14, 14, 4, [(14, 14), (7, 7), (4, 4)]),
    (14, 14, 2, [(14, 14), (7, 7), (4, 4), (2, 2)]),
    (16, 16, 4, [(16, 16), (8, 8), (4, 4)]),
    (8, 8, 4, [(8, 8), (4, 4)]),
    (8, 8, 2, [(8, 8), (4, 4), (2, 2)]),
    (4, 4, 4, [(4, 4)]),
    (5, 9, 4, [(5, 9), (3, 5), (2, 3)]),
])
def test_levels(H, W, lv1, expect):
    assert oracle.levels(H, W, lv1) == expect


# ---------------------------------------------------------------- hand-worked closed forms
def _golden_cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", _golden_cases(), ids=lambda c: c["name"])
def test_hand_worked_examples(case):
    video = np.array(case["frames"], dtype=np.float64)
    T, H, W, D = video.shape
    assert (H, W, D) == (2, 2, 2)
    # the closed forms in the fixture are what the formulas say
    for key in ("child_parent_cos", "temporal_cos"):
        if key in case:
            for formula, value in zip(case[key]["formula"], case[key]["value"]):
                assert math.isclose(eval(formula, {"sqrt": math.sqrt}), value, rel_tol=1e-15)
    if "child_parent_cos" in case:
        r = oracle.merge(video, 0.0, OFF, lv1=1, want_sims=True)
        np.testing.assert_allclose(r.spatial_sims[0], case["child_parent_cos"]["value"], rtol=1e-14)
    for run in case["runs"]:
        w = {"node": oracle.W_NODE, "area": oracle.W_AREA}[run.get("weight", "node")]
        m = {"topleft": oracle.MATCH_TOPLEFT, "best": oracle.MATCH_BEST,
             "topleft_only": oracle.MATCH_TOPLEFT_ONLY}[run.get("match", "topleft")]
        r = oracle.merge(video, run["tau_s"], run["tau_t"], lv1=1, weight_mode=w, match_mode=m,
                         want_pairs=True)
        assert r.count == run["count"]
        assert r.out_pos.tolist() == run["out_pos"]
        assert r.merge_map.tolist() == run["merge_map"]
        assert r.cover_level.ravel().tolist() == run["cover"]
        if "link" in run:
            assert r.link.tolist() == run["link"]
            assert r.root.tolist() == run["root"]
            assert r.out_members.tolist() == run["members"]
        np.testing.assert_allclose(r.out_feats, np.array(run["out_feats"], dtype=np.float64), rtol=1e-14, atol=1e-15)
        if "temporal_cos" in case and run.get("match", "topleft") != "topleft_only":
            np.testing.assert_allclose(sorted(r.tsim), sorted(case["temporal_cos"]["value"]), rtol=1e-13)


# ---------------------------------------------------------------- brute force on tiny inputs
SHAPES = [(1, 2, 2, 1), (2, 3, 3, 2), (3, 4, 4, 2), (3, 3, 4, 2), (2, 5, 5, 2), (3, 5, 3, 4),
          (2, 8, 8, 4), (2, 7, 6, 2), (3, 4, 4, 4), (2, 6, 9, 4), (2, 13, 13, 4)]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "T%dH%dW%dlv%d" % s)
@pytest.mark.parametrize("weight,match", [("node", "topleft"), ("area", "best"), ("node", "topleft_only")])
def test_against_brute_force(shape, weight, match):
    T, H, W, lv1 = shape
    rng = np.random.default_rng(1000 * H + 10 * W + T)
    n_mixed = 0
    for trial in range(4 if H * W > 100 else 8):
        video = small_video(7 * trial + H * 31 + W, T, H, W, D=6, sigma=float(rng.uniform(0.1, 0.5)))
        tau_s, tau_t = float(rng.uniform(0.55, 0.97)), float(rng.uniform(0.3, 0.97))
        bf = sttm_bruteforce(video, tau_s, tau_t, lv1, weight, match)
        r = oracle.merge(video, tau_s, tau_t, lv1=lv1,
                         weight_mode={"node": oracle.W_NODE, "area": oracle.W_AREA}[weight],
                         match_mode={"topleft": oracle.MATCH_TOPLEFT, "best": oracle.MATCH_BEST,
                                     "topleft_only": oracle.MATCH_TOPLEFT_ONLY}[match])
        assert r.count == bf["count"]
        np.testing.assert_array_equal(r.cover_level, bf["cover"])
        np.testing.assert_array_equal(r.link, bf["link"])
        np.testing.assert_array_equal(r.root, bf["root"])
        np.testing.assert_array_equal(r.merge_map, bf["merge_map"])
        np.testing.assert_array_equal(r.out_pos, bf["out_pos"])
        np.testing.assert_array_equal(r.out_members, bf["members"])
        np.testing.assert_allclose(r.out_feats, bf["out_feats"], rtol=1e-12, atol=1e-13)
        assert r.comparisons_spatial == bf["cmp_spatial"]
        assert r.comparisons_temporal == bf["cmp_temporal"]
        if 1 < r.count < T * H * W:
            n_mixed += 1
    assert n_mixed >= 1 or H * W <= 4, "test inputs never produced a partial merge"


# ---------------------------------------------------------------- special cases with a library / textbook answer
@pytest.mark.parametrize("H,W,lv1", [(13, 13, 4), (14, 14, 2), (3, 3, 1), (5, 7, 2), (16, 16, 4), (8, 8, 4)])
def test_everything_passes_equals_average_pooling(H, W, lv1):
    """tau_S below every cosine: each frame collapses to its coarsest map, which is 2x2
    average pooling (ceil mode, border windows divided by the cells they really hold)
    applied level by level."""
    T, D = 2, 5
    video = small_video(3, T, H, W, D=D)
    r = oracle.merge(video, -OFF, OFF, lv1=lv1)
    x = torch.from_numpy(video).permute(0, 3, 1, 2)          # [T, D, H, W]
    sizes = level_sizes(H, W, lv1)
    for _ in range(len(sizes) - 1):
        x = torch.nn.functional.avg_pool2d(x, 2, 2, ceil_mode=True, count_include_pad=False)
    hc, wc = sizes[-1]
    assert tuple(x.shape[2:]) == (hc, wc)
    expect = x.permute(0, 2, 3, 1).reshape(T * hc * wc, D).numpy()
    assert r.count == T * hc * wc
    np.testing.assert_allclose(r.out_feats, expect, rtol=1e-13, atol=1e-14)
    side = 1 << (len(sizes) - 1)
    pos = [t * H * W + i * side * W + j * side for t in range(T) for i in range(hc) for j in range(wc)]
    assert r.out_pos.tolist() == pos
    assert (r.cover_level == len(sizes) - 1).all()


def test_identity_when_nothing_merges():
    video = small_video(5, 3, 5, 6)
    r = oracle.merge(video, OFF, OFF)
    N = video.shape[0] * 30
    assert r.count == N
    assert r.out_pos.tolist() == list(range(N)) and r.merge_map.tolist() == list(range(N))
    np.testing.assert_array_equal(r.out_feats, video.reshape(N, -1))
    assert (r.link == -1).all() and (r.cover_level == 0).all()


def test_cellwise_chain_is_mean_over_time():
    """No spatial merging, every temporal comparison passes: each cell links to the
    same cell of the previous frame, so a video collapses to the per-cell mean over t."""
    video = small_video(6, 5, 4, 6)
    r = oracle.merge(video, OFF, -OFF)
    assert r.count == 24
    np.testing.assert_allclose(r.out_feats, video.mean(axis=0).reshape(24, -1), rtol=1e-13)
    assert r.out_pos.tolist() == list(range(24))
    assert (r.out_members == 5).all()
    assert r.comparisons_temporal == 4 * 24          # (T-1)*H*W, Section 3.3
    assert r.root.tolist() == list(range(24)) * 5


def test_temporal_off_is_concatenation_of_frames():
    video = small_video(8, 4, 8, 8, sigma=0.2)
    tau_s = 0.8
    whole = oracle.merge(video, tau_s, OFF)
    rows, pos = [], []
    for t in range(4):
        one = oracle.merge(video[t:t + 1], tau_s, OFF)
        rows.append(one.out_feats)
        pos += [int(p) + t * 64 for p in one.out_pos]
    assert whole.count == sum(len(r) for r in rows)
    np.testing.assert_array_equal(whole.out_feats, np.concatenate(rows))
    assert whole.out_pos.tolist() == pos
    assert 4 * 16 < whole.count < 4 * 64, "choose tau_s so that the spatial stage merges partially"


def test_identical_frames_collapse_to_frame_zero():
    frame = small_video(9, 1, 13, 13, sigma=0.2)
    video = np.repeat(frame, 6, axis=0)
    for tau_s in (0.7, 0.85, OFF):
        first = oracle.merge(frame, tau_s, OFF)
        r = oracle.merge(video, tau_s, 0.999)
        assert r.count == first.count
        np.testing.assert_array_equal(r.out_pos, first.out_pos)
        np.testing.assert_allclose(r.out_feats, first.out_feats, rtol=1e-14)
        assert (r.out_members == 6).all()
        assert (r.root.reshape(6, -1) == r.root[:169]).all()


def test_position_id_modes():
    video = small_video(10, 3, 8, 8, sigma=0.2)
    a = oracle.merge(video, 0.8, 0.8, pos_mode=oracle.POS_SURVIVED)
    b = oracle.merge(video, 0.8, 0.8, pos_mode=oracle.POS_REASSIGNED)
    assert a.count == b.count and b.out_pos.tolist() == list(range(b.count))
    assert (np.diff(a.out_pos) > 0).all(), "survived ids follow (t, y, x) order"
    # a survived id is the original index of the root's top-left cell
    for row, p in enumerate(a.out_pos):
        assert a.merge_map[p] == row and a.root[p] == p


# ---------------------------------------------------------------- comparison counts (Eq. 1-2, Section 3.3)
@pytest.mark.parametrize("H,W,lv1", [(8, 8, 2), (16, 16, 4), (16, 16, 2), (4, 4, 2), (13, 13, 4), (14, 14, 2)])
def test_worst_case_spatial_comparisons(H, W, lv1):
    video = small_video(11, 2, H, W, D=4)
    r = oracle.merge(video, OFF, OFF, lv1=lv1, want_feats=False)
    sizes = level_sizes(H, W, lv1)
    assert r.comparisons_spatial == 2 * sum(h * w for h, w in sizes[:-1])
    if H == W and H & (H - 1) == 0:
        levels = len(sizes) - 1
        assert r.comparisons_spatial == 2 * sum(H * W // 4 ** i * 4 for i in range(1, levels + 1))   # Eq. 1
        assert r.comparisons_spatial <= 2 * 4 * H * W / 3                                            # Eq. 2
    # the best case touches only the coarsest nodes' children
    r = oracle.merge(video, -OFF, OFF, lv1=lv1, want_feats=False)
    assert r.comparisons_spatial == 2 * sizes[-2][0] * sizes[-2][1]


# ---------------------------------------------------------------- invariants on the block generator
def _check_structure(video, r, tau_t):
    T, H, W, D = video.shape
    HW = H * W
    cover = r.cover_level
    anchors = {}
    for t in range(T):
        covered = np.zeros((H, W), dtype=int)
        for y in range(H):
            for x in range(W):
                l = int(cover[t, y, x]); s = 1 << l
                y0, x0 = y - y % s, x - x % s
                assert (cover[t, y0:min(y0 + s, H), x0:min(x0 + s, W)] == l).all(), "kept regions are whole nodes"
                anchors[t * HW + y0 * W + x0] = (t, y0, min(y0 + s, H), x0, min(x0 + s, W))
                covered[y, x] += 1
        assert (covered == 1).all()
    members = {}
    for a, (t, y0, y1, x0, x1) in anchors.items():
        lk, rt = int(r.link[a]), int(r.root[a])
        if lk >= 0:
            assert lk in anchors and anchors[lk][0] == t - 1, "links go to a kept node of the previous frame"
            _, a0, a1, b0, b1 = anchors[lk]
            assert a0 < y1 and y0 < a1 and b0 < x1 and x0 < b1, "linked nodes overlap"
            assert r.root[lk] == rt
        else:
            assert rt == a
        assert rt // HW <= t and r.link[rt] == -1
        members.setdefault(rt, []).append(a)
    roots = sorted(members)
    assert r.count == len(roots) and r.out_pos.tolist() == roots
    assert sorted(set(r.merge_map.tolist())) == list(range(r.count)), "every row is used, every cell has a row"
    for row, rt in enumerate(roots):
        assert r.out_members[row] == len(members[rt])
        assert (r.merge_map[r.root == rt] == row).all()
    return anchors, members


def test_invariants_tiny_config():
    spec = inputs.config_videos("tiny")[0]
    video = inputs.make_video(spec)
    for lv1 in (4, 2):
        r = oracle.merge(video, 0.9, 0.9, lv1=lv1)
        anchors, members = _check_structure(video, r, 0.9)
        # area weights on a power-of-two grid: a row is the plain mean of its input tokens
        ra = oracle.merge(video, 0.9, 0.9, lv1=lv1, weight_mode=oracle.W_AREA)
        flat = video.reshape(-1, video.shape[-1]).astype(np.float64)
        for row in range(ra.count):
            np.testing.assert_allclose(ra.out_feats[row], flat[ra.merge_map == row].mean(axis=0), rtol=1e-12)


def test_invariants_and_monotonicity_blocks():
    spec = dataclasses.replace(inputs.config_videos("llava")[0], T=12, D=32, dtype="f32", sigma=0.25)
    video = inputs.make_video(spec)
    taus = [0.5, 0.8, 0.9, 0.95, 0.98, 0.995]
    prev_spatial = None
    for tau_s in taus:
        r = oracle.merge(video, tau_s, OFF, want_feats=False)
        per_frame = np.array([len(set(r.root[t * 169:(t + 1) * 169].tolist())) for t in range(spec.T)])
        if prev_spatial is not None:
            assert (per_frame >= prev_spatial).all(), "spatial count per frame grows with tau_S"
        prev_spatial = per_frame
    prev = None
    for tau_t in taus:
        r = oracle.merge(video, 0.9, tau_t)
        _check_structure(video, r, tau_t)
        if prev is not None:
            assert r.count >= prev, "total count grows with tau_T at fixed tau_S"
        prev = r.count


def test_zero_vectors_have_zero_similarity():
    video = np.zeros((2, 2, 2, 3))
    r = oracle.merge(video, 0.5, 0.5, lv1=1, want_sims=True, want_pairs=True)
    assert (r.spatial_sims == 0).all() and (r.tsim == 0).all() and r.count == 8


def test_generator_margins_match_the_stored_thresholds():
    """The stored thresholds keep every decision similarity at least 1e-4 away (tiny)."""
    table = inputs.load_thresholds()
    entry = table["tiny"]
    spec = inputs.config_videos("tiny", entry["seed_bump"])[0]
    video = inputs.make_video(spec)
    fixed = entry["videos"][0]["fixed"]
    r = oracle.merge(video, fixed["tau_s"], fixed["tau_t"], want_sims=True, want_pairs=True)
    assert r.count == fixed["count"]
    m = min(np.abs(r.spatial_sims - fixed["tau_s"]).min(), np.abs(r.tsim - fixed["tau_t"]).min())
    assert m >= 1e-4


def test_merged_positions_closed_forms():
    """Section 3.4, merged strategy: mean member index per row.  Hand values, the identity when
    nothing merges, and the arithmetic-series mean when everything merges into one row."""
    got = oracle.merged_positions(np.array([0, 0, 1, 2, 2, 2, 1]), 3)
    assert got.dtype == np.float32
    np.testing.assert_array_equal(got, np.array([0.5, 4.0, 4.0], dtype=np.float32))      # (0+1)/2, (2+6)/2, (3+4+5)/3
    np.testing.assert_array_equal(oracle.merged_positions(np.arange(37), 37), np.arange(37, dtype=np.float32))
    n = 1001
    np.testing.assert_array_equal(oracle.merged_positions(np.zeros(n, dtype=np.int32), 1),
                                  np.array([(n - 1) / 2.0], dtype=np.float32))
    # against the merge itself: with tau >= 1 nothing merges, so the mean is the survived id
    video = np.random.default_rng(5).standard_normal((3, 4, 4, 8)).astype(np.float32)
    ref = oracle.merge(video, 2.0, 2.0, want_feats=False)
    np.testing.assert_array_equal(oracle.merged_positions(ref.merge_map, ref.count), ref.out_pos.astype(np.float32))


def test_budget_threshold_properties():
    """Budget mode on the oracle: at the returned tau_t the row count is exactly the budget whenever
    the gap at the cut is positive; a budget the spatial stage already meets needs no temporal
    merging; an unreachable one links everything that has a candidate."""
    spec = helpers.small_spec(600, 8, 13, 13, 64, dtype="f32", sigma=0.3, p_static=0.6)
    video = inputs.make_video(spec)
    base = oracle.merge(video, 0.9, 2.0, want_feats=False)
    everything = oracle.merge(video, 0.9, -2.0, want_feats=False)
    checked = 0
    for frac in (0.95, 0.9, 0.8, 0.7, 0.6, 0.5):
        budget = int(base.count * frac)
        if budget < everything.count:
            continue
        tau, gap = oracle.budget_tau_t(video, 0.9, budget)
        if gap > 0:
            assert oracle.merge(video, 0.9, tau, want_feats=False).count == budget
            checked += 1
    assert checked >= 3
    assert oracle.budget_tau_t(video, 0.9, base.count) == (2.0, float("inf"))
    assert oracle.budget_tau_t(video, 0.9, base.count + 7)[0] == 2.0
    assert oracle.budget_tau_t(video, 0.9, 1)[0] == -2.0
    # one frame: no candidates at all
    assert oracle.budget_tau_t(video[:1], 0.9, 1)[0] == -2.0
