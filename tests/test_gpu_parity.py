"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  Structure (cover map, links, roots, merge map, position ids,
counts) must match bit for bit; merged features within the tolerance in helpers."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2507_07990_b200 import binding, inputs
from tests import helpers

pytestmark = pytest.mark.gpu

# (path, cluster size, frames per item) for sttm_set_tuning, then (sum slots, lead frames) for
# sttm_set_ring_split: the library's own choice (the two-stream kernels), the same with item
# borders every frame / every three / every seven frames, the three-pass kernels, single-pass
# launches that force clusters and many item borders, the two-stream kernels with either Gram stage, the single-pass kernel without packing of
# partial border tiles, and two other ways to share out its shared-memory slots
TUNINGS = {"auto": (0, 0, 0, 0, 0), "flowf1": (5, 0, 1, 0, 0), "flowf3": (5, 0, 3, 0, 0), "flowf7": (5, 0, 7, 0, 0),
           "gramsyncf3": (6, 0, 3, 0, 0), "gramsyncf6": (6, 0, 6, 0, 0),
           "threepass": (1, 0, 0, 0, 0), "c1f3": (2, 1, 3, 0, 0), "c2f2": (2, 2, 2, 0, 0),
           "c4f5": (2, 4, 5, 0, 0), "c8f1": (2, 8, 1, 0, 0), "nopack": (3, 0, 0, 0, 0), "sum2lead2": (2, 0, 0, 2, 2),
           "sum4": (2, 0, 7, 4, 1)}


@pytest.fixture(params=list(TUNINGS), ids=list(TUNINGS))
def tuning(request):
    lib = binding.load_library()
    lib.sttm_set_tuning(*TUNINGS[request.param][:3])
    lib.sttm_set_ring_split(*TUNINGS[request.param][3:])
    yield request.param
    lib.sttm_set_tuning(0, 0, 0)
    lib.sttm_set_ring_split(0, 0)


def run_and_compare(video_np, tau_s, tau_t, lv1=4, out_dtype=torch.float32, wt=binding.W_NODE,
                    pos=binding.POS_SURVIVED, stages=True, match=binding.MATCH_TOPLEFT):
    T, H, W, D = video_np.shape
    N = T * H * W
    ref = oracle.merge(video_np, tau_s, tau_t, lv1=lv1, weight_mode=wt, pos_mode=pos, match_mode=match,
                       want_sims=True, want_pairs=True)
    dev = helpers.to_torch(video_np)
    out = binding.sttm_merge_ex(dev, tau_s, tau_t, lv1=lv1, out_dtype=out_dtype, wt=wt, pos=pos, match=match)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    count = int(out.out_count[0].item())
    assert count == ref.count
    assert out.out_offsets.tolist() == [0, ref.count]
    np.testing.assert_array_equal(out.merge_map[0].cpu().numpy(), ref.merge_map)
    np.testing.assert_array_equal(out.out_pos[:count].cpu().numpy(), ref.out_pos)
    helpers.assert_features_close(out.out_feats[:count].float().cpu().numpy(), ref.out_feats,
                                  out_dtype == torch.bfloat16)
    if stages:
        cover, counts, sims, ws = binding.sttm_spatial(dev, tau_s, lv1=lv1, want_sims=True)
        link, root, tsim, status = binding.sttm_temporal(dev, cover, tau_s, tau_t, ws, lv1=lv1, want_sims=True,
                                                         match=match)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        np.testing.assert_array_equal(cover[0].cpu().numpy(), ref.cover_level)
        np.testing.assert_array_equal(link[0].cpu().numpy(), ref.link)
        np.testing.assert_array_equal(root[0].cpu().numpy(), ref.root)
        per_frame = []
        for t in range(T):
            n = 0
            for (y, x), l in np.ndenumerate(ref.cover_level[t]):
                m = (1 << int(l)) - 1
                n += int((y & m) == 0 and (x & m) == 0)      # anchors of kept nodes
            per_frame.append(n)
        assert counts[0].cpu().tolist() == per_frame
        if ref.spatial_sims.size:
            np.testing.assert_allclose(sims[0].cpu().numpy(), ref.spatial_sims, rtol=0, atol=2e-5)
        ts = tsim[0].cpu().numpy()
        got = {}
        for v in np.nonzero(~np.isnan(ts))[0]:
            got[int(v)] = float(ts[v])
        assert len(got) == len(ref.tsim)
        HW = H * W
        for v, u, s in zip(ref.tsim_v, ref.tsim_u, ref.tsim):
            # a pair is stored at the anchor of its finer node, in frame t's numbering
            key = int(v) if ref.cover_level.ravel()[v] <= ref.cover_level.ravel()[u] else int(u) + HW
            assert abs(got[key] - s) < 2e-5
    return ref


SHAPES = [  # T, H, W, D, lv1, dtype
    (4, 8, 8, 64, 4, "f32"),
    (4, 8, 8, 64, 2, "f32"),
    (6, 13, 13, 256, 4, "bf16"),
    (5, 16, 16, 384, 4, "bf16"),
    (3, 14, 14, 128, 4, "bf16"),
    (4, 4, 4, 128, 4, "bf16"),       # single level: temporal only
    (3, 7, 5, 132, 4, "bf16"),       # ragged channel tail, non-square
    (9, 3, 3, 64, 2, "f32"),
    (2, 1, 1, 8, 4, "f32"),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "T%dH%dW%dD%dlv%d%s" % s)
@pytest.mark.parametrize("q_s,q_t", [(0.5, 0.5), (0.15, 0.8), (0.9, 0.2)])
def test_parity_small(shape, q_s, q_t, tuning):
    T, H, W, D, lv1, dtype = shape
    done = 0
    for seed in range(3):
        spec = helpers.small_spec(100 + seed, T, H, W, D, dtype=dtype, sigma=0.3 if D < 200 else 0.05)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, q_s, q_t, lv1)
        if taus is None:
            continue
        for out_dtype in (torch.float32, torch.bfloat16):
            run_and_compare(video, taus[0], taus[1], lv1=lv1, out_dtype=out_dtype)
        done += 1
    assert done >= 1, "no seed gave thresholds with a margin"


def test_parity_weight_and_position_modes(tuning):
    spec = helpers.small_spec(7, 6, 13, 13, 256)
    video = inputs.make_video(spec)
    tau_s, tau_t = helpers.safe_thresholds(video, 0.4, 0.5)
    run_and_compare(video, tau_s, tau_t, wt=binding.W_AREA, stages=False)
    run_and_compare(video, tau_s, tau_t, pos=binding.POS_REASSIGNED, stages=False)


def test_degenerate_thresholds(tuning):
    spec = helpers.small_spec(8, 12, 13, 13, 128)
    video = inputs.make_video(spec)
    for tau_s, tau_t in [(2.0, 2.0), (-2.0, 2.0), (2.0, -2.0), (-2.0, -2.0)]:
        ref = run_and_compare(video, tau_s, tau_t)
    assert ref.count == 16          # everything merges: the 4x4 coarsest map of frame 0


def test_tiny_config_fixed_thresholds():
    entry = inputs.load_thresholds()["tiny"]
    spec = inputs.config_videos("tiny", entry["seed_bump"])[0]
    video = inputs.make_video(spec)
    fixed = entry["videos"][0]["fixed"]
    for lv1, expect in ((4, fixed["count"]), (2, fixed["count_lv1_2"])):
        ref = run_and_compare(video, fixed["tau_s"], fixed["tau_t"], lv1=lv1)
        assert ref.count == expect


def test_long_chains_cross_time_chunks(tuning):
    """A static video: every chain spans all frames, so rows are summed across the
    averaging kernel's time chunks."""
    spec = helpers.small_spec(9, 96, 13, 13, 128, p_static=0.97)
    video = inputs.make_video(spec)
    taus = helpers.safe_thresholds(video, 0.5, 0.3)
    assert taus is not None
    ref = run_and_compare(video, taus[0], taus[1], stages=False)
    assert ref.out_members.max() >= 40


def test_batch_with_per_video_thresholds(tuning):
    specs = [helpers.small_spec(20 + v, 8, 13, 13, 256, p_static=p) for v, p in enumerate((0.9, 0.5, 0.2))]
    videos = [inputs.make_video(s) for s in specs]
    taus = [helpers.safe_thresholds(v, 0.5, 0.5) for v in videos]
    assert all(t is not None for t in taus)
    dev = helpers.to_torch(np.stack(videos))
    out = binding.sttm_merge_ex(dev, [t[0] for t in taus], [t[1] for t in taus], out_dtype=torch.float32)
    torch.cuda.synchronize()
    offs = out.out_offsets.tolist()
    for b, (video, (ts, tt)) in enumerate(zip(videos, taus)):
        ref = oracle.merge(video, ts, tt)
        assert int(out.out_count[b]) == ref.count and offs[b + 1] - offs[b] == ref.count
        np.testing.assert_array_equal(out.merge_map[b].cpu().numpy(), ref.merge_map)
        np.testing.assert_array_equal(out.out_pos[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_pos)
        helpers.assert_features_close(out.out_feats[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_feats, False)


def test_capacity_overflow_is_reported_not_fatal():
    spec = helpers.small_spec(30, 4, 8, 8, 64, dtype="f32", sigma=0.3)
    video = inputs.make_video(spec)
    ref = oracle.merge(video, 2.0, 2.0)
    dev = helpers.to_torch(video)
    out = binding.sttm_merge_ex(dev, 2.0, 2.0, out_dtype=torch.float32, capacity=100)
    torch.cuda.synchronize()
    assert int(out.out_count[0]) == ref.count == 256
    assert int(out.device_status.item()) & (1 << 4)
    helpers.assert_features_close(out.out_feats[:100].cpu().numpy(), ref.out_feats[:100], False)


def test_host_buffer_entry_point_and_simple_merge():
    spec = helpers.small_spec(31, 6, 13, 13, 256)
    video = inputs.make_video(spec)
    tau_s, tau_t = helpers.safe_thresholds(video, 0.5, 0.5)
    ref = oracle.merge(video, tau_s, tau_t)
    h = torch.from_numpy(video.view(np.int16)).view(torch.bfloat16).pin_memory()
    out = binding.sttm_merge_host(h, tau_s, tau_t, want_map=True)
    assert int(out.out_count[0]) == ref.count
    np.testing.assert_array_equal(out.merge_map[0].numpy(), ref.merge_map)
    np.testing.assert_array_equal(out.out_pos[:ref.count].numpy(), ref.out_pos)
    helpers.assert_features_close(out.out_feats[:ref.count].float().numpy(), ref.out_feats, True)
    feats, pos, cnt = binding.sttm_merge(h.cuda(), tau_s, tau_t)
    torch.cuda.synchronize()
    assert int(cnt) == ref.count
    np.testing.assert_array_equal(pos[:ref.count].cpu().numpy(), ref.out_pos)
    helpers.assert_features_close(feats[:ref.count].float().cpu().numpy(), ref.out_feats, True)


def test_bad_arguments_are_rejected_on_the_host():
    dev = torch.zeros((1, 2, 4, 4, 6), dtype=torch.bfloat16, device="cuda")     # D not a multiple of 4
    with pytest.raises(binding.SttmError) as e:
        binding.sttm_merge_ex(dev, 0.5, 0.5)
    assert e.value.code == 1
    dev = torch.zeros((1, 1, 600, 4, 8), dtype=torch.bfloat16, device="cuda")   # 600 -> ... -> 3: nine levels
    with pytest.raises(binding.SttmError) as e:
        binding.sttm_merge_ex(dev, 0.5, 0.5)
    assert e.value.code == 2
    dev = torch.zeros((1, 2, 13, 13, 8), dtype=torch.bfloat16, device="cuda")   # 13 -> 7 -> 4 -> 2: four levels
    for call in (lambda: binding.sttm_spatial(dev, 0.5, lv1=2),
                 lambda: binding.sttm_merge_budget(dev, 0.5, [10], lv1=2)):
        with pytest.raises(binding.SttmError) as e:                             # stage calls and budget mode
            call()                                                              # stop at three levels
        assert e.value.code == 2
    prob = binding.make_params((1, 2, 13, 13, 8), torch.bfloat16, 0.5, 0.5)
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    lib = binding.load_library()
    import ctypes as C
    code = lib.sttm_merge_ex(C.c_void_p(dev.data_ptr()), C.byref(prob.params), C.c_void_p(ws.data_ptr()), 1024,
                             C.c_void_p(dev.data_ptr()), C.c_void_p(dev.data_ptr()), None,
                             C.c_void_p(dev.data_ptr()), None, None, None)
    assert code == 3


# Shapes of the paper's other set-ups at their real feature widths: the 14x14 grid of
# LLaVA-Video (Section 3.2), a non-square dynamic-resolution grid (three levels: grids up to 16 cells a side), and D = 8192 of the 72B
# model (eight CTAs per cluster, eight sum warps per CTA).
@pytest.mark.parametrize("path", [1, 3], ids=["singlepass", "twostream"])
@pytest.mark.parametrize("shape", [(6, 14, 14, 3584), (4, 16, 12, 3584), (5, 13, 13, 8192), (3, 16, 16, 8192),
                                   (5, 9, 5, 3584), (4, 13, 5, 1024)],
                         ids=lambda s: "T%dH%dW%dD%d" % s)
def test_other_workload_shapes_full_width(shape, path):
    # (9x5 and 13x5: grids one cell higher and wider than a multiple of four, whose last row and
    # column the two-stream kernels load as strips of 16 cells)
    T, H, W, D = shape
    lib = binding.load_library()
    done = 0
    for seed in range(3):
        spec = helpers.small_spec(300 + seed, T, H, W, D, sigma=0.05)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, 0.5, 0.5)
        if taus is None:
            continue
        lib.sttm_set_tuning(5 if path == 3 else 0, 0, 2 if path == 3 else 0)
        try:
            for out_dtype in (torch.float32, torch.bfloat16):
                run_and_compare(video, taus[0], taus[1], out_dtype=out_dtype)
            assert lib.sttm_last_path() == path
        finally:
            lib.sttm_set_tuning(0, 0, 0)
        done += 1
        break
    assert done >= 1, "no seed gave thresholds with a margin"


@pytest.mark.parametrize("path", [1, 3], ids=["singlepass", "twostream"])
def test_many_frames_take_the_separate_count_scan(path):
    """More than 4096 frames in a call: the per-frame root counts are scanned by a kernel of their
    own instead of inside the row kernel; two videos, so that the video offsets are in play."""
    lib = binding.load_library()
    T, H, W, D = 2100, 5, 5, 256
    videos, taus, refs = [], [], []
    for v in range(2):
        for seed in range(4):
            spec = helpers.small_spec(930 + 10 * v + seed, T, H, W, D, sigma=0.05, p_static=0.8)
            video = inputs.make_video(spec)
            t = helpers.safe_thresholds(video, 0.5, 0.5)
            if t is not None:
                break
        assert t is not None, "no seed gave thresholds with a margin"
        videos.append(video); taus.append(t); refs.append(oracle.merge(video, t[0], t[1]))
    dev = helpers.to_torch(np.stack(videos))
    lib.sttm_set_tuning(5 if path == 3 else 0, 0, 0)
    try:
        out = binding.sttm_merge_ex(dev, [t[0] for t in taus], [t[1] for t in taus], out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert lib.sttm_last_path() == path
    finally:
        lib.sttm_set_tuning(0, 0, 0)
    assert int(out.device_status.item()) == 0
    offs = out.out_offsets.tolist()
    for b, ref in enumerate(refs):
        assert int(out.out_count[b]) == ref.count and offs[b + 1] - offs[b] == ref.count
        np.testing.assert_array_equal(out.merge_map[b].cpu().numpy(), ref.merge_map)
        np.testing.assert_array_equal(out.out_pos[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_pos)
        helpers.assert_features_close(out.out_feats[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_feats, False)


# Channel counts that give the tensor-memory Gram stage other copy widths and copy counts per slice
# (D / 64 = 3, 7, 15, 64 blocks: copies of 3, 7, 5 and 4 blocks), on grids with clipped tiles and strips,
# runs of frames that are not a multiple of four, both Gram stages of the two-stream kernels.
@pytest.mark.parametrize("gram", [5, 6], ids=["tensormemory", "mmasync"])
@pytest.mark.parametrize("case", [(5, 13, 9, 192, 3), (9, 7, 5, 448, 2), (7, 16, 13, 960, 5), (6, 5, 12, 4096, 0),
                                  (13, 4, 4, 320, 8), (2, 14, 3, 1024, 1)],
                         ids=lambda c: "T%dH%dW%dD%df%d" % c)
def test_two_stream_other_widths(case, gram):
    T, H, W, D, F = case
    lib = binding.load_library()
    for seed in range(4):
        spec = helpers.small_spec(7100 + 7 * seed + T, T, H, W, D, sigma=0.05, p_static=0.8)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, 0.5, 0.5)
        if taus is not None:
            break
    assert taus is not None, "no seed gave thresholds with a margin"
    lib.sttm_set_tuning(gram, 0, F)
    try:
        run_and_compare(video, taus[0], taus[1], out_dtype=torch.float32, stages=False)
        run_and_compare(video, taus[0], taus[1], out_dtype=torch.bfloat16, stages=False, wt=binding.W_AREA)
        assert lib.sttm_last_path() == 3 and lib.sttm_last_gram_stage() == (2 if gram == 5 else 1)
    finally:
        lib.sttm_set_tuning(0, 0, 0)


def test_most_similar_destination(tuning):
    """Section 3.3's other destination rule: among the overlapping nodes above tau_t the most
    similar one instead of the top-left one.  Both sides pick a maximum, so the inputs are
    chosen such that the two best candidates of every node are at least 1e-4 apart."""
    assert binding.MATCH_BEST == oracle.MATCH_BEST
    checked = differs = 0
    for shape in [(6, 13, 13, 256), (5, 16, 16, 384), (4, 8, 8, 64)]:
        T, H, W, D = shape
        for seed in range(4):
            spec = helpers.small_spec(400 + seed, T, H, W, D, dtype="f32" if D == 64 else "bf16",
                                      sigma=0.3 if D < 200 else 0.05, p_static=0.5)
            video = inputs.make_video(spec)
            taus = helpers.safe_thresholds(video, 0.6, 0.15)
            if taus is None:
                continue
            ref = oracle.merge(video, taus[0], taus[1], match_mode=oracle.MATCH_BEST, want_pairs=True, want_feats=False)
            above = {}
            for v, sim in zip(ref.tsim_v.tolist(), ref.tsim.tolist()):
                if sim > taus[1]:
                    above.setdefault(v, []).append(sim)
            gaps = [sorted(c)[-1] - sorted(c)[-2] for c in above.values() if len(c) > 1]
            if gaps and min(gaps) < 1e-4:
                continue
            topleft = oracle.merge(video, taus[0], taus[1], want_feats=False)
            differs += int((topleft.link != ref.link).sum())
            run_and_compare(video, taus[0], taus[1], match=binding.MATCH_BEST)
            run_and_compare(video, taus[0], taus[1], out_dtype=torch.bfloat16, stages=False, match=binding.MATCH_BEST)
            checked += 1
            break
    assert checked >= 2, "no input with a margin between the best candidates"
    assert differs > 0, "the rule never chose another destination than the top-left one"


def test_merged_positions():
    """The "merged" position output (Section 3.4) from the library's own merge map, bit for bit
    against the oracle's definition; a batch of two videos, and the capacity condition."""
    specs = [helpers.small_spec(500 + v, 6, 13, 13, 256, p_static=p) for v, p in enumerate((0.9, 0.4))]
    videos, taus = [], []
    for spec in specs:
        video = inputs.make_video(spec)
        t = helpers.safe_thresholds(video, 0.5, 0.5)
        assert t is not None
        videos.append(video)
        taus.append(t)
    dev = helpers.to_torch(np.stack(videos))
    out = binding.sttm_merge_ex(dev, [t[0] for t in taus], [t[1] for t in taus], out_dtype=torch.bfloat16)
    rows = int(out.out_offsets[-1].item())
    pos, status = binding.sttm_merged_positions(out.merge_map, out.out_offsets, rows)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    offs = out.out_offsets.tolist()
    got = pos.cpu().numpy()
    for v, (video, t) in enumerate(zip(videos, taus)):
        ref = oracle.merge(video, t[0], t[1], want_feats=False)
        np.testing.assert_array_equal(out.merge_map[v].cpu().numpy(), ref.merge_map)
        np.testing.assert_array_equal(got[offs[v]:offs[v + 1]], oracle.merged_positions(ref.merge_map, ref.count))
    short, status = binding.sttm_merged_positions(out.merge_map, out.out_offsets, rows - 5)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << 4                      # capacity exceeded, reported, not fatal
    np.testing.assert_array_equal(short.cpu().numpy()[:offs[1] - 5], got[:offs[1] - 5])


def test_budget_mode():
    """tau_t chosen on the device for a row budget: the threshold agrees with the oracle's rule, the
    count meets the budget exactly (budgets picked where the best cosines leave a clear gap at the
    cut), and the whole output equals the oracle's at the returned threshold."""
    checked = 0
    for seed, shape in [(700, (8, 13, 13, 256)), (701, (6, 16, 16, 384)), (702, (10, 13, 13, 256))]:
        T, H, W, D = shape
        spec = helpers.small_spec(seed, T, H, W, D, p_static=0.6)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, 0.5, 0.5)
        if taus is None:
            continue
        tau_s = taus[0]
        nodes, m = oracle.best_candidate_cosines(video, tau_s)
        gaps = m[:-1] - m[1:]                                   # gap below the k-th largest, k = index + 1
        ks = [int(k) + 1 for k in np.argsort(-gaps)[:12] if gaps[k] >= 2e-4][:4]
        dev = helpers.to_torch(video)
        for k in ks:
            budget = nodes - k
            tau_ref, gap = oracle.budget_tau_t(video, tau_s, budget)
            assert gap >= 2e-4
            out, tau = binding.sttm_merge_budget(dev, tau_s, [budget], out_dtype=torch.float32)
            torch.cuda.synchronize()
            assert int(out.device_status.item()) == 0
            tau_gpu = float(tau[0].item())
            assert abs(tau_gpu - tau_ref) < 1e-5
            count = int(out.out_count[0].item())
            assert count == budget
            ref = oracle.merge(video, tau_s, tau_gpu)
            assert ref.count == count
            np.testing.assert_array_equal(out.merge_map[0].cpu().numpy(), ref.merge_map)
            np.testing.assert_array_equal(out.out_pos[:count].cpu().numpy(), ref.out_pos)
            helpers.assert_features_close(out.out_feats[:count].float().cpu().numpy(), ref.out_feats, False)
            checked += 1
    assert checked >= 6, "too few budgets with a clear gap at the cut"
    # a budget that needs no temporal merging, and one that cannot be met
    out, tau = binding.sttm_merge_budget(dev, tau_s, [10 ** 9])
    torch.cuda.synchronize()
    assert float(tau[0].item()) == 2.0 and int(out.out_count[0].item()) == nodes
    out, tau = binding.sttm_merge_budget(dev, tau_s, [1])
    torch.cuda.synchronize()
    assert float(tau[0].item()) == -2.0
    assert int(out.out_count[0].item()) == oracle.merge(video, tau_s, -2.0, want_feats=False).count


# Quadtrees of four and five levels (the 2x2 coarsest map of the paper's ablation on its real grids,
# and grids of more than 16 cells a side): the general kernels behind sttm_merge_ex.
@pytest.mark.parametrize("shape", [(4, 13, 13, 64, 2, "f32"), (5, 14, 14, 128, 2, "bf16"), (3, 16, 16, 256, 2, "bf16"),
                                   (3, 18, 12, 256, 4, "bf16"), (3, 20, 20, 64, 2, "f32"), (2, 24, 33, 132, 4, "bf16"),
                                   (6, 24, 24, 3584, 4, "bf16")],
                         ids=lambda s: "T%dH%dW%dD%dlv%d%s" % s)
def test_deeper_quadtrees(shape):
    T, H, W, D, lv1, dtype = shape
    done = 0
    for seed in range(4):
        spec = helpers.small_spec(800 + seed, T, H, W, D, dtype=dtype, sigma=0.3 if D < 200 else 0.05, depth_max=4)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, 0.5, 0.5, lv1)
        if taus is None:
            continue
        ref = oracle.merge(video, taus[0], taus[1], lv1=lv1, want_feats=False)
        assert int(ref.cover_level.max()) <= 4
        for out_dtype, wt, pos, match in [(torch.float32, binding.W_NODE, binding.POS_SURVIVED, binding.MATCH_TOPLEFT),
                                          (torch.bfloat16, binding.W_AREA, binding.POS_REASSIGNED, binding.MATCH_TOPLEFT),
                                          (torch.float32, binding.W_NODE, binding.POS_SURVIVED, binding.MATCH_BEST)]:
            run_and_compare(video, taus[0], taus[1], lv1=lv1, out_dtype=out_dtype, wt=wt, pos=pos, stages=False,
                            match=match)
        done += 1
        if done == 2:
            break
    assert done >= 1, "no seed gave thresholds with a margin"


def test_deeper_quadtrees_features_do_not_depend_on_scheduling():
    """The general kernels add a row's members in index order: two runs give the same bits."""
    spec = helpers.small_spec(871, 24, 13, 13, 256, dtype="bf16", sigma=0.05, depth_max=4, p_static=0.9)
    dev = helpers.to_torch(inputs.make_video(spec)[None])
    outs = []
    for _ in range(3):
        out = binding.sttm_merge_ex(dev, 0.6, 0.6, lv1=2, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert int(out.device_status.item()) == 0 and binding.load_library().sttm_last_path() == 2
        n = int(out.out_count[0])
        outs.append(out.out_feats[:n].clone())
    assert n < spec.tokens                       # something was merged
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_deeper_quadtrees_batch_capacity_and_host_entry():
    specs = [helpers.small_spec(840 + v, 5, 18, 20, 64, dtype="bf16", sigma=0.3, depth_max=4, p_static=p)
             for v, p in enumerate((0.9, 0.4))]
    videos = [inputs.make_video(s) for s in specs]
    taus = [helpers.safe_thresholds(v, 0.5, 0.5, 4) for v in videos]
    assert all(t is not None for t in taus)
    refs = [oracle.merge(v, ts, tt) for v, (ts, tt) in zip(videos, taus)]
    dev = helpers.to_torch(np.stack(videos))
    out = binding.sttm_merge_ex(dev, [t[0] for t in taus], [t[1] for t in taus], out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) == 0
    assert binding.load_library().sttm_last_path() == 2
    offs = out.out_offsets.tolist()
    for b, ref in enumerate(refs):
        assert int(out.out_count[b]) == ref.count and offs[b + 1] - offs[b] == ref.count
        np.testing.assert_array_equal(out.merge_map[b].cpu().numpy(), ref.merge_map)
        np.testing.assert_array_equal(out.out_pos[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_pos)
        helpers.assert_features_close(out.out_feats[offs[b]:offs[b + 1]].cpu().numpy(), ref.out_feats, False)
    # fewer rows than the result: the rows that fit are right, the rest is reported
    cap = refs[0].count + refs[1].count // 2
    out = binding.sttm_merge_ex(dev, [t[0] for t in taus], [t[1] for t in taus], out_dtype=torch.float32, capacity=cap)
    torch.cuda.synchronize()
    assert int(out.device_status.item()) & (1 << 4)
    assert [int(c) for c in out.out_count] == [r.count for r in refs]
    both = np.concatenate([r.out_feats for r in refs])
    helpers.assert_features_close(out.out_feats[:cap].cpu().numpy(), both[:cap], False)
    # host buffers in, host buffers out
    h = torch.from_numpy(videos[0].view(np.int16)).view(torch.bfloat16).pin_memory()
    res = binding.sttm_merge_host(h, taus[0][0], taus[0][1], want_map=True)
    assert int(res.out_count[0]) == refs[0].count
    np.testing.assert_array_equal(res.merge_map[0].numpy(), refs[0].merge_map)
    helpers.assert_features_close(res.out_feats[:refs[0].count].float().numpy(), refs[0].out_feats, True)
