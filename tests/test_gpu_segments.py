"""One video cut into segments of consecutive frames, the ranks emulated one after the other on
one GPU: the packed result must be the oracle's result for the whole video."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2507_07990_b200 import binding, inputs, segments
from tests import helpers

pytestmark = pytest.mark.gpu


def run_segments(video_np, world, tau_s, tau_t, lv1=4, out_dtype=torch.float32, wt=binding.W_NODE,
                 pos=binding.POS_SURVIVED, match=binding.MATCH_TOPLEFT):
    T = video_np.shape[0]
    dev = helpers.to_torch(video_np)
    cuts = segments.cut_frames(T, world)
    shared = segments.LocalLink(world)
    parts = []
    for r in range(world):
        halo = 1 if r > 0 else 0
        local = dev[cuts[r] - halo:cuts[r + 1]].contiguous()
        parts.append(segments.SegmentMerge(local, bool(halo), cuts[r], tau_s, tau_t, lv1, out_dtype, pos, wt, match))
        shared.counts[r] = parts[-1].merge_local()
    outs = [None] * world
    for r in reversed(range(world)):
        outs[r] = parts[r].finish(shared.for_rank(r))
    torch.cuda.synchronize()
    assert not shared.box, "a message was left unread"
    feats = torch.cat([o.out_feats[:o.owned_count] for o in outs]).float().cpu().numpy()
    ids = torch.cat([o.out_pos[:o.owned_count] for o in outs]).cpu().numpy()
    for r, o in enumerate(outs):
        assert int(o.device_status.item()) == 0
        assert o.rows_before == sum(x.owned_count for x in outs[:r])
    return feats, ids


@pytest.mark.parametrize("case", [(7, 13, 13, 256, "bf16", 4, 2), (7, 13, 13, 256, "bf16", 4, 4), (9, 8, 8, 64, "f32", 4, 3),
                                  (12, 16, 12, 3584, "bf16", 4, 3), (6, 14, 14, 128, "bf16", 2, 3)],
                         ids=lambda c: "T%dH%dW%dD%d%slv%dx%d" % c)
def test_segments_reproduce_the_whole_video(case):
    T, H, W, D, dtype, lv1, world = case
    done = 0
    for seed in range(4):
        spec = helpers.small_spec(900 + seed, T, H, W, D, dtype=dtype, p_static=0.85, sigma=0.3 if D < 200 else 0.05)
        video = inputs.make_video(spec)
        taus = helpers.safe_thresholds(video, 0.5, 0.5, lv1)
        if taus is None:
            continue
        for out_dtype, wt, pos, match in [(torch.float32, binding.W_NODE, binding.POS_SURVIVED, binding.MATCH_TOPLEFT),
                                          (torch.bfloat16, binding.W_AREA, binding.POS_REASSIGNED, binding.MATCH_BEST)]:
            ref = oracle.merge(video, taus[0], taus[1], lv1=lv1, weight_mode=wt, pos_mode=pos, match_mode=match)
            feats, ids = run_segments(video, world, taus[0], taus[1], lv1, out_dtype, wt, pos, match)
            assert feats.shape[0] == ref.count
            np.testing.assert_array_equal(ids, ref.out_pos)
            helpers.assert_features_close(feats, ref.out_feats, out_dtype == torch.bfloat16)
        if done == 0:
            # the cuts must matter: some chain crosses every cut, one crosses at least two
            cuts = segments.cut_frames(T, world)
            frame_of = lambda a: a // (H * W)
            first = np.array([frame_of(a) for a in ref_roots(ref)])
            last = ref_last_frames(ref, H * W)
            for c in cuts[1:-1]:
                assert np.any((first < c) & (last >= c))
            if world > 2:
                assert np.any((first < cuts[1]) & (last >= cuts[2]))
        done += 1
        if done == 2:
            break
    assert done >= 1, "no seed gave thresholds with a margin"


def ref_roots(ref):
    """Anchor id of every row's root, whatever id mode the run used."""
    first = np.full(ref.count, -1, dtype=np.int64)
    for cell, row in enumerate(ref.merge_map):
        if first[row] < 0:
            first[row] = cell
    return first


def ref_last_frames(ref, HW):
    last = np.zeros(ref.count, dtype=np.int64)
    for cell, row in enumerate(ref.merge_map):
        last[row] = max(last[row], cell // HW)
    return last


def test_single_rank_is_the_plain_merge():
    spec = helpers.small_spec(950, 5, 13, 13, 256)
    video = inputs.make_video(spec)
    taus = helpers.safe_thresholds(video, 0.5, 0.5)
    assert taus is not None
    ref = oracle.merge(video, taus[0], taus[1])
    feats, ids = run_segments(video, 1, taus[0], taus[1])
    np.testing.assert_array_equal(ids, ref.out_pos)
    helpers.assert_features_close(feats, ref.out_feats, False)
