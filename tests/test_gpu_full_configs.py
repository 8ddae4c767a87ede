"""Parity at the full sizes of the five workloads, in the launch configuration the
benchmark times (sttm_merge_ex, bf16 output, stored thresholds).  The C oracle is fast
enough to check every output row, so nothing is sampled."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2507_07990_b200 import binding, inputs
from tests import helpers

pytestmark = pytest.mark.gpu


def check_video(spec, th, lv1=4):
    video = inputs.make_video(spec)
    ref = oracle.merge(video, th["tau_s"], th["tau_t"], lv1=lv1, want_sims=True, want_pairs=True)
    margin = min(float(np.abs(ref.spatial_sims - th["tau_s"]).min()), float(np.abs(ref.tsim - th["tau_t"]).min()))
    assert margin >= 1e-4, "stored thresholds lost their margin on this machine: %g" % margin
    assert ref.count == th["count"]
    dev = helpers.to_torch(video)
    for out_dtype in (torch.bfloat16, torch.float32):
        out = binding.sttm_merge_ex(dev, th["tau_s"], th["tau_t"], lv1=lv1, out_dtype=out_dtype)
        torch.cuda.synchronize()
        assert int(out.device_status) == 0
        n = int(out.out_count[0])
        assert n == ref.count
        np.testing.assert_array_equal(out.merge_map[0].cpu().numpy(), ref.merge_map)
        np.testing.assert_array_equal(out.out_pos[:n].cpu().numpy(), ref.out_pos)
        helpers.assert_features_close(out.out_feats[:n].float().cpu().numpy(), ref.out_feats,
                                      out_dtype == torch.bfloat16)
        del out
    return video, ref


@pytest.mark.parametrize("name", ["llava", "qwen", "long"])
def test_single_video_workloads(name):
    table = inputs.load_thresholds()[name]
    spec = inputs.config_videos(name, table["seed_bump"])[0]
    for budget, th in table["videos"][0].items():
        check_video(spec, th)
    torch.cuda.empty_cache()


def test_mixed_batch_workload():
    """Eight videos in one call, per-video thresholds, packed variable-length output."""
    table = inputs.load_thresholds()["mixed"]
    specs = inputs.config_videos("mixed", table["seed_bump"])
    videos = [inputs.make_video(s) for s in specs]
    dev = helpers.to_torch(np.stack(videos))
    for budget in ("0.50", "0.30"):
        ths = [table["videos"][v][budget] for v in range(len(specs))]
        out = binding.sttm_merge_ex(dev, [t["tau_s"] for t in ths], [t["tau_t"] for t in ths],
                                    out_dtype=torch.bfloat16)
        torch.cuda.synchronize()
        assert int(out.device_status) == 0
        offs = out.out_offsets.tolist()
        for v, (video, th) in enumerate(zip(videos, ths)):
            ref = oracle.merge(video, th["tau_s"], th["tau_t"])
            assert ref.count == th["count"] == int(out.out_count[v]) == offs[v + 1] - offs[v]
            np.testing.assert_array_equal(out.merge_map[v].cpu().numpy(), ref.merge_map)
            np.testing.assert_array_equal(out.out_pos[offs[v]:offs[v + 1]].cpu().numpy(), ref.out_pos)
            helpers.assert_features_close(out.out_feats[offs[v]:offs[v + 1]].float().cpu().numpy(),
                                          ref.out_feats, True)
