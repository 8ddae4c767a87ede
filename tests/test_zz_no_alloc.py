"""The entry point that allocates nothing (sttm_spatial_static), against sttm_spatial.

Some callers of this library cannot hand it a workspace: all of their device memory belongs to
a pool they do not control, or they sit in a loop where an allocation (and the device-wide
synchronisation it may bring) is not acceptable.  For them the spatial stage also exists with
its scratch in a fixed array inside the library.  This file checks, through the C ABI, that the
variant gives exactly what sttm_spatial gives - on two calls in a row, because every call
reuses the same array and must not depend on what the previous one left there - and that a
problem too large for the array is refused instead of run.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2507_07990_b200 import binding, inputs
from tests import helpers

pytestmark = pytest.mark.gpu


def _spatial_both_ways(video_np, tau_s, lv1=4):
    dev = helpers.to_torch(video_np)
    T, H, W, D = video_np.shape
    cover_ref, counts_ref, sims_ref, _ = binding.sttm_spatial(dev, tau_s, lv1=lv1, want_sims=True)
    cover = torch.full((1, T, H, W), -1, dtype=torch.int8, device="cuda")
    counts = torch.full((1, T), -1, dtype=torch.int32, device="cuda")
    sims = torch.full_like(sims_ref, float("nan"))
    binding.sttm_spatial_static(dev, tau_s, cover, counts, sims, lv1=lv1)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(cover.cpu().numpy(), cover_ref.cpu().numpy())
    np.testing.assert_array_equal(counts.cpu().numpy(), counts_ref.cpu().numpy())
    # same kernel, same inputs: the similarities agree far inside the 2e-5 the parity tests allow
    np.testing.assert_allclose(sims.cpu().numpy(), sims_ref.cpu().numpy(), rtol=0, atol=2e-5, equal_nan=True)
    return counts_ref


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # two different problems back to back: the second one finds the first one's norms in the array
    first = inputs.make_video(helpers.small_spec(41, 7, 13, 13, 256))
    second = inputs.make_video(helpers.small_spec(42, 5, 16, 16, 128, p_static=0.4))
    a = _spatial_both_ways(first, 0.97)
    b = _spatial_both_ways(second, 0.5)
    assert int(a.sum()) > 0 and int(b.sum()) > 0
    # and the first problem again, now after a larger one
    _spatial_both_ways(first, 0.97)


def test_static_entry_point_allocates_nothing():
    # the array's address is known by now (first call done above or here); from then on the free
    # device memory must not move across a call: no cudaMalloc, no growing cache behind the scenes
    video = inputs.make_video(helpers.small_spec(44, 6, 13, 13, 256))
    dev = helpers.to_torch(video)
    T, H, W, D = video.shape
    cover = torch.empty((1, T, H, W), dtype=torch.int8, device="cuda")
    counts = torch.empty((1, T), dtype=torch.int32, device="cuda")
    binding.sttm_spatial_static(dev, 0.9, cover, counts)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    binding.sttm_spatial_static(dev, 0.9, cover, counts)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_static_scratch_fp32_and_two_level_grid():
    video = inputs.make_video(helpers.small_spec(43, 4, 8, 8, 64, dtype="f32", sigma=0.3))
    _spatial_both_ways(video, 0.9)
    _spatial_both_ways(video, 0.9, lv1=2)


def test_problem_beyond_the_fixed_scratch_is_refused():
    # 16x16 grid, three levels: 16 columns x 21 nodes x 4 bytes per frame; 4 MiB hold 3120 frames
    T = 4000
    feats = torch.empty((1, T, 16, 16, 8), dtype=torch.bfloat16, device="cuda")
    cover = torch.empty((1, T, 16, 16), dtype=torch.int8, device="cuda")
    counts = torch.empty((1, T), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SttmError) as e:
        binding.sttm_spatial_static(feats, 0.9, cover, counts)
    assert e.value.code == 3
    # exactly at the limit: 3120 frames are accepted
    T = 3120
    binding.sttm_spatial_static(feats[:, :T], 0.9, cover[:, :T], counts[:, :T])
    torch.cuda.synchronize()
    assert int(counts[0, :T].min()) >= 16
