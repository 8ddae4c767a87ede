"""Shared helpers of the GPU parity tests (threshold choice with a safety margin,
feature comparison).  Thresholds are chosen from the ORACLE's similarities only."""
import numpy as np

from oracle import oracle
from paper_2507_07990_b200 import inputs

MARGIN = 1e-4


def _pick(values, quantile, margin=MARGIN):
    """A threshold near the given quantile of `values` that keeps `margin` distance from
    every value: the midpoint of the gap (wider than 2.2 * margin) nearest to the quantile."""
    s = np.unique(np.asarray(values, dtype=np.float64).ravel())
    if len(s) < 2:
        return 0.5 if len(s) == 0 else float(s[0]) - 0.01
    k = int(np.clip(round(quantile * (len(s) - 1)), 0, len(s) - 2))
    wide = np.nonzero(np.diff(s) >= 2.2 * margin)[0]
    if len(wide) == 0:
        return None
    i = int(wide[np.argmin(np.abs(wide - k))])
    return float((s[i] + s[i + 1]) / 2)


def safe_thresholds(video, q_s, q_t, lv1=4):
    """(tau_s, tau_t) near the requested quantiles of the spatial / temporal similarity
    distributions, each at least MARGIN away from every similarity the oracle evaluates.
    Returns None when no such pair exists for this input."""
    base = oracle.merge(video, 2.0, 2.0, lv1=lv1, want_sims=True, want_feats=False)
    tau_s = _pick(base.spatial_sims, q_s) if base.spatial_sims.size else 0.5
    if tau_s is None:
        return None
    r = oracle.merge(video, tau_s, 2.0, lv1=lv1, want_pairs=True, want_feats=False)
    tau_t = _pick(r.tsim, q_t) if len(r.tsim) else 0.5
    if tau_t is None:
        return None
    return tau_s, tau_t


def to_torch(video_np, device="cuda"):
    """numpy video (uint16 bf16 bits or float32) -> torch tensor on the device."""
    import torch
    if video_np.dtype == np.uint16:
        return torch.from_numpy(video_np.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(video_np).to(device)


def assert_features_close(gpu_rows, oracle_rows, out_is_bf16):
    """fp32 output: max relative error 1e-3, relative to max(|x|, 1e-3 * max|row|).
    bf16 output: the bit pattern is at most one step away from the oracle value rounded to
    bf16 (nearest even): a flush that truncated instead of rounding would not pass."""
    g = np.asarray(gpu_rows, dtype=np.float64)
    o = np.asarray(oracle_rows, dtype=np.float64)
    assert g.shape == o.shape
    if g.size == 0:
        return
    if out_is_bf16:
        def ordered(bits):          # sign-magnitude patterns -> integers in value order
            b = bits.astype(np.int32)
            return np.where(b & 0x8000, -(b & 0x7FFF), b)
        gb = ordered(inputs.f32_to_bf16_bits(g.astype(np.float32)))
        ob = ordered(inputs.f32_to_bf16_bits(o.astype(np.float32)))
        assert np.array_equal(inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(g.astype(np.float32))).astype(np.float64), g), \
            "bf16 rows expected"
        bad = np.abs(gb - ob) > 1
    else:
        scale = np.maximum(np.abs(o), 1e-3 * np.abs(o).max(axis=1, keepdims=True))
        bad = np.abs(g - o) > 1e-3 * scale + 1e-30
    assert not bad.any(), "feature mismatch at %s" % (np.argwhere(bad)[:5].tolist(),)


def small_spec(seed, T, H, W, D, dtype="bf16", depth_max=3, p_static=0.7, sigma=0.05):
    return inputs.VideoSpec(T=T, H=H, W=W, D=D, dtype=dtype, depth_max=depth_max, p_static=p_static,
                            sigma=sigma, seed=seed)
