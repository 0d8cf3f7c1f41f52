"""Shared helpers of the test-suite: hand-made scenes and the acceptance rule."""
from __future__ import annotations

import numpy as np

from scenes import custom_scene, make_rig, NOMINAL_DIMS, MOUNT


def single_env(tris, classes, agents, rig=None, H=64, W=64, near=0.5, far=100.0, active=None):
    """agents: list of (x, y, yaw, length, width, height)."""
    agents = np.asarray(agents, dtype=np.float64).reshape(-1, 6)
    poses = agents[None, :, :3]
    dims = agents[None, :, 3:]
    if rig is None:
        rig = make_rig((0.0,), 90.0, 90.0, W, H)
    tris = np.asarray(tris, dtype=np.float32).reshape(-1, 3, 3)
    return custom_scene(tris, classes, poses, dims, rig, H, W, near, far,
                        active=None if active is None else np.asarray(active, np.uint8).reshape(1, -1))


def f16_ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """|a-b| in units in the last place for positive finite binary16 arrays."""
    return np.abs(a.view(np.uint16).astype(np.int32) - b.view(np.uint16).astype(np.int32))


def compare_images(ref_cls, ref_depth, ref_flag, got_cls, got_depth32=None, got_depth16=None,
                   depth_rtol=1e-4, max_mismatch_frac=1e-4):
    """The acceptance rule.  A pixel *mismatches* when its class differs from the reference or its
    float32 depth differs by more than depth_rtol relative.  Every mismatch must sit on a pixel the
    reference flagged as ambiguous, and mismatches must stay below max_mismatch_frac of the pixels
    (at least one pixel is always allowed so that tiny images are not held to zero).  Off the
    mismatching pixels the stored binary16 depth must be within one unit in the last place of
    the correctly rounded reference depth.  Returns a dict of statistics; raises AssertionError."""
    ref_cls = np.asarray(ref_cls); got_cls = np.asarray(got_cls)
    n = ref_cls.size
    bad = ref_cls != got_cls
    if got_depth32 is not None:
        bad |= np.abs(np.asarray(got_depth32, np.float64) - ref_depth) > depth_rtol * ref_depth
    flagged = np.asarray(ref_flag) != 0
    unflagged_bad = bad & ~flagged
    stats = dict(pixels=int(n), mismatches=int(bad.sum()), flagged=int(flagged.sum()),
                 unflagged_mismatches=int(unflagged_bad.sum()))
    assert stats["unflagged_mismatches"] == 0, f"mismatch on unflagged pixels: {stats}, first at " \
        f"{np.argwhere(unflagged_bad)[:5].tolist()}"
    allowed = max(1, int(np.floor(max_mismatch_frac * n)))
    assert stats["mismatches"] <= allowed, f"too many mismatches: {stats}"
    if got_depth16 is not None:
        ref16 = ref_depth.astype(np.float16)
        ulp = f16_ulp_distance(np.asarray(got_depth16).view(np.float16), ref16)
        ulp = np.where(bad, 0, ulp)
        stats["f16_one_ulp"] = int((ulp == 1).sum())
        assert ulp.max() <= 1, f"binary16 depth off by more than 1 ulp at {np.argwhere(ulp > 1)[:5].tolist()}"
    return stats
