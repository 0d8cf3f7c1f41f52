"""Shared helpers of the test-suite: hand-made scenes and the acceptance rule."""
from __future__ import annotations

import numpy as np

from scenes import custom_scene, make_rig, NOMINAL_DIMS, MOUNT


def single_env(tris, classes, agents, rig=None, H=64, W=64, near=0.5, far=100.0, active=None, tri_vis_cos=None, agent_classes=None):
    """agents: list of (x, y, yaw, length, width, height)."""
    agents = np.asarray(agents, dtype=np.float64).reshape(-1, 6)
    poses = agents[None, :, :3]
    dims = agents[None, :, 3:]
    if rig is None:
        rig = make_rig((0.0,), 90.0, 90.0, W, H)
    tris = np.asarray(tris, dtype=np.float32).reshape(-1, 3, 3)
    return custom_scene(tris, classes, poses, dims, rig, H, W, near, far,
                        active=None if active is None else np.asarray(active, np.uint8).reshape(1, -1),
                        tri_vis_cos=tri_vis_cos, agent_classes=agent_classes)


def f16_ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """|a-b| in units in the last place for positive finite binary16 arrays."""
    return np.abs(a.view(np.uint16).astype(np.int32) - b.view(np.uint16).astype(np.int32))


def compare_images(ref_cls, ref_depth, ref_flag, got_cls, got_depth32=None, got_depth16=None,
                   depth_rtol=1e-4, max_mismatch_frac=1e-4, ref_kappa=None):
    """The acceptance rule.  A pixel *mismatches* when its class differs from the reference or its
    float32 depth differs by more than the depth tolerance: depth_rtol relative, widened to
    5e-7 * kappa where the reference reports that the winning primitive's plane grazes the camera
    centre (kappa > 200: depth is ill-conditioned in float32 there).  Every mismatch must sit on a
    pixel the reference flagged as ambiguous (edge, depth gap, clip plane, horizon), and mismatches
    must stay below max_mismatch_frac of the pixels (at least one pixel is always allowed so that
    tiny images are not held to zero).  Off the mismatching pixels the stored binary16 depth must be
    within one unit in the last place of the correctly rounded reference depth (or within the
    widened tolerance).  Returns a dict of statistics; raises AssertionError."""
    ref_cls = np.asarray(ref_cls); got_cls = np.asarray(got_cls)
    n = ref_cls.size
    tol = np.full(ref_cls.shape, depth_rtol, np.float64)
    if ref_kappa is not None:
        tol = np.maximum(tol, 5e-7 * np.asarray(ref_kappa))
    bad = ref_cls != got_cls
    if got_depth32 is not None:
        bad |= np.abs(np.asarray(got_depth32, np.float64) - ref_depth) > tol * ref_depth
    flagged = (np.asarray(ref_flag) & 47) != 0
    unflagged_bad = bad & ~flagged
    stats = dict(pixels=int(n), mismatches=int(bad.sum()), flagged=int(flagged.sum()),
                 unflagged_mismatches=int(unflagged_bad.sum()))
    assert stats["unflagged_mismatches"] == 0, f"mismatch on unflagged pixels: {stats}, first at " \
        f"{np.argwhere(unflagged_bad)[:5].tolist()}"
    allowed = max(1, int(np.floor(max_mismatch_frac * n)))
    assert stats["mismatches"] <= allowed, f"too many mismatches: {stats}"
    if got_depth16 is not None:
        ref16 = ref_depth.astype(np.float16)
        got16 = np.asarray(got_depth16).view(np.float16)
        ulp = f16_ulp_distance(got16, ref16)
        close = np.abs(got16.astype(np.float64) - ref_depth) <= (tol + 2.0 ** -11) * ref_depth
        off = (ulp > 1) & ~close & ~bad
        stats["f16_one_ulp"] = int(((ulp == 1) & ~bad).sum())
        assert not off.any(), f"binary16 depth off by more than 1 ulp at {np.argwhere(off)[:5].tolist()}"
    return stats


def assert_same_as_exhaustive(prod, brute, sl=slice(None)):
    """Production kernel vs exhaustive kernel: classes identical; float32 depths identical up to a
    few float32 ulps (the exhaustive kernel also draws the box faces turned away from the camera,
    which meet the facing ones along silhouette edges at the same depth up to rounding)."""
    assert (prod[0][sl] == brute[0][sl]).all(), "classes differ between the production and the exhaustive kernel"
    a, b = prod[2][sl].astype(np.float64), brute[2][sl].astype(np.float64)
    assert (np.abs(a - b) <= 5e-7 * b).all(), "depths differ between the production and the exhaustive kernel"


def random_scene(seed: int, full_tiles: bool = False):
    """A seeded random scene for fuzzing: triangle soups far from the origin with planar quad pairs
    and a degenerate triangle, random rigs (mounts, yaw, pitch up to 0.5 rad, unequal focal lengths),
    random image sizes incl. ragged ones (`full_tiles`: multiples of 64 only, the sizes that take the
    kernels' full-tile instantiations), random near/far, inactive agents."""
    car = (4.5, 1.9, 1.5)
    rng = np.random.default_rng(seed)
    H = int(rng.choice([16, 36, 54, 64, 70, 128])); W = int(rng.choice([16, 48, 64, 96, 100, 160]))
    if full_tiles:
        H = 64 * (1 + seed % 2); W = 64 * (1 + (seed // 2) % 3)
    K = int(rng.integers(1, 5)); A = int(rng.integers(1, 7)); E = int(rng.integers(1, 3))
    n = int(rng.integers(0, 150))
    scale = float(rng.choice([3.0, 10.0, 40.0]))
    origin = rng.uniform(-2000, 2000, size=2)
    centre = rng.uniform(-scale, scale, size=(n, 1, 3)) * np.array([1, 1, 0.15]) + np.array([origin[0], origin[1], 0.5])
    tris = centre + rng.uniform(-scale / 3, scale / 3, size=(n, 3, 3)) * np.array([1, 1, 0.4])
    classes = rng.integers(2, 9, size=n)
    if n > 10:   # planar quads given as triangle pairs of one class, and one degenerate triangle
        for i in range(0, min(n - 1, 40), 2):
            p = rng.uniform(-scale, scale, size=(4, 3)) * np.array([1, 1, 0.0]) + np.array([origin[0], origin[1], rng.uniform(0, 0.5)])
            c = p.mean(0); ang = np.arctan2(p[:, 1] - c[1], p[:, 0] - c[0]); p = p[np.argsort(ang)]
            tris[i] = p[[0, 1, 2]]; tris[i + 1] = p[[0, 2, 3]]
            classes[i + 1] = classes[i]
        tris[-1, 2] = tris[-1, 1]
    poses = np.zeros((E, A, 3))
    poses[..., 0] = origin[0] + rng.uniform(-scale, scale, (E, A)); poses[..., 1] = origin[1] + rng.uniform(-scale, scale, (E, A))
    poses[..., 2] = rng.uniform(-3.2, 3.2, (E, A))
    dims = np.tile(np.array(car), (E, A, 1)) * rng.uniform(0.5, 2.0, (E, A, 3))
    rig = np.zeros((K, 7), np.float32)
    for k in range(K):
        rig[k] = (rng.uniform(-2, 3), rng.uniform(-1, 1), rng.uniform(0.3, 3.0), rng.uniform(-3.2, 3.2), rng.uniform(-0.5, 0.5),
                  W / 2 / np.tan(np.radians(rng.uniform(30, 120)) / 2), H / 2 / np.tan(np.radians(rng.uniform(30, 110)) / 2))
    near = float(rng.choice([0.1, 0.5, 1.0])); far = float(rng.choice([20.0, 100.0, 300.0]))
    active = (rng.uniform(size=(E, A)) > 0.15).astype(np.uint8)
    return custom_scene(tris, classes, poses, dims, rig, H, W, near, far, active=active, name=f"fuzz{seed}")
