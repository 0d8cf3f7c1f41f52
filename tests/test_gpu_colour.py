"""The colour output (RGB, optionally antialiased by analytic coverage) through the C ABI against the oracle."""
import numpy as np
import pytest

from scenes import make_config, make_rig, make_paper_workload, custom_scene, default_palette, disk_triangles
from tests.util import single_env

pytestmark = pytest.mark.gpu
CAR = (4.5, 1.9, 1.5)
PAL = default_palette()


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


def compare_colour(ref, got, tol=1, max_mismatch_frac=2e-3, max_flag_frac=2e-2):
    """Acceptance rule for colour images: a pixel mismatches if a channel differs from the oracle's rounded colour by
    more than `tol` levels (one level: the two sides round the same real number); every mismatch must sit on a pixel
    the oracle flagged as ambiguous, and mismatches stay below max_mismatch_frac of the pixels (one always allowed)."""
    diff = np.abs(ref.rgb.astype(np.int32) - got.astype(np.int32)).max(axis=-1)
    mism = diff > tol
    flagged = (ref.flag & 47) != 0
    bad = mism & ~flagged
    n = mism.size
    assert not bad.any(), f"{bad.sum()} colour mismatches on unflagged pixels; first at {np.argwhere(bad)[:5].tolist()}, " \
                          f"oracle {ref.rgb[bad][:3].tolist()} got {got[bad][:3].tolist()}"
    assert mism.sum() <= max(1, int(max_mismatch_frac * n)), f"{mism.sum()} mismatches of {n} pixels"
    assert flagged.mean() <= max_flag_frac
    return dict(pixels=n, mismatches=int(mism.sum()), flagged=int(flagged.sum()), max_diff_unflagged=int(diff[~flagged].max()))


def check_colour(gu, scene, views=None, palette=PAL, modes=(False, True), **kw):
    import oracle
    g = gu.CudaRun(scene)
    try:
        V = scene.E * scene.A * scene.K
        views = np.arange(V) if views is None else np.asarray(views, np.int64)
        out = {}
        for aa in modes:
            got, status = g.render_rgb(palette, aa)
            assert status == 0, f"status {status} with antialias={aa}"
            ref = oracle.render_rgb(scene, palette, aa, views)
            out[aa] = compare_colour(ref, got[views], **kw)
            out[aa]["changed"] = float((np.abs(ref.rgbf - oracle.render_rgb(scene, palette, False, views).rgbf).max(-1) > 0.5).mean()) if aa else 0.0
        return out
    finally:
        g.close()


def ego(x=0.0, y=0.0, yaw=0.0, dims=CAR):
    return (x, y, yaw) + tuple(dims)


def wall(x, col0, col1, row0, row1, scale=1.0, centre=4.0):
    y0, y1 = (centre - col0) * scale, (centre - col1) * scale
    z0, z1 = 1.0 + (centre - row0) * scale, 1.0 + (centre - row1) * scale
    return [[(x, y0, z0), (x, y1, z0), (x, y1, z1)], [(x, y0, z0), (x, y1, z1), (x, y0, z1)]]


def test_hand_made_scenes(gu):
    rig8 = make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0))
    pole = wall(2.0, 3.1, 3.3, 0.0, 8.0, scale=0.5)
    back = wall(4.0, 3.3, 7.0, 0.0, 8.0)
    xs, ys = np.linspace(1.45, 6.55, 4), np.linspace(1.7, 5.9, 4)
    mesh = [t for i in range(3) for j in range(3) for t in wall(4.0, xs[i], xs[i + 1], ys[j], ys[j + 1])]
    for tris, classes in ((wall(4.0, 2.3, 5.75, 1.5, 6.25), [7, 7]), (wall(4.0, 3.1, 3.3, 0.0, 8.0), [6, 6]),
                          (pole + back, [6, 6, 7, 7]), (pole + back, [7, 7, 7, 7]), (mesh, [7] * 18)):
        st = check_colour(gu, single_env(tris, classes, [ego()], rig=rig8, H=8, W=8), tol=1, max_mismatch_frac=0.1, max_flag_frac=0.2)
        assert st[True]["max_diff_unflagged"] <= 1
    # a box turned by 40 degrees in front of a wall; box faces at near and far
    rig = make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, 1.5))
    big = [[(30.0, 40.0, -10.0), (30.0, -40.0, -10.0), (30.0, -40.0, 30.0)], [(30.0, 40.0, -10.0), (30.0, -40.0, 30.0), (30.0, 40.0, 30.0)]]
    check_colour(gu, single_env(big, [7, 7], [ego(), (12.0, 0.3, np.deg2rad(40.0), 4.5, 1.9, 3.0)], rig=rig))
    check_colour(gu, single_env(np.zeros((0, 3, 3)), [], [ego(), (12.5, 0.0, 0.0, 4.5, 1.9, 1.0)], rig=make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, 4.0))))


def test_config0_all_views(gu):
    st = check_colour(gu, make_config(0))
    print("cfg0 colour:", st)
    assert st[True]["changed"] > 0.02      # antialiasing does change the image


def test_config2_sampled_views_and_classes(gu):
    base = make_config(2, E=2)
    rng = np.random.default_rng(11)
    agent_classes = rng.choice([4, 7, 8], size=(base.E, base.A), p=[0.7, 0.15, 0.15]).astype(np.uint8)
    s = custom_scene(base.tri_xyz, base.tri_class, base.poses, base.dims, base.rig, base.H, base.W, base.near, base.far,
                     map_tri_offset=base.map_tri_offset, env_map_id=base.env_map_id, agent_classes=agent_classes)
    st = check_colour(gu, s, views=np.arange(0, s.E * s.A * s.K, 5))
    print("cfg2 colour:", st)


def test_paper_rig_96x54_and_ragged_sizes(gu):
    s = make_paper_workload(96, 54, E=2)
    V = s.E * s.A * s.K
    act = np.flatnonzero(np.repeat(s.active.reshape(-1), s.K))
    views = np.concatenate([act[::7], np.arange(V - 8, V)])       # views of active agents, and some of inactive slots (sky)
    st = check_colour(gu, s, views=views)
    print("paper 96x54 colour:", st)
    # rows that allow no vector stores (W = 100), several tiles per view, a signal disk with a limited angular range
    base = make_config(2, E=1)
    disk = disk_triangles((base.poses[0, 0, 0] + 15.0 * np.cos(base.poses[0, 0, 2]), base.poses[0, 0, 1] + 15.0 * np.sin(base.poses[0, 0, 2]), 3.0),
                          (-np.cos(base.poses[0, 0, 2]), -np.sin(base.poses[0, 0, 2]), 0.0), 0.5, n=10)
    tris = np.concatenate([base.tri_xyz, disk]); cls = np.concatenate([base.tri_class, np.full(len(disk), 6, np.uint8)])
    lim = np.concatenate([np.zeros(len(base.tri_xyz), np.float32), np.full(len(disk), np.cos(np.radians(50.0)), np.float32)])
    rig = make_rig((0.0, 120.0), 80.0, 60.0, 100, 70)
    s2 = custom_scene(tris, cls, base.poses[:, :12], base.dims[:, :12], rig, 70, 100, base.near, base.far, tri_vis_cos=lim)
    st = check_colour(gu, s2)
    print("70x100 colour:", st)


def test_view_subrange_and_relative_output(gu):
    import torch
    import oracle
    import paper_2607_26005_b200 as pic
    s = make_config(1, E=1)
    g = gu.CudaRun(s)
    try:
        full, _ = g.render_rgb(PAL, True)
        part, _ = g.render_rgb(PAL, True, view_first=9, view_count=5)
        assert (part[9:14] == full[9:14]).all() and (part[:9] == 7).all() and (part[14:] == 7).all()
        out = torch.full((5, s.H, s.W, 3), 9, dtype=torch.uint8, device=g.dev)
        g.scene.set_option(pic.OPT_VIEW_FIRST, 9); g.scene.set_option(pic.OPT_VIEW_COUNT, 5); g.scene.set_option(pic.OPT_OUT_RELATIVE, 1)
        g.scene.render_rgb(g.poses, g.dims, s.rig, active=g.active, out_rgb=out, antialias=True)
        torch.cuda.synchronize()
        g.scene.set_option(pic.OPT_VIEW_FIRST, 0); g.scene.set_option(pic.OPT_VIEW_COUNT, 0); g.scene.set_option(pic.OPT_OUT_RELATIVE, 0)
        assert (out.cpu().numpy() == full[9:14]).all()
    finally:
        g.close()


def test_paper_chunk_of_2048_egos_in_colour(gu):
    # the bench's own launch: 31 map instances x 120 slots x 4 cameras at 96 x 54, antialiased; the oracle on sampled views
    s = make_paper_workload(96, 54, egos=2048)
    rng = np.random.default_rng(3)
    act = np.flatnonzero(np.repeat(s.active.reshape(-1), s.K))
    views = np.sort(rng.choice(act, size=96, replace=False))
    st = check_colour(gu, s, views=views, modes=(True,))
    print("paper chunk colour:", st)
    # configs[2] at 16 environments (4 096 views of 64 x 64), plain and antialiased
    s2 = make_config(2, E=16)
    st2 = check_colour(gu, s2, views=np.sort(rng.choice(s2.E * s2.A * s2.K, size=64, replace=False)))
    print("cfg2 E=16 colour:", st2)


def test_random_scenes_in_colour(gu):
    # seeded random scenes (soups of triangles through the camera plane, pitched cameras, ragged sizes): plain and antialiased
    from tests.util import random_scene
    import oracle
    pixels = flagged = mism = 0
    for i, seed in enumerate([143, 209, 904, 1236] + list(range(1000, 1024))):
        s = random_scene(seed, full_tiles=(i % 3 == 2))
        g = gu.CudaRun(s)
        try:
            for aa in (False, True):
                got, status = g.render_rgb(PAL, aa)
                assert status == 0, f"seed {seed}: status {status}"
                ref = oracle.render_rgb(s, PAL, aa)
                try:
                    st = compare_colour(ref, got, max_mismatch_frac=5e-3, max_flag_frac=0.1)
                except AssertionError as ex:
                    raise AssertionError(f"seed {seed}, antialias {aa}: {ex}") from ex
                pixels += st["pixels"]; flagged += st["flagged"]; mism += st["mismatches"]
        finally:
            g.close()
    print("random scenes in colour:", dict(pixels=pixels, flagged=flagged, mismatches=mism))
    assert flagged < 0.02 * pixels


def test_many_tiles_per_view_in_colour(gu):
    # configs[3] (128 x 256: 8 tiles per view, one 37 k-triangle map, far 150 m) and the paper's rig at 384 x 216 (24 tiles)
    s = make_config(3, E=1)
    st = check_colour(gu, s, views=[0, 101, 202])
    print("cfg3 colour:", st)
    s = make_paper_workload(384, 216, E=1)
    act = np.flatnonzero(np.repeat(s.active.reshape(-1), s.K))
    st = check_colour(gu, s, views=act[:3], modes=(True,))
    print("paper 384x216 colour:", st)


def test_step_with_colour_output(gu):
    # pic_step_rgb = the bicycle update of pic_step, then the colour images of the new state
    import torch
    from scenes import make_actions
    s = make_config(1, E=1)
    g = gu.CudaRun(s)
    try:
        g.scene.set_palette(PAL)
        state = torch.from_numpy(s.state()).to(g.dev)
        acts = torch.from_numpy(make_actions(4, 1, s.E, s.A)).to(g.dev)
        g.scene.set_state(state, g.dims, g.active)
        rgb = g.scene.step_rgb(acts, s.rig, antialias=True)
        new_state = g.scene.get_state()
        g.scene.set_state(state, g.dims, g.active)
        g.scene.step(acts, s.rig)
        assert torch.equal(new_state, g.scene.get_state())                  # the same update as pic_step
        again = g.scene.render_rgb(new_state[..., :3].contiguous(), g.dims, s.rig, active=g.active, antialias=True)
        torch.cuda.synchronize()
        assert torch.equal(rgb, again) and g.scene.status() == 0
        assert not torch.equal(rgb, g.scene.render_rgb(g.poses, g.dims, s.rig, active=g.active, antialias=True))   # the agents moved
    finally:
        g.close()
