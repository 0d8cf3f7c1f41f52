"""Pins of the CPU oracle against things other than itself: closed forms worked by hand, values the
paper prints (camera table), invariants, an independent world-space ray caster, hand-counted tiny
scenes and a library binary16 conversion.  No GPU needed."""
import os

import numpy as np
import pytest

import oracle
from scenes import make_config, make_rig, custom_scene, focal_px, disk_triangles
from tests.util import single_env, compare_images

HERE = os.path.dirname(os.path.abspath(__file__))
CAR = (4.5, 1.9, 1.5)


def ego(x=0.0, y=0.0, yaw=0.0, dims=CAR):
    return (x, y, yaw) + tuple(dims)


# ------------------------------------------------------------------------------------------------
# closed form: empty scene = analytic ground plane below the horizon row, sky above
# ------------------------------------------------------------------------------------------------
def test_empty_scene_ground_sky_split():
    s = single_env(np.zeros((0, 3, 3)), [], [ego()])
    r = oracle.render(s)
    cls, z = r.cls[0], r.depth[0]
    assert (cls[:32] == 0).all() and (z[:32] == 100.0).all()
    assert (cls[32:] == 1).all()
    # camera 1.5 m high, fy = 32: the ray of row v drops (v - 31.5)/32 per metre -> z = 48 / (v - 31.5)
    for v, zz in ((32, 96.0), (33, 32.0), (34, 19.2), (35, 13.714285714285714), (63, 1.5238095238095237)):
        assert np.allclose(z[v], zz, rtol=1e-14, atol=0), (v, z[v, 0])
    f16 = r.depth_f16[0]
    assert f16[34, 0] == np.float16(19.203125) and f16[35, 5] == np.float16(13.7109375)
    assert f16[63, 63] == np.float16(1.5234375) and f16[0, 0] == np.float16(100.0)
    assert (r.index[0] == -1).all() and (r.flag[0] == 0).all()
    assert r.counts[0].tolist() == [0, 0, 0, 0]


def test_empty_scene_pitch_moves_horizon():
    # pitch up by atan(0.25): horizon at v + 0.5 = 32 + 32*0.25 = 40 -> rows 0..39 sky, 40.. ground
    phi = np.degrees(np.arctan(0.25))
    s = single_env(np.zeros((0, 3, 3)), [], [ego()], rig=make_rig((0.0,), 90.0, 90.0, pitch_deg=phi))
    r = oracle.render(s)
    assert (r.cls[0][:40] == 0).all() and (r.cls[0][40:] == 1).all()
    # row 40: ray (0, 8.5/32, 1) in camera axes; with tan(phi) = 1/4 its world slope per unit of
    # horizontal travel is (1/4 - 8.5/32) / (1 + 8.5/128); depth along the axis follows from that
    ry = 8.5 / 32
    p32 = float(s.rig[0, 4])               # the pitch as the float32 the renderer is given
    down_per_depth = ry * np.cos(p32) - np.sin(p32)   # metres of descent per metre of view depth
    assert np.allclose(r.depth[0][40], 1.5 / down_per_depth, rtol=1e-12)
    assert abs(r.depth[0][40, 0] - 1.5 / (ry * np.cos(np.arctan(0.25)) - np.sin(np.arctan(0.25)))) < 1e-3


def test_empty_scene_wide_camera_far_clamp():
    # 128 x 256, hfov 96, vfov 40: fy = 64 / tan(20 deg) = 175.8386; rows 64, 65 see the ground
    # beyond the 150 m far plane (1.5 fy / 0.5 = 527.5 m, / 1.5 = 175.8 m), row 66 at 105.503 m
    s = single_env(np.zeros((0, 3, 3)), [], [ego()], rig=make_rig((0.0,), 96.0, 40.0, 256, 128), H=128, W=256, far=150.0)
    r = oracle.render(s)
    assert (r.cls[0][:64] == 0).all() and (r.cls[0][64:] == 1).all()
    assert (r.depth[0][64] == 150.0).all() and (r.depth[0][65] == 150.0).all()
    assert np.allclose(r.depth[0][66], 105.503, rtol=1e-5)


# ------------------------------------------------------------------------------------------------
# closed form: one box straight ahead (all numbers exact in binary)
# ------------------------------------------------------------------------------------------------
def _one_box(width=1.9, height=1.5, mount_z=1.5):
    rig = make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, mount_z))
    return single_env(np.zeros((0, 3, 3)), [], [ego(), (12.5, 0.0, 0.0, 4.5, width, height)], rig=rig)


def test_one_box_rectangle_and_depth():
    # rear face 8 m ahead of the camera, 1.9 wide, 1.5 tall, camera at its top height:
    # columns 32 +- 3.8 -> centres 28.5..35.5 ; rows 32..38 -> centres 32.5..37.5
    r = oracle.render(_one_box(), view_ids=[0])
    cls, z = r.cls[0], r.depth[0]
    box = np.zeros((64, 64), bool)
    box[32:38, 28:36] = True
    assert (cls[box] == 4).all() and (cls[~box] != 4).all() and box.sum() == 48
    assert np.allclose(z[box], 8.0, rtol=1e-13)
    assert (r.depth_f16[0][box] == np.float16(8.0)).all()
    assert set(np.unique(r.index[0][box])) <= {12 + 0, 12 + 1, 12 + 4, 12 + 5}  # rear face (agent 1) or an exact tie on its rim
    # the second view (from the box towards nothing) never shows the ego itself
    r1 = oracle.render(_one_box(), view_ids=[1])
    assert (r1.cls[0] != 4).all()


def test_fill_rule_left_and_top_edges_owned():
    # width 1.75: vertical edges exactly on the centres of columns 28 and 35 -> 28 owned, 35 not
    r = oracle.render(_one_box(width=1.75), view_ids=[0])
    got = r.cls[0] == 4
    want = np.zeros((64, 64), bool)
    want[32:38, 28:35] = True
    assert (got == want).all() and got.sum() == 42
    # height 1.375: top edge exactly on the centre of row 32 (camera 0.125 above it) -> owned
    r = oracle.render(_one_box(height=1.375), view_ids=[0])
    want = np.zeros((64, 64), bool)
    want[32:38, 28:36] = True
    assert ((r.cls[0] == 4) == want).all()
    # camera at 1.375: bottom edge exactly on the centre of row 37 -> not owned; top edge at
    # 32 - 4*0.125 = 31.5 -> row 31 centre exactly on the top edge -> owned
    r = oracle.render(_one_box(mount_z=1.375), view_ids=[0])
    want = np.zeros((64, 64), bool)
    want[31:37, 28:36] = True
    assert ((r.cls[0] == 4) == want).all()


def test_flat_map_depth_closed_form():
    # pitch 0, camera 1.5 m high: road pixels of row v lie at 48/(v-31.5), markings 2 cm higher
    s = make_config(0)
    r = oracle.render(s)
    v = np.broadcast_to(np.arange(64)[None, :, None], r.cls.shape)
    road, mark = r.cls == 2, r.cls == 3
    assert road.sum() > 1000 and mark.sum() > 20
    assert np.allclose(r.depth[road], 48.0 / (v[road] - 31.5), rtol=1e-9)
    assert np.allclose(r.depth[mark], 47.36 / (v[mark] - 31.5), rtol=1e-9)
    assert (r.depth >= s.near).all() and (r.depth <= s.far).all()
    assert (r.depth[r.cls == 0] == s.far).all()


# ------------------------------------------------------------------------------------------------
# the paper's camera table: focal length <-> field of view, yaw sign
# ------------------------------------------------------------------------------------------------
def _golden_rig():
    vals, cams = {}, {}
    for line in open(os.path.join(HERE, "golden", "camera_rig.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if len(t) == 2:
            vals[t[0]] = float(t[1])
        else:
            cams[t[0]] = tuple(float(x) for x in t[1:])
    return vals, cams


def test_paper_intrinsics_focal_vs_fov():
    g, _ = _golden_rig()
    # render at 1/10 of the sensor; the focal length scales with the resolution
    W, H = int(g["sensor_width_px"]) // 10, int(g["sensor_height_px"]) // 10
    s = single_env(np.zeros((0, 3, 3)), [], [ego()], rig=make_rig((0.0,), g["hfov_deg"], g["vfov_deg"], W, H), H=H, W=W)
    r = oracle.render(s)
    # ground depth of row v is C_z * fy / (v + 0.5 - H/2): read fy back from the image
    v = H - 1
    fy = r.depth[0][v, 0] * (v + 0.5 - H / 2) / 1.5
    assert abs(fy * 10 - g["focal_px"]) < 2.0          # 38.5 deg is printed to 3 digits
    # a wall edge at azimuth atan(0.25) to the right lands 0.25*fx right of centre
    wall = [[(4.0, -1.0, -50.0), (400.0, -100.0, -50.0), (400.0, -100.0, 50.0)],
            [(4.0, -1.0, -50.0), (400.0, -100.0, 50.0), (4.0, -1.0, 50.0)]]
    far_wall = [[(50.0, -200.0, -50.0), (50.0, 200.0, 50.0), (50.0, 200.0, -50.0)],
                [(50.0, -200.0, -50.0), (50.0, -200.0, 50.0), (50.0, 200.0, 50.0)]]
    rig0 = make_rig((0.0,), g["hfov_deg"], g["vfov_deg"], W, H, mount=(0.0, 0.0, 1.5))
    s = single_env(wall + far_wall, [5, 5, 6, 6], [ego()], rig=rig0, H=H, W=W, far=1000.0)
    r = oracle.render(s)
    row = r.cls[0][10]
    # the near wall (class 5) is seen edge-on and covers nothing; the far wall fills the row
    assert (row == 6).all()
    # slant the near wall a little so that it occludes everything right of its leading edge
    wall2 = [[(4.0, -1.0, -50.0), (400.0, -120.0, -50.0), (400.0, -120.0, 50.0)],
             [(4.0, -1.0, -50.0), (400.0, -120.0, 50.0), (4.0, -1.0, 50.0)]]
    wall3 = [[(4.0, -1.0, -50.0), (40.0, -10.0, 50.0), (40.0, -10.0, -50.0)],
             [(4.0, -1.0, -50.0), (4.0, -1.0, 50.0), (40.0, -10.0, 50.0)]]
    s = single_env(wall2 + wall3 + far_wall, [5, 5, 5, 5, 6, 6], [ego()], rig=rig0, H=H, W=W, far=1000.0)
    r = oracle.render(s)
    row = r.cls[0][10]
    edge = np.flatnonzero(row == 5)
    fx = (edge.min() - W / 2) / 0.25      # first column whose centre is right of the leading edge
    assert abs(fx * 10 - g["focal_px"]) < 25.0   # one pixel of 1/10-scale image = 40 px of focal length
    assert abs(2 * np.degrees(np.arctan(g["sensor_width_px"] / 2 / g["focal_px"])) - g["hfov_deg"]) < 0.05


def test_paper_rig_yaw_sign_front_left_sees_left():
    g, cams = _golden_rig()
    W, H = int(g["render_width_px"]), int(g["render_height_px"])
    rig = np.zeros((4, 7), np.float32)
    for i, name in enumerate(("front", "front_left", "front_right", "back")):
        x, y, z, yaw = cams[name]
        rig[i] = (x, y, z, np.radians(yaw), 0.0, focal_px(W, g["hfov_deg"]), focal_px(H, g["vfov_deg"]))
    # a second car 20 m down the optical axis of the front-left camera (ahead and to the LEFT, +y),
    # heading along that axis, so its rear face is centred and fronto-parallel in that camera
    b = np.radians(55.0)
    cx_, cy_ = cams["front_left"][0], cams["front_left"][1]
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), (cx_ + 20 * np.cos(b), cy_ + 20 * np.sin(b), b) + CAR],
                   rig=rig, H=H, W=W)
    r = oracle.render(s, view_ids=[0, 1, 2, 3])
    n4 = [(r.cls[i] == 4).sum() for i in range(4)]
    assert n4[1] > 20 and n4[2] == 0 and n4[3] == 0
    cols = np.flatnonzero((r.cls[1] == 4).any(axis=0))
    assert abs(cols.mean() - (W - 1) / 2) <= 0.5     # centred in the front-left image
    # and in the front camera (hfov 63.7 -> +-31.85 deg) a car at +20 deg is in the LEFT half
    b = np.radians(20.0)
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), (20 * np.cos(b), 20 * np.sin(b), 0.0) + CAR], rig=rig, H=H, W=W)
    r = oracle.render(s, view_ids=[0])
    cols = np.flatnonzero((r.cls[0] == 4).any(axis=0))
    assert len(cols) and cols.max() < W / 2


# ------------------------------------------------------------------------------------------------
# independent ray caster: world-space Moeller-Trumbore, no camera-space transform, no edge normals
# ------------------------------------------------------------------------------------------------
def _ray_cast(scene, e, a, k):
    s = scene
    x, y, th = (float(t) for t in s.poses[e, a])
    mx, my, mz, yaw, pitch, fx, fy = (float(t) for t in s.rig[k])
    az = th + yaw
    fwd = np.array([np.cos(pitch) * np.cos(az), np.cos(pitch) * np.sin(az), np.sin(pitch)])
    right = np.array([np.sin(az), -np.cos(az), 0.0])
    down = np.cross(fwd, right)
    origin = np.array([x + np.cos(th) * mx - np.sin(th) * my, y + np.sin(th) * mx + np.cos(th) * my, mz])
    t0, t1 = s.map_slice(e)
    tris = [(s.tri_xyz[i].astype(np.float64), int(s.tri_class[i])) for i in range(t0, t1)]
    assert s.A == 1, "ray caster handles map triangles only"
    cls = np.full((s.H, s.W), -1, int)
    depth = np.full((s.H, s.W), np.inf)
    for v in range(s.H):
        for u in range(s.W):
            d = fwd + (u + 0.5 - s.W / 2) / fx * right + (v + 0.5 - s.H / 2) / fy * down
            for tri, c in tris:
                e1, e2 = tri[1] - tri[0], tri[2] - tri[0]
                pvec = np.cross(d, e2)
                det = e1 @ pvec
                if det == 0:
                    continue
                tvec = origin - tri[0]
                uu = (tvec @ pvec) / det
                qvec = np.cross(tvec, e1)
                vv = (d @ qvec) / det
                t = (e2 @ qvec) / det
                if uu < 0 or vv < 0 or uu + vv > 1 or t < s.near or t > s.far:
                    continue
                if t < depth[v, u]:
                    depth[v, u], cls[v, u] = t, c
    return cls, depth


@pytest.mark.parametrize("seed", range(6))
def test_against_world_space_ray_caster(seed):
    rng = np.random.default_rng(seed)
    n = 12
    # triangles scattered around a camera at the origin region, many crossing the camera plane
    centre = rng.uniform(-6, 6, size=(n, 1, 3)) + np.array([4.0, 0.0, 1.0])
    tris = centre + rng.uniform(-6, 6, size=(n, 3, 3))
    classes = rng.integers(2, 9, size=n)
    H, W = (12, 16) if seed % 2 else (16, 12)
    rig = make_rig((float(rng.uniform(-180, 180)),), 80.0, 60.0, W, H, mount=(0.7, -0.3, 1.2),
                   pitch_deg=float(rng.uniform(-20, 20)))
    s = single_env(tris, classes, [ego(rng.uniform(-2, 2), rng.uniform(-2, 2), rng.uniform(-3, 3))],
                   rig=rig, H=H, W=W, near=0.5, far=30.0)
    r = oracle.render(s)
    cls, depth = _ray_cast(s, 0, 0, 0)
    hit = cls >= 0
    ok = r.flag[0] != 0                       # either answer is acceptable on flagged pixels
    assert hit.sum() > 20
    assert (((r.index[0] >= 0) == hit) | ok).all()
    assert ((r.cls[0] == cls) | ~hit | ok).all()
    both = hit & (r.index[0] >= 0) & ~ok
    assert np.allclose(r.depth[0][both], depth[both], rtol=1e-9)


# ------------------------------------------------------------------------------------------------
# hand-counted tiny scenes
# ------------------------------------------------------------------------------------------------
RIG0 = make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0))   # 8x8 image, fx = fy = 4, at (0,0,1) looking along +x
RIG32 = make_rig((0.0,), 90.0, 90.0, 32, 32)
RIG16 = make_rig((0.0,), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 1.0))


def _wall(x, y0, y1, z0, z1):
    """Rectangle in the plane x = const facing the camera: two triangles."""
    return [[(x, y0, z0), (x, y1, z0), (x, y1, z1)], [(x, y0, z0), (x, y1, z1), (x, y0, z1)]]


def test_single_triangle_hand_counted():
    # 8x8 image, fx = fy = 4, wall triangle at x = 4: one pixel per metre, column = 4 - y, row = 4 - (z-1)
    # vertices (y,z): (2,3) (-2,3) (2,-1) -> pixel-space corners (2,2) (6,2) (2,6): right triangle,
    # centres (u+.5, v+.5) inside iff (u+.5-2) + (v+.5-2) < 4, i.e. u+v < 7 (u,v >= 2); hypotenuse is not top-left
    tri = [[(4.0, 2.0, 3.0), (4.0, -2.0, 3.0), (4.0, 2.0, -1.0)]]
    s = single_env(tri, [7], [ego()], rig=RIG0, H=8, W=8)
    r = oracle.render(s)
    want = np.zeros((8, 8), bool)
    for v in range(2, 8):
        for u in range(2, 8):
            want[v, u] = (u + v) < 7
    assert ((r.cls[0] == 7) == want).all() and want.sum() == 6
    assert np.allclose(r.depth[0][want], 4.0)
    assert r.counts[0, 0] == 1 and r.counts[0, 1] == 1 and r.counts[0, 2] == 6


def test_two_walls_nearest_wins_and_occluded_box_is_invisible():
    near_wall = _wall(4.0, -1.0, 1.0, 0.0, 2.0)     # covers columns 3..4, rows 3..4 of an 8x8 image
    far_wall = _wall(8.0, -6.0, 6.0, -3.0, 5.0)     # covers columns 1..6, rows 2..5
    s = single_env(far_wall + near_wall, [5, 5, 6, 6], [ego()], rig=RIG0, H=8, W=8)
    r = oracle.render(s)
    c = r.cls[0]
    assert (c[3:5, 3:5] == 6).all() and (c == 6).sum() == 4
    assert (c == 5).sum() == 6 * 4 - 4
    assert np.allclose(r.depth[0][c == 6], 4.0) and np.allclose(r.depth[0][c == 5], 8.0)
    # a car hidden behind the near wall changes nothing (occlusion is real)
    wall = _wall(4.0, -3.9, 3.9, -2.9, 4.9)
    s0 = single_env(wall, [6, 6], [ego()], rig=RIG0, H=8, W=8)
    s1 = single_env(wall, [6, 6], [ego(), (10.0, 0.0, 0.3) + CAR], rig=RIG0, H=8, W=8)
    r0, r1 = oracle.render(s0, view_ids=[0]), oracle.render(s1, view_ids=[0])
    assert (r0.cls == r1.cls).all() and (r0.depth == r1.depth).all()
    assert (r1.cls != 4).all()


def test_exact_depth_tie_goes_to_lower_index():
    a = _wall(4.0, -2.0, 2.0, -1.0, 3.0)
    b = _wall(4.0, -1.0, 3.0, 0.0, 4.0)
    for tris, classes, want in ((a + b, [5, 5, 6, 6], 5), (b + a, [6, 6, 5, 5], 6)):
        s = single_env(tris, classes, [ego()], rig=RIG0, H=8, W=8)
        r = oracle.render(s)
        # overlap of the two walls: y in [-1,2] -> columns 2..4, z in [0,3] -> rows 2..4
        assert (r.cls[0][2:5, 2:5] == want).all()
        assert (r.flag[0][2:5, 2:5] & 2).all()      # and the tie is reported as a depth ambiguity


def test_near_and_far_planes_inclusive():
    s = single_env(_wall(0.5, -4, 4, -3, 5) , [5, 5], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=100.0)
    assert (oracle.render(s).cls[0] == 5).all()
    s = single_env(_wall(0.4375, -4, 4, -3, 5), [5, 5], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=100.0)
    assert (oracle.render(s).cls[0] != 5).all()
    s = single_env(_wall(64.0, -400, 400, -300, 500), [5, 5], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=64.0)
    assert (oracle.render(s).cls[0] == 5).all()
    s = single_env(_wall(64.5, -400, 400, -300, 500), [5, 5], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=64.0)
    assert (oracle.render(s).cls[0] != 5).all()


def test_triangle_through_camera_plane_needs_no_clipping():
    # a ground-level strip from 10 m behind the camera to 20 m ahead, 2 m wide, 1 m below the camera
    strip = [[(-10.0, -1.0, 0.0), (20.0, -1.0, 0.0), (20.0, 1.0, 0.0)], [(-10.0, -1.0, 0.0), (20.0, 1.0, 0.0), (-10.0, 1.0, 0.0)]]
    s = single_env(strip, [2, 2], [ego()], rig=RIG16, H=16, W=16, near=0.5, far=100.0)
    r = oracle.render(s)
    fx = 8.0
    for v in range(16):
        for u in range(16):
            ry = (v + 0.5 - 8) / fx
            rx = (u + 0.5 - 8) / fx
            inside = False
            if ry > 0:
                z = 1.0 / ry                       # ground hit at view depth z, lateral offset rx*z
                inside = (0.5 <= z <= 20.0) and -1.0 <= rx * z < 1.0   # left edge owned, right edge not
            assert (r.cls[0][v, u] == 2) == inside, (u, v)


def test_frustum_counts():
    def t_vis(tri, **kw):
        s = single_env([tri], [5], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=50.0, **kw)
        return int(oracle.render(s).counts[0, 0])
    assert t_vis([(4, -1, 0.5), (4, 1, 0.5), (4, 0, 1.5)]) == 1            # inside
    assert t_vis([(-4, -1, 0.5), (-4, 1, 0.5), (-4, 0, 1.5)]) == 0         # behind
    assert t_vis([(60, -1, 0.5), (60, 1, 0.5), (60, 0, 1.5)]) == 0         # beyond far
    assert t_vis([(4, 10, 0.5), (4, 12, 0.5), (4, 11, 1.5)]) == 0          # off to the left
    assert t_vis([(-4, 0, 0), (20, -1, 0), (20, 1, 0)]) == 1               # straddles the camera plane
    assert t_vis([(10, -100, -100), (10, 100, -100), (10, 0, 200)]) == 1   # encloses the whole frustum
    assert t_vis([(0.2, -0.1, 1.0), (0.3, 0.1, 1.0), (0.3, 0.0, 1.1)]) == 0  # in front of the near plane
    assert t_vis([(4, 3.9, 1), (4, 12, 1), (4, 12, 2)]) == 1               # clips the left frustum side (y = x)
    assert t_vis([(4, 4.1, 1), (4, 12, 1), (4, 12, 2)]) == 0


# ------------------------------------------------------------------------------------------------
# invariants
# ------------------------------------------------------------------------------------------------
def _small_world(seed=3):
    rng = np.random.default_rng(seed)
    gm_tris = []
    for i in range(40):
        c = np.array([rng.integers(-640, 640) / 16.0, rng.integers(-640, 640) / 16.0, 0.0])
        gm_tris.append(c + np.round(rng.uniform(-8, 8, size=(3, 3)) * 16) / 16 * np.array([1, 1, 0.2]))
    classes = rng.integers(2, 6, size=40)
    agents = [ego(0.0, 0.0, 0.0)] + [(rng.integers(-300, 300) / 16.0, rng.integers(-300, 300) / 16.0,
                                      float(np.float32(rng.uniform(-3, 3)))) + CAR for _ in range(5)]
    return np.array(gm_tris), classes, agents


def test_translation_by_powers_of_two_is_bit_exact():
    tris, classes, agents = _small_world()
    rig = make_rig((0.0, 90.0, 180.0, 270.0), 90.0, 90.0, 32, 32)
    base = oracle.render(single_env(tris, classes, agents, rig=rig, H=32, W=32))
    assert (base.cls == 4).sum() > 50 and (base.cls >= 2).sum() > 500
    for dx, dy in ((256.0, -512.0), (-1024.0, 64.0)):
        t2 = tris + np.array([dx, dy, 0.0])
        a2 = [(a[0] + dx, a[1] + dy) + tuple(a[2:]) for a in agents]
        moved = oracle.render(single_env(t2, classes, a2, rig=rig, H=32, W=32))
        assert (moved.cls == base.cls).all() and (moved.index == base.index).all()
        on_map = base.index < len(tris)           # map vertices minus the ego position is exact in binary
        assert (moved.depth[on_map] == base.depth[on_map]).all()
        assert np.allclose(moved.depth, base.depth, rtol=1e-11, atol=0)   # box corners round at 1e-16 * 1024


def test_rotation_and_general_motion_leave_image_unchanged():
    tris, classes, agents = _small_world(5)
    rig = make_rig((0.0, 90.0), 90.0, 90.0, 32, 32)
    base = oracle.render(single_env(tris, classes, agents, rig=rig, H=32, W=32))
    for ang, dx, dy in ((np.pi / 2, 0.0, 0.0), (0.7, 13.25, -7.5)):
        c, s_ = np.cos(ang), np.sin(ang)
        R = np.array([[c, -s_, 0], [s_, c, 0], [0, 0, 1]])
        t2 = tris @ R.T + np.array([dx, dy, 0.0])
        a2 = [(c * a[0] - s_ * a[1] + dx, s_ * a[0] + c * a[1] + dy, a[2] + ang) + tuple(a[3:]) for a in agents]
        moved = oracle.render(single_env(t2, classes, a2, rig=rig, H=32, W=32))
        # inputs are re-rounded to float32, so equality holds off the flagged pixels, depth to ~1e-6
        compare_images(base.cls, base.depth, base.flag | moved.flag, moved.cls, moved.depth, depth_rtol=1e-5,
                       max_mismatch_frac=5e-3)


def test_primitive_order_does_not_matter_without_ties():
    tris, classes, agents = _small_world(7)
    base = oracle.render(single_env(tris, classes, agents, rig=RIG32, H=32, W=32), view_ids=[0])
    perm = np.random.default_rng(0).permutation(len(tris))
    shuf = oracle.render(single_env(tris[perm], classes[perm], agents, rig=RIG32, H=32, W=32), view_ids=[0])
    assert (base.cls == shuf.cls).all() and (base.depth == shuf.depth).all()


def test_mirror_scene_mirrors_image():
    tris, classes, agents = _small_world(11)
    m = np.array([1.0, -1.0, 1.0])
    base = oracle.render(single_env(tris, classes, agents, rig=RIG32, H=32, W=32), view_ids=[0])
    a2 = [(a[0], -a[1], -a[2]) + tuple(a[3:]) for a in agents]
    mir = oracle.render(single_env(tris * m, classes, a2, rig=RIG32, H=32, W=32), view_ids=[0])
    flag = base.flag | mir.flag[:, :, ::-1]
    diff = (base.cls != mir.cls[:, :, ::-1]) & (flag == 0)
    assert diff.sum() == 0
    same = base.cls == mir.cls[:, :, ::-1]
    assert np.allclose(base.depth[same & (flag == 0)], mir.depth[:, :, ::-1][same & (flag == 0)], rtol=1e-6)


def test_ego_excluded_inactive_and_other_envs():
    # camera INSIDE the ego's own box (mount at the centre): the ego must not be drawn
    rig = make_rig((0.0,), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 0.75))
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), (10.0, 0.0, 0.0) + CAR], rig=rig, H=16, W=16)
    r = oracle.render(s)
    assert (r.cls[0] == 4).sum() > 0 and (r.cls[0] == 4).sum() < 60      # only the other car
    s1 = single_env(np.zeros((0, 3, 3)), [], [ego()], rig=rig, H=16, W=16)
    assert (oracle.render(s1).cls != 4).all()
    # inactive other agent is not drawn; inactive ego renders sky/far everywhere
    s2 = single_env(np.zeros((0, 3, 3)), [], [ego(), (10.0, 0.0, 0.0) + CAR], rig=rig, H=16, W=16, active=[1, 0])
    r2 = oracle.render(s2)
    assert (r2.cls[0] != 4).all()
    assert (r2.cls[1] == 0).all() and (r2.depth[1] == 100.0).all()
    # two envs on one shared map: agents of env 1 never show up in env 0
    poses = np.array([[[0, 0, 0]], [[10, 0, 0]]], np.float32)
    dims = np.tile(np.array(CAR, np.float32), (2, 1, 1))
    s3 = custom_scene(np.zeros((0, 3, 3)), [], poses, dims, rig, 16, 16)
    assert (oracle.render(s3).cls != 4).all()


def test_determinism():
    s = make_config(0)
    a, b = oracle.render(s, n_threads=1), oracle.render(s, n_threads=4)
    assert (a.cls == b.cls).all() and (a.depth == b.depth).all() and (a.counts == b.counts).all()


def test_flag_fraction_is_small_on_a_real_workload():
    s = make_config(1, E=1)
    r = oracle.render(s, view_ids=np.arange(0, 128, 5))
    frac = (r.flag != 0).mean()
    assert frac < 3e-3, frac


# ------------------------------------------------------------------------------------------------
# binary16 rounding against the library conversion
# ------------------------------------------------------------------------------------------------
def test_f16_rounding_matches_numpy():
    rng = np.random.default_rng(0)
    vals = np.concatenate([rng.uniform(0.4, 160.0, 20000), 2.0 ** rng.uniform(-26, 17, 5000),
                           [0.0, 1.0, 100.0, 150.0, 65504.0, 65519.9, 65520.0, 1e-8, 6e-8, 2.0 ** -24, 2.0 ** -25,
                            1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24]])
    # exact ties between neighbouring binary16 values
    h = rng.integers(0x0001, 0x7bfe, 5000).astype(np.uint16)
    lo, hi = h.view(np.float16).astype(np.float64), (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    vals = np.concatenate([vals, (lo + hi) / 2, -vals[:100]])
    with np.errstate(over="ignore"):
        want = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f64_to_f16_bits(v) for v in vals], np.uint16)
    assert (got == want).all()


# ------------------------------------------------------------------------------------------------
# kinematic bicycle closed forms
# ------------------------------------------------------------------------------------------------
def test_bicycle_straight_line_and_clamps():
    st = np.array([[1.0, 2.0, 0.5, 10.0], [0.0, 0.0, 0.0, 0.5], [0.0, 0.0, 0.0, 29.5]])
    act = np.array([[1.0, 0.0], [-3.0, 0.0], [2.0, 0.0]], np.float32)
    x = st.copy()
    dist = 0.0
    for n in range(20):
        dist += x[0, 3] * 0.1
        x = oracle.step(x, act, None, 0.1, 2.8, 30.0)
    # v_t = 10 + 0.1 t ; travelled = sum_{t<20} v_t dt = 0.1*(200 + 0.1*190) = 21.9
    assert np.isclose(dist, 21.9) and np.allclose(x[0], [1 + 21.9 * np.cos(0.5), 2 + 21.9 * np.sin(0.5), 0.5, 12.0])
    assert x[1, 3] == 0.0 and np.isclose(x[1, 0], 0.05 + 0.02)       # 0.5, 0.2, 0 ... then stopped
    assert x[2, 3] == 30.0


def test_bicycle_constant_steer_heading_is_linear():
    st = np.array([[0.0, 0.0, 0.25, 8.0]])
    act = np.array([[0.0, 0.2]], np.float32)
    x = st.copy()
    for n in range(50):
        x = oracle.step(x, act, None, 0.1, 2.8, 30.0)
    delta = float(np.float32(0.2))
    assert np.isclose(x[0, 2], 0.25 + 50 * (8.0 / 2.8) * np.tan(delta) * 0.1, rtol=1e-13)
    assert x[0, 3] == 8.0
    # one hand-worked step: x += v cos(yaw) dt from the OLD heading
    y = oracle.step(np.array([[0.0, 0.0, np.pi / 2, 10.0]]), np.array([[0.0, 0.3]], np.float32), None, 0.1, 2.8, 30.0)
    assert abs(y[0, 0]) < 1e-15 * 10 + 1e-15 and np.isclose(y[0, 1], 1.0)
    # inactive agents do not move
    z = oracle.step(st, act, np.array([0], np.uint8), 0.1, 2.8, 30.0)
    assert (z == st).all()


# ------------------------------------------------------------------------------------------------
# further pins: ambiguity mask semantics, box indices, map selection per environment
# ------------------------------------------------------------------------------------------------
def test_ambiguity_mask_flags_only_near_boundaries():
    # a wall whose left edge passes a given distance (in pixels) from the centres of column 3
    def wall_with_left_edge_offset(eps_px):
        # 8x8 image, fx = 4, wall at x = 4: image column coordinate = 4 - y ; left edge at u = 3.5 + eps
        y_left = 4.0 - (3.5 + eps_px)
        return _wall(4.0, -1.5, y_left, 0.0, 2.0)
    for eps, want_flag in ((1e-7, True), (-1e-7, True), (1e-2, False), (-1e-2, False)):
        s = single_env(wall_with_left_edge_offset(eps), [5, 5], [ego()], rig=RIG0, H=8, W=8)
        r = oracle.render(s)
        col3 = r.flag[0][3:5, 3] & 1          # rows 3, 4 see the wall (z in [0,2] -> rows 3..4)
        assert bool(col3.all()) == want_flag, (eps, r.flag[0])
        # pixels well inside or well outside are never flagged for an edge
        assert (r.flag[0][3:5, 4] & 1).sum() == 0 and (r.flag[0][:, 0] & 1).sum() == 0
    # a second surface 1e-6 relative behind the first, other class: depth ambiguity, and only there
    s = single_env(_wall(4.0, -1, 1, 0, 2) + _wall(4.0 * (1 + 1e-6), -1, 1, 0, 2), [5, 5, 6, 6], [ego()], rig=RIG0, H=8, W=8)
    r = oracle.render(s)
    assert (r.cls[0][3:5, 3:5] == 5).all() and (r.flag[0][3:5, 3:5] & 2).all() and (r.flag[0][0:2] & 2).sum() == 0
    s = single_env(_wall(4.0, -1, 1, 0, 2) + _wall(4.1, -1, 1, 0, 2), [5, 5, 6, 6], [ego()], rig=RIG0, H=8, W=8)
    assert (oracle.render(s).flag[0] & 2).sum() == 0


def test_ambiguity_mask_near_far_planes_and_horizon():
    """The two remaining branches of the mask.  Bit 4: a covered fragment whose depth is within 1e-5 relative of
    the near or the far plane, on either side of it, and that would be visible; bit 8: a background pixel whose
    ray is within 1e-5 of horizontal."""
    for plane, other in ((0.5, 100.0), (64.0, 0.5)):
        near, far = (plane, other) if plane < other else (other, plane)
        size = 8.0 * plane                                    # the wall fills the 90-degree image
        for rel, want in ((0.0, True), (1e-6, True), (-1e-6, True), (1e-2, False), (-1e-2, False)):
            x = np.float32(plane * (1.0 + rel))
            s = single_env(_wall(float(x), -size, size, -size, size), [5, 5], [ego()], rig=RIG0, H=8, W=8, near=near, far=far)
            r = oracle.render(s)
            assert bool((r.flag[0] & 4).all()) == want and bool((r.flag[0] & 4).any()) == want, (plane, rel, r.flag[0])
            # on which side of the plane the wall sits decides whether it is drawn -- flagged or not
            inside = near <= float(x) <= far
            assert (r.cls[0] == 5).all() == inside
    # a wall at the near plane hidden behind nothing but in front of another wall: the nearer one matters, the
    # farther one (at 2 m, well inside the range) does not raise the flag by itself
    s = single_env(_wall(2.0, -16, 16, -16, 16), [6, 6], [ego()], rig=RIG0, H=8, W=8, near=0.5, far=100.0)
    assert (oracle.render(s).flag[0] & 4).sum() == 0
    # horizon: 8 x 8 image, fy = 4, row 5 has ray slope 1.5 / 4; pitch the camera so that this ray is horizontal
    for d, want in ((1e-6, True), (-1e-6, True), (1e-2, False), (-1e-2, False)):
        phi = np.degrees(np.arctan(0.375) + d)
        s = single_env(np.zeros((0, 3, 3)), [], [ego()], rig=make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0), pitch_deg=phi),
                       H=8, W=8)
        r = oracle.render(s)
        assert bool((r.flag[0][5] & 8).all()) == want, (d, r.flag[0])
        assert (np.delete(r.flag[0], 5, axis=0) & 8).sum() == 0
        # above the horizon row sky, below it ground, whatever the flagged row itself shows
        assert (r.cls[0][:5] == 0).all() and (r.cls[0][6:] == 1).all()
    # a primitive covering the pixel takes the horizon flag away: it is about the background only
    s = single_env(_wall(4.0, -8, 8, -8, 8), [5, 5], [ego()],
                   rig=make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0), pitch_deg=np.degrees(np.arctan(0.375))), H=8, W=8)
    assert (oracle.render(s).flag[0] & 8).sum() == 0


def test_box_primitive_indices_and_tie_between_identical_boxes():
    # two identical boxes at the same pose: every pixel is an exact tie, the lower agent index wins,
    # and the winning index is N + 12 b + t with N map triangles
    tri = [[(50.0, -1.0, 0.0), (51.0, -1.0, 0.0), (51.0, 1.0, 0.0)]]      # one map triangle, far away
    agents = [ego(), (12.5, 0.0, 0.0) + CAR, (12.5, 0.0, 0.0) + CAR]
    s = single_env(tri, [2], agents)
    r = oracle.render(s, view_ids=[0])
    on_box = r.cls[0] == 4
    assert on_box.sum() == 48
    idx = r.index[0][on_box]
    assert idx.min() >= 1 + 12 * 1 and idx.max() < 1 + 12 * 2            # agent 1's triangles only
    assert set(np.unique(idx)) <= {1 + 12 + 0, 1 + 12 + 1, 1 + 12 + 4, 1 + 12 + 5}   # rear face, or a tie on its rim
    # agent 2's camera sits on the front face of both boxes and looks away: nothing of them is in range
    r2 = oracle.render(s, view_ids=[2])
    assert (r2.cls[0] != 4).all()


def test_each_environment_sees_its_own_map():
    # two maps: a class-5 wall and a class-6 wall; env_map_id swaps them
    a = np.array(_wall(6.0, -20, 20, -10, 10), np.float32)
    b = np.array(_wall(9.0, -20, 20, -10, 10), np.float32)
    poses = np.zeros((3, 1, 3), np.float32)
    dims = np.tile(np.array(CAR, np.float32), (3, 1, 1))
    s = custom_scene(np.concatenate([a, b]), [5, 5, 6, 6], poses, dims, RIG16, 16, 16,
                     env_map_id=[1, 0, 1], map_tri_offset=[0, 2, 4])
    r = oracle.render(s)
    assert (r.cls[0] == 6).all() and (r.cls[1] == 5).all() and (r.cls[2] == 6).all()
    assert np.allclose(r.depth[0], 9.0) and np.allclose(r.depth[1], 6.0)
    assert (r.index[0] < 2).all()             # indices restart at 0 in every map


def test_grazing_plane_flag():
    # a huge ground-parallel sheet 5 cm below the camera: its plane passes the camera centre at
    # 0.05 m while its vertices are up to 85 m away (ratio 1 700) -> every pixel showing it is flagged
    # (only the first row below the horizon sees it beyond the near plane: z = 0.05 / (0.5/8) = 0.8 m)
    sheet = [[(0.25, -60.0, 0.95), (60.0, -60.0, 0.95), (60.0, 60.0, 0.95)], [(0.25, -60.0, 0.95), (60.0, 60.0, 0.95), (0.25, 60.0, 0.95)]]
    s = single_env(sheet, [5, 5], [ego()], rig=RIG16, H=16, W=16, far=100.0)
    r = oracle.render(s)
    on = r.cls[0] == 5
    assert on.sum() == 16 and on[8].all() and np.allclose(r.depth[0][8], 0.8)
    assert (r.flag[0][on] & 16).all() and (r.flag[0][~on] & 16).sum() == 0
    assert np.allclose(r.kappa[0][on], np.sqrt(60.0 ** 2 + 60.0 ** 2 + 0.05 ** 2) / 0.05, rtol=1e-6) and (r.kappa[0][~on] == 0).all()
    # the same sheet 1 m below the camera (ratio ~85) is an ordinary road: never flagged as grazing
    road = [[(1.0, -60.0, 0.0), (60.0, -60.0, 0.0), (60.0, 60.0, 0.0)], [(1.0, -60.0, 0.0), (60.0, 60.0, 0.0), (1.0, 60.0, 0.0)]]
    s = single_env(road, [2, 2], [ego()], rig=RIG16, H=16, W=16, far=100.0)
    r = oracle.render(s)
    assert (r.cls[0] == 2).sum() > 50 and (r.flag[0] & 16).sum() == 0
    assert np.allclose(r.kappa[0][r.cls[0] == 2], np.sqrt(7201.0), rtol=1e-9)       # farthest vertex / 1 m
    # and none of the benchmark workloads' pixels are (camera 1.5 m above the roads)
    r = oracle.render(make_config(0))
    assert (r.flag & 16).sum() == 0


# ------------------------------------------------------------------------------------------------
# occlusion counts (visible pixels of a road user / pixels its box would cover alone)
# ------------------------------------------------------------------------------------------------
def test_occlusion_counts_closed_forms():
    """Worked by hand on the one-box scene (camera 1.5 m high at the ego's box front, 64 x 64, fx = fy = 32): a car
    of the nominal size 12.5 m ahead shows its rear face 8 m in front of the camera as the rectangle rows 32..37 x
    columns 28..35 = 48 pixels; its other faces project inside that rectangle."""
    car = ego(12.5, 0.0, 0.0)
    # alone: fully visible
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), car])
    vis, un, sv, su = oracle.occlusion_counts(s, [0])
    assert vis[0].tolist() == [0, 48] and un[0].tolist() == [0, 48]
    # behind a wall that spans the whole image: fully hidden, but still 48 pixels when alone
    wall6 = [[(6.0, -40, -5), (6.0, 40, -5), (6.0, 40, 30)], [(6.0, -40, -5), (6.0, 40, 30), (6.0, -40, 30)]]
    s = single_env(wall6, [5, 5], [ego(), car])
    vis, un, *_ = oracle.occlusion_counts(s, [0])
    assert vis[0, 1] == 0 and un[0, 1] == 48
    # a wall 3.75 m ahead of the camera (x = 6) that ends at y = 0: at depth 3.75 its edge projects to the image
    # centre u = 32, and y > 0 is the left half -- columns 28..31 of the car are hidden, 32..35 stay: 4 x 6 = 24
    half = [[(6.0, 0.0, -5), (6.0, 40, -5), (6.0, 40, 30)], [(6.0, 0.0, -5), (6.0, 40, 30), (6.0, 0.0, 30)]]
    s = single_env(half, [5, 5], [ego(), car])
    r = oracle.render(s, [0])
    assert (r.cls[0][32:38, 28:32] == 5).all() and (r.cls[0][32:38, 32:36] == 4).all()
    vis, un, sv, su = oracle.occlusion_counts(s, [0])
    assert vis[0, 1] == 24 and un[0, 1] == 48
    # a second car right behind the first (20 m ahead): it projects to a smaller rectangle inside the first
    # one's footprint (rear face at 15.5 m: rows 32..34, half-width 0.95 * 32 / 15.5 = 1.96 px -> columns 30..33),
    # so all of it is hidden; the first car is untouched.  The ego itself and an inactive car count nothing.
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), car, ego(20.0, 0.0, 0.0), ego(30.0, 20.0, 0.0)], active=[1, 1, 1, 0])
    vis, un, *_ = oracle.occlusion_counts(s, [0])
    assert vis[0].tolist() == [0, 48, 0, 0] and un[0, 1] == 48 and un[0, 2] == 3 * 4 and un[0, 0] == 0 and un[0, 3] == 0
    # the counts of all road users add up to the vehicle-class pixels of the image
    s = make_config(2, E=1)
    views = [0, 5, 130, 255]
    vis, un, sv, su = oracle.occlusion_counts(s, views)
    r = oracle.render(s, views)
    assert (vis.sum(1) == (r.cls == 4).reshape(len(views), -1).sum(1)).all()
    assert (vis <= un + sv).all() and (un[vis > 0] > 0).all()
    assert ((un > 0).sum(1) >= (vis > 0).sum(1)).all() and (un > vis).any()     # heavy occlusion: somebody is partly hidden


# ------------------------------------------------------------------------------------------------
# road users with their own class; triangles with a limited angular range (traffic-light disks)
# ------------------------------------------------------------------------------------------------
def test_per_agent_classes():
    # the 48-pixel car 12.5 m ahead, as a pedestrian (class 7); a second agent keeps class 9; the sums still hold
    agents = np.array([ego(), ego(12.5, 0.0, 0.0), ego(14.0, 6.0, 0.0)])
    s = custom_scene(np.zeros((0, 3, 3)), [], agents[None, :, :3], agents[None, :, 3:], make_rig((0.0,), 90.0, 90.0), 64, 64,
                     agent_classes=[[5, 7, 9]])
    r = oracle.render(s, [0])
    assert (r.cls[0][32:38, 28:36] == 7).all() and (r.cls[0] == 7).sum() == 48
    assert (r.cls[0] == 9).sum() > 0 and (r.cls[0] == 4).sum() == 0 and (r.cls[0] == 5).sum() == 0
    vis, un, *_ = oracle.occlusion_counts(s, [0])
    assert vis[0, 1] == 48 and vis[0, 2] == (r.cls[0] == 9).sum()
    # seen from the third agent (view 2), the ego's own box shows the ego's class
    assert (oracle.render(s, [2]).cls[0] == 9).sum() == 0


def test_angular_range_of_one_sided_triangles():
    """A wall 10 m ahead whose normal points back at the camera (-x), drawn only within 30 degrees of that normal.
    8 x 8 image, fx = 4: camera at (0, L, 1) looking along +x.  Each of the wall's two triangles is judged from its
    own centroid; the wall is small (1 x 1 m around the axis at camera height), so both centroids sit within
    0.24 m of (10, 0, 1) and the angle is atan(L / 10) to within a degree and a half."""
    lim = np.cos(np.radians(30.0))
    # wound counter-clockwise when seen from -x (the camera's side): normal (V1-V0)x(V2-V0) = -x
    wall = [[(10.0, -0.5, 0.5), (10.0, -0.5, 1.5), (10.0, 0.5, 1.5)], [(10.0, -0.5, 0.5), (10.0, 0.5, 1.5), (10.0, 0.5, 0.5)]]
    n = np.cross(np.subtract(wall[0][1], wall[0][0]), np.subtract(wall[0][2], wall[0][0]))
    assert n[0] < 0 and n[1] == 0 and n[2] == 0
    rig = make_rig((0.0,), 90.0, 90.0, 64, 64, mount=(0.0, 0.0, 1.0))

    def seen(L, yaw, vis):
        s = single_env(wall, [5, 5], [ego(0.0, L, yaw)], rig=rig, tri_vis_cos=vis)
        r = oracle.render(s, [0])
        return int((r.cls[0] == 5).sum()), r

    for L, want in ((0.0, True), (4.0, True), (5.0, True), (6.5, False), (10.0, False)):     # 0, 21.8, 26.6, 33.0, 45 degrees
        yaw = np.arctan2(-L, 10.0)                                                         # keep the wall on the optical axis
        n_on, r = seen(L, yaw, [lim, lim])
        n_free, _ = seen(L, yaw, None)
        assert n_free > 0 and (n_on == n_free if want else n_on == 0), (L, n_on, n_free)
        assert (r.flag[0] & 32).sum() == 0
    # from behind it is never drawn, whatever the angle; without a limit it is two-sided
    s_back = single_env(wall, [5, 5], [ego(20.0, 0.0, np.pi)], rig=rig, tri_vis_cos=[lim, lim])
    assert (oracle.render(s_back, [0]).cls[0] == 5).sum() == 0
    s_back = single_env(wall, [5, 5], [ego(20.0, 0.0, np.pi)], rig=rig)
    assert (oracle.render(s_back, [0]).cls[0] == 5).sum() > 0
    # one triangle limited, the other not: only the limited one disappears at 45 degrees
    n_half, _ = seen(10.0, np.arctan2(-10.0, 10.0), [lim, 0.0])
    n_free, _ = seen(10.0, np.arctan2(-10.0, 10.0), None)
    assert 0 < n_half < n_free
    # exactly at the limit (the limit is set to the float32 of the first triangle's own cosine): decided by the exact
    # comparison, and every pixel the triangle covers is flagged; 1e-3 away from it nothing is flagged
    L = 5.0
    g = np.mean(np.asarray(wall[0], np.float64), axis=0)
    d = np.array([0.0, L, 1.0]) - g
    c_exact = float(-d[0] / np.linalg.norm(d))
    for delta, flagged in ((0.0, True), (3e-6, True), (-3e-6, True), (1e-3, False), (-1e-3, False)):
        s = single_env(wall[:1], [5], [ego(0.0, L, np.arctan2(-L, 10.0))], rig=rig, tri_vis_cos=[np.float32(c_exact + delta)])
        r = oracle.render(s, [0])
        drawn = (r.cls[0] == 5).sum()
        assert ((r.flag[0] & 32).sum() > 0) == flagged, (delta, drawn)
        if not flagged:
            assert (drawn > 0) == (delta < 0)


def test_traffic_light_disk():
    # a disk of radius 0.5 m, 8 m in front of the camera and facing it: a circle of radius 2 pixels (fx = 32) around
    # the image centre; pixel centres within it: the 12 with |du|, |dv| in {0.5, 1.5} and du^2 + dv^2 < 4
    rig = make_rig((0.0,), 90.0, 90.0, 64, 64, mount=(0.0, 0.0, 1.0))
    tris = disk_triangles((8.0, 0.0, 1.0), (-1.0, 0.0, 0.0), 0.5, n=64)
    lim = float(np.cos(np.radians(40.0)))
    s = single_env(tris, [6] * len(tris), [ego()], rig=rig, tri_vis_cos=[lim] * len(tris))
    r = oracle.render(s, [0])
    ys, xs = np.nonzero(r.cls[0] == 6)
    assert len(xs) == 12 and set(zip(xs.tolist(), ys.tolist())) == {(x, y) for x in range(30, 34) for y in range(30, 34)
                                                                    if (x + 0.5 - 32) ** 2 + (y + 0.5 - 32) ** 2 < 4}
    assert np.allclose(r.depth[0][r.cls[0] == 6], 8.0)
    # the ego turns away until the signal's centre is 50 degrees off its normal as seen from the disk: culled
    a = np.radians(50.0)
    s = single_env(tris, [6] * len(tris), [ego(8.0 - 8.0 * np.cos(a), 8.0 * np.sin(a), -a)], rig=rig, tri_vis_cos=[lim] * len(tris))
    assert (oracle.render(s, [0]).cls[0] == 6).sum() == 0
    s = single_env(tris, [6] * len(tris), [ego(8.0 - 8.0 * np.cos(a), 8.0 * np.sin(a), -a)], rig=rig)
    assert (oracle.render(s, [0]).cls[0] == 6).sum() > 0
