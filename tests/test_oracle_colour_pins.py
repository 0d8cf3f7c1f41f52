"""Pins of the oracle's colour output (O11) and analytic-coverage antialiasing (O12): closed forms, special
cases with hand values, an independent polygon-clipping area, invariants.  CPU only."""
import numpy as np
import pytest

import oracle
from scenes import make_config, make_rig, default_palette
from tests.util import single_env

CAR = (4.5, 1.9, 1.5)
PAL = default_palette()
SKY, GROUND, VEH = PAL[0].astype(float), PAL[1].astype(float), PAL[4].astype(float)
# 8 x 8 image, fx = fy = 4, camera at (0, 0, 1) looking along +x: a wall in the plane x = 4 shows one pixel per
# metre, column = 4 - y, row = 5 - z; rows 0..3 are sky, rows 4..7 ground
RIG8 = make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0))
RIG16 = make_rig((0.0,), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 1.0))


def ego(x=0.0, y=0.0, yaw=0.0, dims=CAR):
    return (x, y, yaw) + tuple(dims)


def wall(x, col0, col1, row0, row1, scale=1.0, centre=4.0):
    """Rectangle in the plane x = const covering image columns [col0, col1] and rows [row0, row1] (pixel
    coordinates of the image whose centre is `centre`; scale = metres per pixel at that depth): two triangles."""
    y0, y1 = (centre - col0) * scale, (centre - col1) * scale
    z0, z1 = 1.0 + (centre - row0) * scale, 1.0 + (centre - row1) * scale
    return [[(x, y0, z0), (x, y1, z0), (x, y1, z1)], [(x, y0, z0), (x, y1, z1), (x, y0, z1)]]


def bg(v):
    return SKY if v < 4 else GROUND


# ------------------------------------------------------------------------------------------------
# O12: coverage of a pixel by a half-plane -- closed forms and an independent clipped-polygon area
# ------------------------------------------------------------------------------------------------
def _clipped_area(e0, a, b):
    """Area of the unit square around the origin where e0 + a x + b y >= 0: Sutherland-Hodgman + shoelace."""
    poly = [(-0.5, -0.5), (0.5, -0.5), (0.5, 0.5), (-0.5, 0.5)]
    out = []
    for i in range(4):
        p, q = poly[i], poly[(i + 1) % 4]
        fp, fq = e0 + a * p[0] + b * p[1], e0 + a * q[0] + b * q[1]
        if fp >= 0:
            out.append(p)
        if (fp >= 0) != (fq >= 0):
            t = fp / (fp - fq)
            out.append((p[0] + t * (q[0] - p[0]), p[1] + t * (q[1] - p[1])))
    if len(out) < 3:
        return 0.0
    x, y = np.array(out).T
    return 0.5 * abs(np.dot(x, np.roll(y, -1)) - np.dot(y, np.roll(x, -1)))


def test_edge_coverage_closed_forms():
    cov = oracle.edge_coverage
    for d in (-0.5, -0.3, 0.0, 0.125, 0.5):                 # axis-aligned edge d pixels from the centre: 1/2 + d
        assert cov(d * 3.0, 3.0, 0.0) == pytest.approx(0.5 + d, abs=1e-15)
        assert cov(d * 0.7, 0.0, -0.7) == pytest.approx(0.5 + d, abs=1e-15)
    assert cov(0.0, 1.0, 1.0) == 0.5 and cov(0.0, 2.0, -5.0) == 0.5            # any line through the centre halves the pixel
    for s in (0.1, 0.5, 1.0):                               # 45 degrees: cuts a corner triangle with legs s off: area s^2 / 2
        assert cov(-1.0 + s, 1.0, 1.0) == pytest.approx(s * s / 2, abs=1e-15)
        assert cov(1.0 - s, 1.0, 1.0) == pytest.approx(1 - s * s / 2, abs=1e-15)
    assert cov(5.0, 1.0, 2.0) == 1.0 and cov(-5.0, 1.0, 2.0) == 0.0 and cov(1.5, 1.0, 2.0) == 1.0 and cov(-1.5, 1.0, 2.0) == 0.0
    assert cov(0.0, 0.0, 0.0) == 0.0 and cov(1e-9, 0.0, 0.0) == 1.0           # a constant: positive everywhere or nowhere
    # slope 1:2 through the lower left corner region: the line x + 2 y = -1 cuts the triangle (-.5,-.25) (-.5,-.5) (0,-.5): 1/16
    assert cov(1.0, 1.0, 2.0) == pytest.approx(1 - 1 / 16, abs=1e-15)


def test_pixel_coverage_of_three_edges():
    cov = oracle.pixel_coverage
    big = 10.0
    # one edge crossing, the other two far away: the one-edge closed form
    rng = np.random.default_rng(6)
    for _ in range(500):
        a, b = rng.normal(size=2)
        e0 = rng.uniform(-1, 1) * 0.7 * (abs(a) + abs(b))
        assert cov([e0, big, big], [a, 0, 0], [b, 0, 0]) == pytest.approx(oracle.edge_coverage(e0, a, b), abs=1e-12)
    # a corner: x >= -0.2 and y >= 0.1 -> 0.7 * 0.4; a strip 0.3 wide; a triangle that lies inside the pixel: its own area
    assert cov([0.2, -0.1, big], [1, 0, 0], [0, 1, 0]) == pytest.approx(0.28, abs=1e-15)
    assert cov([0.25, 0.05, big], [1, -1, 0], [0, 0, 0]) == pytest.approx(0.3, abs=1e-15)
    assert cov([0.25, 0.25, 0.1], [1, 0, -1], [0, 1, -1]) == pytest.approx(0.5 * 0.6 * 0.6, abs=1e-15)   # legs 0.6
    assert cov([-1, big, big], [1, 0, 0], [0, 0, 0]) == 0.0 and cov([big, big, big], [1, 2, 3], [3, 2, 1]) == 1.0
    # two triangles that share an edge cover the sum: the shared line's two sides
    for _ in range(200):
        e = rng.uniform(-0.5, 0.5, size=3); a = rng.normal(size=3); b = rng.normal(size=3)
        one = cov([e[0], e[1], big], [a[0], a[1], 0], [b[0], b[1], 0])
        two = cov(e, a, b) + cov([e[0], e[1], -e[2]], [a[0], a[1], -a[2]], [b[0], b[1], -b[2]])
        assert two == pytest.approx(one, abs=1e-12)


def test_edge_coverage_against_clipped_polygon_area():
    rng = np.random.default_rng(5)
    for _ in range(2000):
        a, b = rng.normal(size=2) * rng.choice([1e-3, 1.0, 50.0])
        if rng.random() < 0.1:
            b = 0.0
        e0 = rng.uniform(-1, 1) * 0.7 * (abs(a) + abs(b))
        got = oracle.edge_coverage(e0, a, b)
        assert got == pytest.approx(_clipped_area(e0, a, b), abs=1e-12)
        assert got + oracle.edge_coverage(-e0, -a, -b) == pytest.approx(1.0, abs=1e-12)   # the two sides of a line


# ------------------------------------------------------------------------------------------------
# O11: colour -- special cases with hand values (beta = 1 at near, 1/2 at far; the face factors)
# ------------------------------------------------------------------------------------------------
def _box_ahead(yaw, near, far, height=1.5, cls=None, mount_z=1.5):
    rig = make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, mount_z))
    other = (12.5, 0.0, yaw, 4.5, 1.9, height) if abs(np.sin(yaw)) < 0.5 else (12.5, 0.0, yaw, 1.9, 4.5, height)
    return single_env(np.zeros((0, 3, 3)), [], [ego(), other], rig=rig, near=near, far=far,
                      agent_classes=None if cls is None else np.array([[4, cls]], np.uint8))


def test_box_face_colours_at_near_and_far():
    # the box's facing face is 8 m ahead of the camera and covers rows 32..37, columns 28..35 (see the class pins)
    inside = (slice(33, 37), slice(29, 35))
    for aa in (False, True):
        # rear face (factor 0.60) exactly at near: beta = 1 -> 0.6 * (40, 110, 220) = (24, 66, 132), exactly
        r = oracle.render_rgb(_box_ahead(0.0, 8.0, 100.0), PAL, aa, view_ids=[0])
        assert (r.rgb[0][inside] == (24, 66, 132)).all()
        # ... and exactly at far: beta = 1/2 -> (12, 33, 66)
        r = oracle.render_rgb(_box_ahead(0.0, 0.5, 8.0), PAL, aa, view_ids=[0])
        assert (r.rgb[0][inside] == (12, 33, 66)).all()
        # near 0.5, far 15.5: beta(8) = 1 - 0.5 * 7.5 / 15 = 3/4.  Front face (1.00): the other car faces the ego
        r = oracle.render_rgb(_box_ahead(np.pi, 0.5, 15.5), PAL, aa, view_ids=[0])
        assert np.allclose(r.rgbf[0][inside], (30.0, 82.5, 165.0), atol=1e-5)
        # heading left: its left side (0.85) faces the ego; heading right: its right side (0.70)
        r = oracle.render_rgb(_box_ahead(np.pi / 2, 0.5, 15.5), PAL, aa, view_ids=[0])
        assert np.allclose(r.rgbf[0][inside], (25.5, 70.125, 140.25), atol=1e-5)
        r = oracle.render_rgb(_box_ahead(-np.pi / 2, 0.5, 15.5), PAL, aa, view_ids=[0])
        assert np.allclose(r.rgbf[0][inside], (21.0, 57.75, 115.5), atol=1e-5) and (r.rgb[0][inside][..., 1] == 58).all()
        # a pedestrian in its own hue
        r = oracle.render_rgb(_box_ahead(0.0, 8.0, 100.0, cls=8), PAL, aa, view_ids=[0])
        assert np.allclose(r.rgbf[0][inside], 0.6 * PAL[8].astype(float), atol=1e-9)
        # background: sky above the horizon row, ground below
        assert (r.rgb[0][:32, :20] == PAL[0]).all() and (r.rgb[0][40:, :20] == PAL[1]).all()


def test_top_face_and_depth_aware_brightness():
    # a 1 m high box seen from 4 m: its top (0.92) shows above its rear face (0.60); brightness falls linearly with depth
    r = oracle.render_rgb(_box_ahead(0.0, 0.5, 100.0, height=1.0, mount_z=4.0), PAL, False, view_ids=[0])
    ref = oracle.render(_box_ahead(0.0, 0.5, 100.0, height=1.0, mount_z=4.0), view_ids=[0])
    top = np.isin(ref.index[0], (12 + 10, 12 + 11)) & (ref.flag[0] == 0)
    rear = np.isin(ref.index[0], (12 + 0, 12 + 1)) & (ref.flag[0] == 0)
    assert top.sum() > 4 and rear.sum() > 20
    beta = 1 - 0.5 * (ref.depth[0] - 0.5) / 99.5
    assert np.allclose(r.rgbf[0][top], (0.92 * beta[top])[:, None] * VEH, atol=1e-9)
    assert np.allclose(r.rgbf[0][rear], (0.60 * beta[rear])[:, None] * VEH, atol=1e-9)
    z = ref.depth[0][top]
    assert z.max() > z.min() + 1.0          # the top recedes: its colour is not constant


def test_colour_without_antialiasing_follows_the_pinned_class_image():
    s = make_config(0)
    views = [0, 3]
    ref = oracle.render(s, views)
    r = oracle.render_rgb(s, PAL, False, views)
    for c in (0, 1, 2, 3):                                  # sky, ground, road, markings: the class's colour, unshaded
        m = ref.cls == c
        assert m.sum() > 0 and (r.rgb[m] == PAL[c]).all()
    veh = (ref.cls == 4)
    face = (ref.index[veh] - s.map_slice(0)[1]) % 12 // 2
    shade = np.array([0.60, 1.00, 0.70, 0.85, 0.40, 0.92])[face] * (1 - 0.5 * (ref.depth[veh] - s.near) / (s.far - s.near))
    assert np.allclose(r.rgbf[veh], shade[:, None] * VEH, atol=1e-9)
    assert ((r.flag & 47) == (ref.flag & 47))[~veh].all()   # same ambiguity mask where no box is involved


# ------------------------------------------------------------------------------------------------
# O12: antialiased images -- closed forms on an 8 x 8 image
# ------------------------------------------------------------------------------------------------
def test_rectangle_edges_cover_their_fraction_of_a_pixel():
    # wall over columns 2.3 .. 5.75 and rows 1.5 .. 6.25 (two triangles, class 7)
    s = single_env(wall(4.0, 2.3, 5.75, 1.5, 6.25), [7, 7], [ego()], rig=RIG8, H=8, W=8)
    r = oracle.render_rgb(s, PAL, True)
    img, w7 = r.rgbf[0], PAL[7].astype(float)
    for v in range(2, 6):                                   # left edge: column 2 is covered 0.7, right edge: column 5 by 0.75
        assert np.allclose(img[v, 2], 0.7 * w7 + 0.3 * bg(v), atol=1e-9)
        assert np.allclose(img[v, 5], 0.75 * w7 + 0.25 * bg(v), atol=1e-9)
        assert np.allclose(img[v, 3], w7, atol=1e-9) and np.allclose(img[v, 4], w7, atol=1e-9)   # inside, across the diagonal: no seam
        assert np.allclose(img[v, 1], bg(v), atol=1e-9) and np.allclose(img[v, 6], bg(v), atol=1e-9)
    for u in (3, 4):                                        # top edge: row 1 by 0.5, bottom edge: row 6 by 0.25
        assert np.allclose(img[1, u], 0.5 * w7 + 0.5 * SKY, atol=1e-9)
        assert np.allclose(img[6, u], 0.25 * w7 + 0.75 * GROUND, atol=1e-9)
    # corner pixels: the exact area cx cy of the rectangle inside the pixel, whichever way the diagonal runs
    for (v, u), cx, cy in (((1, 2), 0.7, 0.5), ((1, 5), 0.75, 0.5), ((6, 2), 0.7, 0.25), ((6, 5), 0.75, 0.25)):
        assert np.allclose(img[v, u], cx * cy * w7 + (1 - cx * cy) * bg(v), atol=1e-9)
    # without antialiasing the same pixels are all or nothing
    r0 = oracle.render_rgb(s, PAL, False)
    assert (r0.rgb[0][3, 2] == PAL[7]).all() and (r0.rgb[0][3, 5] == PAL[7]).all() and (r0.rgb[0][6, 3] == PAL[1]).all()


def test_a_strip_thinner_than_a_pixel_stays_visible():
    # a pole 0.2 pixels wide between columns 3.1 and 3.3: no pixel centre is covered
    s = single_env(wall(4.0, 3.1, 3.3, 0.0, 8.0), [6, 6], [ego()], rig=RIG8, H=8, W=8)
    r0 = oracle.render_rgb(s, PAL, False)
    assert all((r0.rgb[0][v, 3] == bg(v)).all() for v in range(8))            # vanishes without antialiasing
    r = oracle.render_rgb(s, PAL, True)
    for v in range(8):
        assert np.allclose(r.rgbf[0][v, 3], 0.2 * PAL[6] + 0.8 * bg(v), atol=1e-9)
        assert np.allclose(r.rgbf[0][v, 2], bg(v), atol=1e-9) and np.allclose(r.rgbf[0][v, 4], bg(v), atol=1e-9)
    # straddling two columns: 3.9 .. 4.1 gives 0.1 to each
    s = single_env(wall(4.0, 3.9, 4.1, 0.0, 8.0), [6, 6], [ego()], rig=RIG8, H=8, W=8)
    r = oracle.render_rgb(s, PAL, True)
    assert np.allclose(r.rgbf[0][2, 3], 0.1 * PAL[6] + 0.9 * SKY, atol=1e-9) and np.allclose(r.rgbf[0][2, 4], 0.1 * PAL[6] + 0.9 * SKY, atol=1e-9)


def test_layers_are_composited_front_to_back():
    # a pole (class 6) at depth 2 covering 0.2 of column 3, in front of a wall (class 7) at depth 4 whose left edge
    # covers 0.7 of the same column: 0.2 pole + 0.8 (0.7 wall + 0.3 background)
    pole = wall(2.0, 3.1, 3.3, 0.0, 8.0, scale=0.5)
    back = wall(4.0, 3.3, 7.0, 0.0, 8.0)
    for tris, classes in ((pole + back, [6, 6, 7, 7]), (back + pole, [7, 7, 6, 6])):     # whatever the order of the primitives
        r = oracle.render_rgb(single_env(tris, classes, [ego()], rig=RIG8, H=8, W=8), PAL, True)
        for v in range(8):
            assert np.allclose(r.rgbf[0][v, 3], 0.2 * PAL[6] + 0.8 * (0.7 * PAL[7] + 0.3 * bg(v)), atol=1e-9)
    # two pieces of ONE surface (same class) are complementary instead: 0.2 + 0.7 of the pixel, the rest background
    r = oracle.render_rgb(single_env(pole + back, [7, 7, 7, 7], [ego()], rig=RIG8, H=8, W=8), PAL, True)
    assert np.allclose(r.rgbf[0][2, 3], 0.9 * PAL[7] + 0.1 * SKY, atol=1e-9)
    # a layer never holds more than the whole pixel: the pole in front of a wall of its own class that covers the pixel
    # fully adds nothing (0.2 + 1 is capped at 1), and nothing behind the layer shows
    full = wall(4.0, 1.0, 7.0, 0.0, 8.0)
    hidden = wall(6.0, 0.0, 8.0, 0.0, 8.0, scale=1.5)
    r = oracle.render_rgb(single_env(pole + full + hidden, [7, 7, 7, 7, 6, 6], [ego()], rig=RIG8, H=8, W=8), PAL, True)
    assert np.allclose(r.rgbf[0][2, 3], PAL[7], atol=1e-9) and np.allclose(r.rgbf[0][5, 3], PAL[7], atol=1e-9)


def test_a_mesh_has_no_seams_and_does_not_depend_on_its_triangulation():
    # the same 5.1 x 4.2 pixel wall as 2 triangles and as a 3 x 3 grid of rectangles (18 triangles)
    c0, c1, r0_, r1 = 1.45, 6.55, 1.7, 5.9
    coarse = wall(4.0, c0, c1, r0_, r1)
    xs, ys = np.linspace(c0, c1, 4), np.linspace(r0_, r1, 4)
    fine = [t for i in range(3) for j in range(3) for t in wall(4.0, xs[i], xs[i + 1], ys[j], ys[j + 1])]
    a = oracle.render_rgb(single_env(coarse, [7] * 2, [ego()], rig=RIG8, H=8, W=8), PAL, True).rgbf[0]
    b = oracle.render_rgb(single_env(fine, [7] * 18, [ego()], rig=RIG8, H=8, W=8), PAL, True).rgbf[0]
    assert np.allclose(a[2:5, 2:6], PAL[7], atol=1e-9) and np.allclose(b[2:5, 2:6], PAL[7], atol=1e-9)
    assert np.allclose(a, b, atol=1e-9)                     # also in the pixels that hold a vertex, inside or on the outline


def test_coverage_adds_up_to_the_projected_area():
    # white square of side 6.37 pixels turned by 27 degrees in the plane x = 8 of a 16 x 16 image (one pixel per metre), black
    # background: the image's sum is the square's area
    pal = PAL.copy(); pal[0] = pal[1] = 0; pal[7] = 255
    side, ang = 6.37, np.deg2rad(27.0)
    c, s_ = np.cos(ang), np.sin(ang)
    pts = [(8.0 + side / 2 * (sx * c - sy * s_), 8.3 + side / 2 * (sx * s_ + sy * c)) for sx, sy in ((-1, -1), (1, -1), (1, 1), (-1, 1))]
    P = [(8.0, 8.0 - u, 1.0 + 8.0 - v) for u, v in pts]
    tris = [[P[0], P[1], P[2]], [P[0], P[2], P[3]]]
    r = oracle.render_rgb(single_env(tris, [7, 7], [ego()], rig=RIG16, H=16, W=16), pal, True)
    total = r.rgbf[0][..., 0].sum() / 255.0
    assert total == pytest.approx(side * side, abs=1e-5)        # (the vertices are float32)
    assert 0.0 <= r.rgbf[0].min() and r.rgbf[0].max() <= 255.0 + 1e-9


def test_box_edges_blend_the_two_faces_without_a_hole():
    # a red box turned by 40 degrees in front of a blue wall: along the edge between its two visible faces no blue shows,
    # on its silhouette blue and red mix, and inside a face antialiasing changes nothing
    pal = PAL.copy(); pal[4] = (200, 0, 0); pal[7] = (0, 0, 255); pal[0] = pal[1] = (0, 0, 255)
    rig = make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, 1.5))
    big = [[(30.0, 40.0, -10.0), (30.0, -40.0, -10.0), (30.0, -40.0, 30.0)], [(30.0, 40.0, -10.0), (30.0, -40.0, 30.0), (30.0, 40.0, 30.0)]]
    s = single_env(big, [7, 7], [ego(), (12.0, 0.3, np.deg2rad(40.0), 4.5, 1.9, 3.0)], rig=rig)
    ref = oracle.render(s, [0])
    r, r0 = oracle.render_rgb(s, pal, True, [0]), oracle.render_rgb(s, pal, False, [0])
    idx = ref.index[0]
    box = idx >= 2
    face = np.where(box, (idx - 2) % 12 // 2, -1)
    # pixels of the box whose four neighbours are all box pixels: a face's inside, or the edge between two faces
    inner = box.copy()
    inner[1:-1, 1:-1] &= box[:-2, 1:-1] & box[2:, 1:-1] & box[1:-1, :-2] & box[1:-1, 2:]
    inner[0, :] = inner[-1, :] = False; inner[:, 0] = inner[:, -1] = False
    assert inner.sum() > 100 and len(np.unique(face[inner])) >= 2
    assert np.allclose(r.rgbf[0][inner][:, 2], 0.0, atol=1e-9)               # no blue: the two faces' coverages add up to 1
    same = inner.copy()
    same[1:-1, 1:-1] &= (face[:-2, 1:-1] == face[1:-1, 1:-1]) & (face[2:, 1:-1] == face[1:-1, 1:-1]) & \
                        (face[1:-1, :-2] == face[1:-1, 1:-1]) & (face[1:-1, 2:] == face[1:-1, 1:-1])
    assert same.sum() > 50 and np.allclose(r.rgbf[0][same], r0.rgbf[0][same], atol=1e-9)
    between = inner & ~same                                   # the edge between the faces: a mix of the two reds
    assert between.sum() > 5 and (np.abs(r.rgbf[0][between] - r0.rgbf[0][between]).max(axis=1) > 1.0).any()
    rim = box & ~inner
    mixed = (r.rgbf[0][rim][:, 2] > 1.0) & (r.rgbf[0][rim][:, 0] > 1.0)
    assert mixed.mean() > 0.5                                 # the silhouette mixes red and blue


def test_antialiasing_changes_only_pixels_next_to_an_edge_and_flags_are_rare():
    s = make_config(0)
    views = [0, 5]
    ref = oracle.render(s, views)
    a, b = oracle.render_rgb(s, PAL, True, views), oracle.render_rgb(s, PAL, False, views)
    idx = ref.index
    same = np.ones(idx.shape, bool)
    for dv in (-1, 0, 1):
        for du in (-1, 0, 1):
            same &= np.roll(np.roll(idx, dv, 1), du, 2) == idx
    same[:, 0, :] = same[:, -1, :] = False; same[:, :, 0] = same[:, :, -1] = False
    # where the 3 x 3 neighbourhood shows one primitive (or none), the pixel is covered fully by it -- except that a
    # primitive thinner than a pixel may hide between the centres: allow a few
    diff = np.abs(a.rgbf - b.rgbf).max(axis=-1)
    assert same.mean() > 0.5 and (diff[same] > 0.5).mean() < 0.02
    assert (diff[~same] > 0.5).mean() > 0.2
    assert (a.flag != 0).mean() < 5e-3 and (a.flag & 1).sum() == 0


def test_coverage_is_cut_at_the_near_and_far_planes_inside_a_pixel():
    # a road quad on the ground from 1 m to 50 m ahead, camera 1 m up, fy = 4: depth d shows at row 4 + 4 / d.
    # far = 8 falls on row 4.5 and near = 1.6 on row 6.5, the middles of pixel rows 4 and 6: half of each is in range
    quad = [[(1.0, 30.0, 0.0), (50.0, 30.0, 0.0), (50.0, -30.0, 0.0)], [(1.0, 30.0, 0.0), (50.0, -30.0, 0.0), (1.0, -30.0, 0.0)]]
    s = single_env(quad, [2, 2], [ego()], rig=RIG8, H=8, W=8, near=1.6, far=8.0)
    r = oracle.render_rgb(s, PAL, True)
    road = PAL[2].astype(float)
    for u in range(8):
        assert np.allclose(r.rgbf[0][4, u], 0.5 * road + 0.5 * GROUND, atol=1e-6)
        assert np.allclose(r.rgbf[0][5, u], road, atol=1e-9)
        assert np.allclose(r.rgbf[0][6, u], 0.5 * road + 0.5 * GROUND, atol=1e-6)
        assert np.allclose(r.rgbf[0][7, u], GROUND, atol=1e-9) and np.allclose(r.rgbf[0][3, u], SKY, atol=1e-9)
    # whether the quad ends at the far plane or runs on beyond it makes no difference
    cut = [[(1.0, 30.0, 0.0), (8.0, 30.0, 0.0), (8.0, -30.0, 0.0)], [(1.0, 30.0, 0.0), (8.0, -30.0, 0.0), (1.0, -30.0, 0.0)]]
    r2 = oracle.render_rgb(single_env(cut, [2, 2], [ego()], rig=RIG8, H=8, W=8, near=1.6, far=8.0), PAL, True)
    assert np.allclose(r.rgbf, r2.rgbf, atol=1e-6)
