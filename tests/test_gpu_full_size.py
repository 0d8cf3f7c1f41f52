"""The benchmark workloads at their FULL sizes, in the launch configuration bench.py times:
sampled views against the oracle, and -- a property that holds at any size -- bit-equality of the
production kernel with the exhaustive kernel on a range of views.  Also the shapes that stress the
kernel's list capacities and multi-round paths."""
import numpy as np
import pytest

from scenes import make_config, make_rig, make_actions, custom_scene, DT, WHEELBASE, V_MAX
from tests.util import single_env, compare_images, assert_same_as_exhaustive

pytestmark = pytest.mark.gpu
CAR = (4.5, 1.9, 1.5)


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


def _sample_and_check(gu, s, n_oracle, n_brute, seed, env0_views=None):
    """Full-size run in the launch configuration the benchmark times (no float32 depth image: the full-tile
    kernels), compared with the oracle on `n_oracle` seeded views plus every view of environment 0; the same
    views once more with the float32 depth image (the general kernels) at the literal 1e-4 depth tolerance; and a
    window of `n_brute` views against the exhaustive kernel."""
    import oracle
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        cls, d16, _ = g.render(depth32=False)
        assert (cls != 255).all()                              # every view was written
        rng = np.random.default_rng(seed)
        views = np.union1d(rng.choice(V, size=n_oracle, replace=False), np.arange(s.A * s.K if env0_views is None else env0_views))
        ref = oracle.render(s, views)
        # the comparisons below are given no conditioning numbers: the depth tolerance tested on the benchmark
        # workloads is the literal 1e-4 everywhere, also on the handful of pixels whose winning plane grazes the
        # camera centre (mask bit 16, counted here)
        grazing = int(((ref.flag & 16) != 0).sum())
        assert grazing <= 1e-4 * ref.flag.size
        st = compare_images(ref.cls, ref.depth, ref.flag, cls[views], None, d16[views])
        cls32, d16b, d32 = g.render(depth32=True)
        assert (cls32 == cls).all() and (d16b.view(np.uint16) == d16.view(np.uint16)).all()
        compare_images(ref.cls, ref.depth, ref.flag, cls32[views], d32[views], d16b[views])
        del cls32, d16b, d32
        st["views"] = int(len(views)); st["grazing_pixels"] = grazing
        first = int(rng.integers(0, V - n_brute))
        a = g.render(view_first=first, view_count=n_brute)
        b = g.render(brute=True, view_first=first, view_count=n_brute)
        assert_same_as_exhaustive(a, b, slice(first, first + n_brute))
        assert (a[0][first:first + n_brute] == cls[first:first + n_brute]).all()
        return st
    finally:
        g.close()


def test_config1_full(gu):
    st = _sample_and_check(gu, make_config(1), n_oracle=512, n_brute=1024, seed=1)
    assert st["views"] >= 512 + 100
    print("cfg1 full", st)


def test_config2_full(gu):
    st = _sample_and_check(gu, make_config(2), n_oracle=512, n_brute=1024, seed=2)
    assert st["views"] >= 512 + 200
    print("cfg2 full", st)


def test_config3_full(gu):
    # (the oracle needs 0.8 s per 128 x 256 view of this 37 504-triangle map: 64 seeded views plus the 16 views
    # of environment 0's first four agents, not all 256 views of environment 0)
    st = _sample_and_check(gu, make_config(3), n_oracle=64, n_brute=48, seed=3, env0_views=16)
    assert st["views"] >= 64
    print("cfg3 full", st)


def _camera_inside_a_box(s, state, view):
    """Is the camera of `view` inside (or within 5 cm of) the box of another active agent of its environment?"""
    e, a, k = view // (s.A * s.K), (view // s.K) % s.A, view % s.K
    x, y, th = (float(t) for t in state[e, a, :3])
    mx, my, mz = (float(t) for t in s.rig[k, :3])
    cx, cy = x + np.cos(th) * mx - np.sin(th) * my, y + np.sin(th) * mx + np.cos(th) * my
    for b in range(s.A):
        if b == a or not s.active[e, b]:
            continue
        bx, by, bth = (float(t) for t in state[e, b, :3])
        dx, dy = cx - bx, cy - by
        u, v = np.cos(bth) * dx + np.sin(bth) * dy, -np.sin(bth) * dx + np.cos(bth) * dy
        if abs(u) <= 0.5 * s.dims[e, b, 0] + 0.05 and abs(v) <= 0.5 * s.dims[e, b, 1] + 0.05 and mz <= s.dims[e, b, 2] + 0.05:
            return True
    return False


def test_config4_full_hundred_steps(gu):
    import torch
    import oracle
    s = make_config(4)
    g = gu.CudaRun(s)
    try:
        dev = g.dev
        g.scene.set_state(torch.from_numpy(s.state()).to(dev), g.dims, g.active)
        cls, dep = g.scene.alloc_outputs()
        rng = np.random.default_rng(4)
        agents = np.sort(rng.choice(s.E * s.A, size=256, replace=False))
        st64 = s.state().astype(np.float64).reshape(-1, 4)[agents]
        n_inside = 0
        for step in range(1, 101):
            act = make_actions(4, step, s.E, s.A)
            g.scene.step(torch.from_numpy(act).to(dev), s.rig, cls, dep)
            st64 = oracle.step(st64, act.reshape(-1, 2)[agents], None, DT, WHEELBASE, V_MAX)
            if step in (1, 50, 100):
                got = g.scene.get_state().cpu().numpy()
                views = np.sort(rng.choice(s.E * s.A * s.K, size=128, replace=False))
                ref = oracle.render(s, views, poses=got[..., :3])
                c = cls.cpu().numpy().reshape(-1, s.H, s.W)[views]
                d = dep.cpu().numpy().reshape(-1, s.H, s.W)[views]
                # The protocol has no collision handling, so after some steps a few agents overlap.  A camera
                # that sits inside another agent's box looks at that box's bottom face from above, which is
                # coplanar with the road: a whole surface of exact depth ties between two classes.  Those
                # views are held to "every mismatch on a flagged pixel" only; all the others to the full rule.
                inside = np.array([_camera_inside_a_box(s, got, int(v)) for v in views])
                compare_images(ref.cls[~inside], ref.depth[~inside], ref.flag[~inside], c[~inside], None, None)
                if inside.any():
                    compare_images(ref.cls[inside], ref.depth[inside], ref.flag[inside], c[inside], None, None, max_mismatch_frac=1.0)
                n_inside += int(inside.sum())
                ok = (c == ref.cls) & (ref.flag == 0)
                ulp = np.abs(d.view(np.uint16).astype(np.int32) - ref.depth.astype(np.float16).view(np.uint16).astype(np.int32))
                assert (ulp[ok] <= 1).all()
                sub = got.reshape(-1, 4)[agents]
                assert np.abs(sub[:, :2] - st64[:, :2]).max() <= 1e-3
                assert np.abs((sub[:, 2] - st64[:, 2] + np.pi) % (2 * np.pi) - np.pi).max() <= 1e-5 * max(1.0, np.abs(st64[:, 2]).max())
                assert np.abs(sub[:, 3] - st64[:, 3]).max() <= 1e-4
        assert g.scene.status() == 0
        assert n_inside <= 12, "more than a handful of the 384 sampled cameras sit inside another agent's box"
    finally:
        g.close()


# ------------------------------------------------------------------------------------------------
# shapes that push the kernel's internal lists and rounds
# ------------------------------------------------------------------------------------------------
def test_many_large_primitives_overflow_the_lists(gu):
    # 400 big overlapping triangles right in front of the camera: far more survivors and records per
    # tile than the per-round lists hold
    rng = np.random.default_rng(11)
    n = 400
    centre = rng.uniform(-10, 10, size=(n, 1, 3)) * np.array([0.3, 1, 0.3]) + np.array([12.0, 0.0, 1.5])
    tris = centre + rng.uniform(-5, 5, size=(n, 3, 3))
    s = single_env(tris, rng.integers(2, 9, size=n), [(0, 0, 0) + CAR], near=0.5, far=60.0)
    st = gu.check_against_oracle(s, max_mismatch_frac=1e-3)
    g = gu.CudaRun(s)
    try:
        *_, cnt = g.render(counters=True)
        assert cnt[7] > 0, "expected the record list to overflow in this scene"
        assert_same_as_exhaustive(g.render(), g.render(brute=True))
    finally:
        g.close()


def test_many_agents_and_groups_take_several_rounds(gu):
    # 150 agents (three rounds of boxes) on a map of 24 groups (two rounds of groups)
    s0 = make_config(3, E=1)
    rng = np.random.default_rng(5)
    A = 150
    poses = np.zeros((1, A, 3), np.float32)
    poses[0, :, 0] = rng.uniform(-60, 60, A); poses[0, :, 1] = rng.uniform(-60, 60, A); poses[0, :, 2] = rng.uniform(-3, 3, A)
    keep = 6200 * 2                                           # triangles -> about 24 groups of 256 primitives
    dims = np.tile(np.array(CAR, np.float32), (1, A, 1))
    s = custom_scene(s0.tri_xyz[:keep], s0.tri_class[:keep], poses, dims, make_rig((0.0, 120.0), 90.0, 70.0, 96, 54),
                     54, 96, near=0.5, far=150.0)
    views = np.arange(0, 2 * A, 13)
    st = gu.check_against_oracle(s, view_ids=views)
    g = gu.CudaRun(s)
    try:
        assert_same_as_exhaustive(g.render(), g.render(brute=True))
    finally:
        g.close()


def test_degenerate_triangles_inactive_agents_and_sixteen_cameras(gu):
    rng = np.random.default_rng(3)
    good = rng.uniform(-8, 8, size=(20, 3, 3)) + np.array([10.0, 0.0, 2.0])
    dup = good[:5].copy(); dup[:, 2] = dup[:, 1]                       # two identical vertices
    line = np.stack([np.linspace(0, 1, 3)[:, None] * np.array([5.0, 3.0, 1.0]) + np.array([6.0, -2.0, 0.5])] * 3)
    point = np.full((2, 3, 3), 7.0)
    tris = np.concatenate([good, dup, line, point])
    rig = make_rig(tuple(np.arange(16) * 22.5), 90.0, 90.0, 32, 32)
    agents = [(0, 0, 0) + CAR, (9, 1, 0.5) + CAR, (5, -7, 2.0) + CAR]
    s = single_env(tris, rng.integers(2, 9, size=len(tris)), agents, rig=rig, H=32, W=32, far=50.0, active=[1, 0, 1])
    st = gu.check_against_oracle(s)
    cls = st["gpu"][0]
    assert (cls[16:32] == 0).all()                                    # the inactive agent's 16 views are sky
    import paper_2607_26005_b200 as pic
    with pytest.raises(pic.PicError):
        pic.Scene(1, 1, 17, 8, 8, 0.5, 100.0, [], [])


def test_large_ragged_image(gu):
    rng = np.random.default_rng(8)
    tris = rng.uniform(-10, 10, size=(40, 3, 3)) + np.array([14.0, 0.0, 2.0])
    rig = make_rig((0.0,), 100.0, 70.0, 330, 201, pitch_deg=-8.0)
    s = single_env(tris, rng.integers(2, 9, size=40), [(0, 0, 0) + CAR, (11, 2, 1.0) + CAR], rig=rig, H=201, W=330, far=60.0)
    gu.check_against_oracle(s, view_ids=[0])
