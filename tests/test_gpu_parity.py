"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element."""
import numpy as np
import pytest

from scenes import make_config, make_rig, custom_scene, make_actions, DT, WHEELBASE, V_MAX
from tests.util import single_env, compare_images, assert_same_as_exhaustive

pytestmark = pytest.mark.gpu

CAR = (4.5, 1.9, 1.5)


def ego(x=0.0, y=0.0, yaw=0.0, dims=CAR):
    return (x, y, yaw) + tuple(dims)


def _wall(x, y0, y1, z0, z1):
    return [[(x, y0, z0), (x, y1, z0), (x, y1, z1)], [(x, y0, z0), (x, y1, z1), (x, y0, z1)]]


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


# ------------------------------------------------------------------------------------------------
# exact small cases (the same closed forms that pin the oracle)
# ------------------------------------------------------------------------------------------------
def test_empty_scene_exact(gu):
    s = single_env(np.zeros((0, 3, 3)), [], [ego()])
    st = gu.check_against_oracle(s)
    cls, d16, d32 = st["gpu"]
    assert st["mismatches"] == 0
    assert (cls[0][:32] == 0).all() and (cls[0][32:] == 1).all()
    assert d16[0][34, 0] == np.float16(19.203125) and d16[0][0, 0] == np.float16(100.0)


@pytest.mark.parametrize("kw", [dict(), dict(width=1.75), dict(height=1.375), dict(mount_z=1.375)])
def test_one_box_and_fill_rule_exact(gu, kw):
    width, height, mount_z = kw.get("width", 1.9), kw.get("height", 1.5), kw.get("mount_z", 1.5)
    rig = make_rig((0.0,), 90.0, 90.0, mount=(2.25, 0.0, mount_z))
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), (12.5, 0.0, 0.0, 4.5, width, height)], rig=rig)
    st = gu.check_against_oracle(s)
    # all quantities are exact in binary: no mismatch is tolerated, flagged or not
    assert st["mismatches"] == 0
    cls = st["gpu"][0]
    assert (cls[0] == 4).sum() == (st["ref"].cls[0] == 4).sum() > 0
    assert (cls[1] != 4).all()


def test_hand_scenes_exact(gu):
    rig8 = make_rig((0.0,), 90.0, 90.0, 8, 8, mount=(0.0, 0.0, 1.0))
    cases = [
        ([[(4.0, 2.0, 3.0), (4.0, -2.0, 3.0), (4.0, 2.0, -1.0)]], [7]),
        (_wall(8.0, -6.0, 6.0, -3.0, 5.0) + _wall(4.0, -1.0, 1.0, 0.0, 2.0), [5, 5, 6, 6]),
        (_wall(4.0, -2.0, 2.0, -1.0, 3.0) + _wall(4.0, -1.0, 3.0, 0.0, 4.0), [5, 5, 6, 6]),     # exact depth tie
        (_wall(4.0, -1.0, 3.0, 0.0, 4.0) + _wall(4.0, -2.0, 2.0, -1.0, 3.0), [6, 6, 5, 5]),
        (_wall(0.5, -4, 4, -3, 5), [5, 5]),                                                       # on the near plane
        (_wall(0.4375, -4, 4, -3, 5), [5, 5]),
    ]
    for tris, classes in cases:
        s = single_env(tris, classes, [ego()], rig=rig8, H=8, W=8)
        st = gu.check_against_oracle(s)
        # ties and plane hits are flagged by the oracle, yet these inputs are exact: demand equality
        assert (st["gpu"][0] == st["ref"].cls).all(), (tris, st["gpu"][0], st["ref"].cls)
    for far, x in ((64.0, 64.0), (64.0, 64.5)):
        s = single_env(_wall(x, -400, 400, -300, 500), [5, 5], [ego()], rig=rig8, H=8, W=8, near=0.5, far=far)
        st = gu.check_against_oracle(s)
        assert (st["gpu"][0] == st["ref"].cls).all()


def test_strip_through_camera_plane(gu):
    rig = make_rig((0.0,), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 1.0))
    strip = [[(-10.0, -1.0, 0.0), (20.0, -1.0, 0.0), (20.0, 1.0, 0.0)], [(-10.0, -1.0, 0.0), (20.0, 1.0, 0.0), (-10.0, 1.0, 0.0)]]
    s = single_env(strip, [2, 2], [ego()], rig=rig, H=16, W=16)
    st = gu.check_against_oracle(s)
    assert (st["gpu"][0] == st["ref"].cls).all()


def test_ego_excluded_inactive_and_shared_map(gu):
    rig = make_rig((0.0,), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 0.75))
    s = single_env(np.zeros((0, 3, 3)), [], [ego(), (10.0, 0.0, 0.0) + CAR], rig=rig, H=16, W=16, active=[1, 0])
    st = gu.check_against_oracle(s)
    cls, d16, _ = st["gpu"]
    assert (cls[0] != 4).all() and (cls[1] == 0).all() and (d16[1] == np.float16(100.0)).all()
    poses = np.array([[[0, 0, 0]], [[10, 0, 0]]], np.float32)
    dims = np.tile(np.array(CAR, np.float32), (2, 1, 1))
    s3 = custom_scene(np.zeros((0, 3, 3)), [], poses, dims, rig, 16, 16)
    st = gu.check_against_oracle(s3)
    assert (st["gpu"][0] != 4).all()


# ------------------------------------------------------------------------------------------------
# random triangle soups: general planes, camera-plane crossings, pitch, ragged image sizes
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed,H,W", [(0, 64, 64), (1, 54, 96), (2, 70, 100), (3, 128, 256), (4, 17, 33)])
def test_triangle_soup(gu, seed, H, W):
    rng = np.random.default_rng(seed)
    n = 60
    centre = rng.uniform(-15, 15, size=(n, 1, 3)) * np.array([1, 1, 0.2]) + np.array([8.0, 0.0, 1.0])
    tris = centre + rng.uniform(-6, 6, size=(n, 3, 3)) * np.array([1, 1, 0.5])
    classes = rng.integers(2, 9, size=n)
    rig = make_rig((10.0, -95.0), 80.0, 60.0, W, H, mount=(0.7, -0.3, 1.2), pitch_deg=float(rng.uniform(-15, 15)))
    agents = [ego(rng.uniform(-2, 2), rng.uniform(-2, 2), rng.uniform(-3, 3)), (9.0, 2.0, 0.4) + CAR, (4.0, -6.0, 2.0) + CAR]
    s = single_env(tris, classes, agents, rig=rig, H=H, W=W, near=0.5, far=40.0)
    st = gu.check_against_oracle(s, max_mismatch_frac=1e-3)
    assert st["flagged"] < 0.02 * st["pixels"]


# ------------------------------------------------------------------------------------------------
# the benchmark workloads at sizes the oracle finishes in seconds
# ------------------------------------------------------------------------------------------------
def test_cfg0_full(gu):
    s = make_config(0)
    st = gu.check_against_oracle(s)
    print("cfg0", {k: v for k, v in st.items() if k not in ("ref", "gpu")})


@pytest.mark.parametrize("cfg,E,n_sample", [(1, 3, 96), (2, 2, 96), (3, 1, 12)])
def test_cfg_sampled_views(gu, cfg, E, n_sample):
    s = make_config(cfg, E=E)
    rng = np.random.default_rng(cfg)
    V = s.E * s.A * s.K
    views = np.unique(np.concatenate([np.arange(s.K * 2), rng.choice(V, size=n_sample, replace=False)]))
    st = gu.check_against_oracle(s, view_ids=views)
    print(f"cfg{cfg}", {k: v for k, v in st.items() if k not in ("ref", "gpu")})
    assert st["flagged"] < 5e-3 * st["pixels"]


@pytest.mark.parametrize("cfg,E", [(1, 4), (2, 4), (3, 2)])
def test_production_kernel_equals_exhaustive_kernel(gu, cfg, E):
    """Culling, binning and the small/large split must not change a single bit."""
    s = make_config(cfg, E=E)
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        count = V if cfg != 3 else 64
        a = g.render(brute=False, view_first=0, view_count=count)
        b = g.render(brute=True, view_first=0, view_count=count)
        assert_same_as_exhaustive(a, b, slice(0, count))
        if count < V:
            assert (a[0][count:] == 255).all()          # views outside the range are left untouched
        # switching the kernel's shortcuts off / forcing its overflow path must not change the image
        for flags in (1, 2, 3, 4, 8, 9):
            c = g.render(brute=False, view_first=0, view_count=count, debug_flags=flags)
            assert (a[0][:count] == c[0][:count]).all() and (a[2][:count] == c[2][:count]).all()
    finally:
        g.close()


def test_determinism_and_host_entry_point(gu):
    import torch
    s = make_config(1, E=2)
    g = gu.CudaRun(s)
    try:
        a = g.render(depth32=False)
        b = g.render(depth32=False)
        assert (a[0] == b[0]).all() and (a[1].view(np.uint16) == b[1].view(np.uint16)).all()
        V = s.E * s.A * s.K
        oc = np.empty((V, s.H, s.W), np.uint8)
        od = np.empty((V, s.H, s.W), np.float16)
        g.scene.render_host(np.ascontiguousarray(s.poses), np.ascontiguousarray(s.dims), s.rig, oc, od,
                            active=np.ascontiguousarray(s.active))
        assert (oc == a[0]).all() and (od.view(np.uint16) == a[1].view(np.uint16)).all()
    finally:
        g.close()


def test_counters_are_plausible(gu):
    s = make_config(2, E=1)
    g = gu.CudaRun(s)
    try:
        *_, cnt = g.render(counters=True)
        V = s.E * s.A * s.K
        assert cnt[0] == V
        # tiles, group tests, leaf tests, primitives tested, set up, rasterized by their thread, records,
        # record-list overflows, records classified per cell, cells visited
        # (a record may be classified once per 16-row strip it reaches)
        assert 0 < cnt[4] <= cnt[3] and cnt[5] + cnt[6] + cnt[7] == cnt[4] and cnt[7] == 0 and cnt[8] <= 4 * cnt[6] and cnt[6] <= cnt[9]
        print("counters per view:", (cnt / V).round(1).tolist())
        # [10]: tiles the fused kernel left to the cooperative kernel -- a few at most here, all of
        # them when the test aid asks for it, and the work counts of both routes agree
        assert cnt[10] <= 0.2 * V
        *_, cnt_coop = g.render(counters=True, debug_flags=4)
        assert cnt_coop[0] == V and cnt_coop[10] == V
        # both routes set up the same primitives; the cull kernel finds its candidates through the uniform grid,
        # the cooperative kernel through the box hierarchy, so the numbers of candidates tested differ
        assert cnt_coop[4] == cnt[4] and 0 < cnt[3] < cnt_coop[3]
    finally:
        g.close()


# ------------------------------------------------------------------------------------------------
# pic_step: kinematic update + render
# ------------------------------------------------------------------------------------------------
def test_step_state_and_images(gu):
    import torch
    import oracle
    s = make_config(4, E=2)
    g = gu.CudaRun(s)
    try:
        dev = g.dev
        st64 = s.state().astype(np.float64)
        g.scene.set_state(torch.from_numpy(s.state()).to(dev), g.dims, g.active)
        cls, dep = g.scene.alloc_outputs()
        rng = np.random.default_rng(0)
        views = rng.choice(s.E * s.A * s.K, size=24, replace=False)
        for step in range(1, 101):
            act = make_actions(4, step, s.E, s.A)
            g.scene.step(torch.from_numpy(act).to(dev), s.rig, cls, dep)
            st64 = oracle.step(st64, act, s.active, DT, WHEELBASE, V_MAX)
            if step in (1, 50, 100):
                got = g.scene.get_state().cpu().numpy()
                # image parity from the GPU's own post-update state, so integrator drift is kept out of it
                ref = oracle.render(s, views, poses=got[..., :3])
                c = cls.cpu().numpy().reshape(-1, s.H, s.W)[views]
                d = dep.cpu().numpy().reshape(-1, s.H, s.W)[views]
                compare_images(ref.cls, ref.depth, ref.flag, c, None, None)
                ok = c == ref.cls
                ref16 = ref.depth.astype(np.float16)
                ulp = np.abs(d.view(np.uint16).astype(np.int32) - ref16.view(np.uint16).astype(np.int32))
                assert (ulp[ok & (ref.flag == 0)] <= 1).all()
                # state against the double-precision integration
                assert np.abs(got[..., 0] - st64[..., 0]).max() <= 1e-3
                assert np.abs(got[..., 1] - st64[..., 1]).max() <= 1e-3
                dth = np.abs((got[..., 2] - st64[..., 2] + np.pi) % (2 * np.pi) - np.pi)
                assert dth.max() <= 1e-5 * max(1.0, np.abs(st64[..., 2]).max())
                assert np.abs(got[..., 3] - st64[..., 3]).max() <= 1e-4
        assert g.scene.status() == 0
    finally:
        g.close()


# ------------------------------------------------------------------------------------------------
# error behaviour: return codes, never a fault
# ------------------------------------------------------------------------------------------------
def test_error_codes(gu):
    import torch
    import paper_2607_26005_b200 as pic
    with pytest.raises(pic.PicError) as ei:
        pic.Scene(0, 1, 1, 8, 8, 0.5, 100.0, [], [])
    assert ei.value.status == 2
    with pytest.raises(pic.PicError) as ei:
        pic.Scene(1, 1, 1, 8, 8, 0.5, 0.25, [], [])
    assert ei.value.status == 1
    with pytest.raises(pic.PicError) as ei:
        pic.Scene(1, 1, 1, 8, 8, 0.5, 100.0, np.full((1, 3, 3), np.nan), [2])
    assert ei.value.status == 1
    with pytest.raises(pic.PicError):
        pic.Scene(2, 1, 1, 8, 8, 0.5, 100.0, np.zeros((2, 3, 3)), [2, 2], map_tri_offset=[0, 2], env_map_id=[0, 1])
    s = single_env(np.zeros((0, 3, 3)), [], [ego()], H=16, W=16, rig=make_rig((0.0,), 90.0, 90.0, 16, 16))
    g = gu.CudaRun(s)
    try:
        cls, dep = g.scene.alloc_outputs()
        bad_rig = s.rig.copy(); bad_rig[0, 5] = 0.0
        with pytest.raises(pic.PicError) as ei:
            g.scene.render(g.poses, g.dims, bad_rig, out_class=cls, out_depth=dep)
        assert ei.value.status == 1
        # a non-finite pose is reported through the sticky flag and the call still completes
        poses = g.poses.clone(); poses[0, 0, 0] = float("nan")
        g.scene.render(poses, g.dims, s.rig, out_class=cls, out_depth=dep)
        assert g.scene.status() & pic.FLAG_NONFINITE_POSE
        assert g.scene.status() == 0
        assert (cls.cpu().numpy() == 0).all()          # that agent is treated as inactive: sky
        # a non-finite action (or a step that overflows) is flagged as well; the agent keeps its state and
        # is drawn as sky for that step, and a finite action afterwards moves it again
        state0 = torch.tensor([[[1.0, 2.0, 0.3, 5.0]]], dtype=torch.float32, device=g.dev)
        g.scene.set_state(state0, g.dims)
        for bad in ((float("nan"), 0.0), (0.0, float("nan")), (float("inf"), 0.0), (0.0, float("inf"))):
            act = torch.tensor([[list(bad)]], dtype=torch.float32, device=g.dev)
            cls.fill_(7)
            g.scene.step(act, s.rig, cls, dep)
            assert g.scene.status() & pic.FLAG_NONFINITE_POSE
            assert torch.equal(g.scene.get_state(), state0)
            assert (cls.cpu().numpy() == 0).all()
        g.scene.step(torch.zeros((1, 1, 2), dtype=torch.float32, device=g.dev), s.rig, cls, dep)
        assert g.scene.status() == 0
        moved = g.scene.get_state().cpu().numpy()[0, 0]
        assert abs(moved[0] - (1.0 + 5.0 * np.cos(0.3) * 0.1)) < 1e-5 and moved[3] == 5.0
        assert (cls.cpu().numpy()[..., 8:, :] == 1).all()      # an empty scene below the horizon: ground
    finally:
        g.close()


def test_environment_to_map_assignment_and_tied_boxes(gu):
    a = np.array(_wall(6.0, -20, 20, -10, 10), np.float32)
    b = np.array(_wall(9.0, -20, 20, -10, 10), np.float32)
    rig = make_rig((0.0, 180.0), 90.0, 90.0, 16, 16, mount=(0.0, 0.0, 1.0))
    poses = np.zeros((3, 1, 3), np.float32)
    dims = np.tile(np.array(CAR, np.float32), (3, 1, 1))
    s = custom_scene(np.concatenate([a, b]), [5, 5, 6, 6], poses, dims, rig, 16, 16, env_map_id=[1, 0, 1],
                     map_tri_offset=[0, 2, 4])
    st = gu.check_against_oracle(s)
    cls = st["gpu"][0]
    assert (cls[0] == 6).all() and (cls[2] == 5).all() and (cls[4] == 6).all()
    # identical boxes at one pose: exact ties everywhere on them, resolved identically on both sides
    agents = [ego(), (12.5, 0.0, 0.0) + CAR, (12.5, 0.0, 0.0) + CAR]
    s = single_env([[(50.0, -1.0, 0.0), (51.0, -1.0, 0.0), (51.0, 1.0, 0.0)]], [2], agents)
    st = gu.check_against_oracle(s)
    assert (st["gpu"][0] == st["ref"].cls).all()
