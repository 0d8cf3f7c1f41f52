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


def _sample_and_check(gu, s, n_oracle, n_brute, seed):
    import oracle
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        cls, d16, _ = g.render(depth32=False)
        assert (cls != 255).all()                              # every view was written
        rng = np.random.default_rng(seed)
        views = np.sort(rng.choice(V, size=n_oracle, replace=False))
        ref = oracle.render(s, views)
        st = compare_images(ref.cls, ref.depth, ref.flag, cls[views], None, d16[views], ref_kappa=ref.kappa)
        first = int(rng.integers(0, V - n_brute))
        a = g.render(view_first=first, view_count=n_brute)
        b = g.render(brute=True, view_first=first, view_count=n_brute)
        assert_same_as_exhaustive(a, b, slice(first, first + n_brute))
        assert (a[0][first:first + n_brute] == cls[first:first + n_brute]).all()
        return st
    finally:
        g.close()


def test_config1_full(gu):
    st = _sample_and_check(gu, make_config(1), n_oracle=96, n_brute=1024, seed=1)
    print("cfg1 full", st)


def test_config2_full(gu):
    st = _sample_and_check(gu, make_config(2), n_oracle=96, n_brute=1024, seed=2)
    print("cfg2 full", st)


def test_config3_full(gu):
    st = _sample_and_check(gu, make_config(3), n_oracle=12, n_brute=48, seed=3)
    print("cfg3 full", st)


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
        for step in range(1, 101):
            act = make_actions(4, step, s.E, s.A)
            g.scene.step(torch.from_numpy(act).to(dev), s.rig, cls, dep)
            st64 = oracle.step(st64, act.reshape(-1, 2)[agents], None, DT, WHEELBASE, V_MAX)
            if step in (1, 50, 100):
                got = g.scene.get_state().cpu().numpy()
                views = np.sort(rng.choice(s.E * s.A * s.K, size=16, replace=False))
                ref = oracle.render(s, views, poses=got[..., :3])
                c = cls.cpu().numpy().reshape(-1, s.H, s.W)[views]
                d = dep.cpu().numpy().reshape(-1, s.H, s.W)[views]
                compare_images(ref.cls, ref.depth, ref.flag, c, None, None)
                ok = (c == ref.cls) & (ref.flag == 0)
                ulp = np.abs(d.view(np.uint16).astype(np.int32) - ref.depth.astype(np.float16).view(np.uint16).astype(np.int32))
                assert (ulp[ok] <= 1).all()
                sub = got.reshape(-1, 4)[agents]
                assert np.abs(sub[:, :2] - st64[:, :2]).max() <= 1e-3
                assert np.abs((sub[:, 2] - st64[:, 2] + np.pi) % (2 * np.pi) - np.pi).max() <= 1e-5 * max(1.0, np.abs(st64[:, 2]).max())
                assert np.abs(sub[:, 3] - st64[:, 3]).max() <= 1e-4
        assert g.scene.status() == 0
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
