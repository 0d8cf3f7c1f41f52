"""Road users with their own class and triangles with a limited angular range (traffic-light disks as fans),
through the C ABI against the oracle: every kernel that sets a primitive up -- the full-tile kernels, the general
kernels, the cooperative kernel alone, the exhaustive kernel -- must drop a triangle outside its range alike and
write each agent's own class."""
import numpy as np
import pytest

from scenes import make_config, custom_scene, disk_triangles, make_rig
from tests.util import assert_same_as_exhaustive

pytestmark = pytest.mark.gpu
CAR = (4.5, 1.9, 1.5)


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


def _signals(rng, gm_scene, n):
    """n traffic-light disks (radius 0.4 m, 5 m above the road) over a scene's map, each facing a random heading,
    visible within 35 degrees of that heading; returns (triangles, classes, limits)."""
    tris, lim = [], []
    lo = gm_scene.tri_xyz[..., :2].reshape(-1, 2).min(0); hi = gm_scene.tri_xyz[..., :2].reshape(-1, 2).max(0)
    for _ in range(n):
        c = np.array([rng.uniform(lo[0], hi[0]), rng.uniform(lo[1], hi[1]), 5.0])
        a = rng.uniform(-np.pi, np.pi)
        t = disk_triangles(c, (np.cos(a), np.sin(a), 0.0), 0.4, n=8)
        tris.append(t); lim += [np.cos(np.radians(35.0))] * len(t)
    return np.concatenate(tris), np.full(sum(len(t) for t in tris), 6, np.uint8), np.asarray(lim, np.float32)


def test_platoons_with_pedestrians_cyclists_and_signals(gu):
    base = make_config(2, E=2)
    rng = np.random.default_rng(5)
    # signals near the agents so that some are in view: one in front of every fourth agent, facing it or not
    tris, cls, lim = [], [], []
    for e in range(base.E):
        t0, t1 = base.map_slice(e)
        et, el = [base.tri_xyz[t0:t1]], [np.zeros(t1 - t0, np.float32)]
        for a in range(0, base.A, 4):
            x, y, th = base.poses[e, a]
            d = rng.uniform(10.0, 40.0)
            c = np.array([x + d * np.cos(th) + rng.uniform(-3, 3), y + d * np.sin(th) + rng.uniform(-3, 3), rng.uniform(1.0, 5.0)])
            facing = th + np.pi + rng.uniform(-1.2, 1.2)           # roughly back at the agent, up to 69 degrees off
            t = disk_triangles(c, (np.cos(facing), np.sin(facing), 0.0), 0.6, n=8)
            et.append(t); el.append(np.full(len(t), np.cos(np.radians(35.0)), np.float32))
        tris.append(np.concatenate(et)); lim.append(np.concatenate(el))
        cls.append(np.concatenate([base.tri_class[t0:t1], np.full(len(tris[-1]) - (t1 - t0), 6, np.uint8)]))
    counts = [len(t) for t in tris]
    agent_classes = rng.choice([4, 7, 8], size=(base.E, base.A), p=[0.8, 0.1, 0.1]).astype(np.uint8)   # vehicle, pedestrian, cyclist
    s = custom_scene(np.concatenate(tris), np.concatenate(cls), base.poses, base.dims, base.rig, base.H, base.W, base.near, base.far,
                     map_tri_offset=np.concatenate([[0], np.cumsum(counts)]), env_map_id=[0, 1], agent_classes=agent_classes,
                     tri_vis_cos=np.concatenate(lim))
    views = np.arange(0, s.E * s.A * s.K, 3)
    st = gu.check_against_oracle(s, view_ids=views)
    ref = st["ref"]
    print("road users and signals:", {k: v for k, v in st.items() if k not in ("ref", "gpu")},
          "signal pixels", int((ref.cls == 6).sum()), "pedestrian/cyclist pixels", int(np.isin(ref.cls, (7, 8)).sum()))
    assert (ref.cls == 6).sum() > 20 and np.isin(ref.cls, (7, 8)).sum() > 100
    # the same scene without the limits shows more signal pixels: some disks are culled by their angular range
    s_free = custom_scene(s.tri_xyz, s.tri_class, s.poses, s.dims, s.rig, s.H, s.W, s.near, s.far, map_tri_offset=s.map_tri_offset,
                          env_map_id=[0, 1], agent_classes=agent_classes)
    import oracle
    assert (oracle.render(s_free, views).cls == 6).sum() > (ref.cls == 6).sum()
    g = gu.CudaRun(s)
    try:
        a = g.render()
        assert_same_as_exhaustive(a, g.render(brute=True))
        assert_same_as_exhaustive(g.render(debug_flags=4), a)          # the cooperative kernel alone
        # back to one class for all: the scene-wide class again
        g.scene.set_agent_classes(None)
        c0 = g.render()[0]
        assert not np.isin(c0, (7, 8)).any() and ((c0 == 4) == np.isin(a[0], (4, 7, 8))).all()
    finally:
        g.close()


def test_disk_at_its_limit_and_ragged_tiles(gu):
    # one disk straight ahead, the ego turning from 0 to 60 degrees off its normal in steps; 70 x 100 images (general kernels)
    rig = make_rig((0.0,), 80.0, 60.0, 100, 70, mount=(0.0, 0.0, 1.0))
    tris = disk_triangles((9.0, 0.0, 1.2), (-1.0, 0.0, 0.0), 0.7, n=16)
    angs = np.radians(np.arange(0.0, 61.0, 5.0))
    poses = np.stack([9.0 - 9.0 * np.cos(angs), 9.0 * np.sin(angs), -angs], 1)[:, None, :]       # one environment per angle, one agent each
    dims = np.tile(np.array(CAR, np.float32), (len(angs), 1, 1))
    s = custom_scene(tris, [6] * len(tris), poses, dims, rig, 70, 100, tri_vis_cos=[np.cos(np.radians(32.0))] * len(tris),
                     env_map_id=np.zeros(len(angs), np.int32))
    st = gu.check_against_oracle(s)
    seen = (st["ref"].cls == 6).reshape(len(angs), -1).sum(1)
    assert (seen[:6] > 0).all() and (seen[8:] == 0).all()              # 0..25 degrees off the normal drawn, 40.. culled
