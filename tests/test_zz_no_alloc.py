"""pic_render_static -- the entry point for callers that may not allocate device memory (a locked
memory pool, a real-time loop, a host application that owns the heap).  It keeps its working
buffers in a fixed array inside the library, so these tests check that (a) it draws the same
images as the scene-based pic_render, on two calls in a row (the array is reused and must be
re-initialised by the call itself), (b) the calls really allocate nothing, (c) its images satisfy
the same acceptance rule against the CPU oracle as the scene path, (d) the index arithmetic for
several environments, cameras, ragged multi-tile images, inactive agents and an empty map holds,
and (e) requests beyond its limits are refused before anything is launched.  Collected last so
that a failure here cannot hide the other tests' results."""
import numpy as np
import pytest

from scenes import make_config
from tests.util import compare_images, custom_scene, make_rig

CAR = (4.5, 1.9, 1.5)

pytestmark = pytest.mark.gpu


def _f16_ulps(a, b):
    return np.abs(a.view(np.uint16).astype(np.int32) - b.view(np.uint16).astype(np.int32))


def _static_render(s, dev, poses=None):
    import torch
    import paper_2607_26005_b200 as pic
    tri = torch.from_numpy(np.ascontiguousarray(s.tri_xyz)).to(dev) if len(s.tri_xyz) else None
    cls = torch.from_numpy(np.ascontiguousarray(s.tri_class)).to(dev) if len(s.tri_xyz) else None
    V = s.E * s.A * s.K
    out_c = torch.full((V, s.H, s.W), 255, dtype=torch.uint8, device=dev)
    out_d = torch.full((V, s.H, s.W), -1.0, dtype=torch.float16, device=dev)
    p = torch.from_numpy(np.ascontiguousarray(s.poses if poses is None else poses)).to(dev)
    pic.render_static(s.E, s.A, s.K, s.H, s.W, s.near, s.far, tri, cls, p, torch.from_numpy(np.ascontiguousarray(s.dims)).to(dev),
                      s.rig, out_c, out_d, active=torch.from_numpy(np.ascontiguousarray(s.active)).to(dev),
                      agent_class=s.agent_class, sky_class=s.sky_class, ground_class=s.ground_class)
    torch.cuda.synchronize()
    return out_c.cpu().numpy(), out_d.cpu().numpy()


def test_static_entry_point_matches_pic_render_twice_without_allocating():
    import torch
    import paper_2607_26005_b200 as pic
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    s = make_config(0)                       # 1 env, 8 agents, 1 camera, 64x64, ~800 triangles
    tri = torch.from_numpy(s.tri_xyz).to(dev)
    cls = torch.from_numpy(s.tri_class).to(dev)
    dims = torch.from_numpy(s.dims).to(dev)
    active = torch.from_numpy(s.active).to(dev)
    scene = pic.Scene(s.E, s.A, s.K, s.H, s.W, s.near, s.far, s.tri_xyz, s.tri_class, map_tri_offset=s.map_tri_offset,
                      env_map_id=s.env_map_id)
    try:
        rng = np.random.default_rng(7)
        ref_c, ref_d = scene.alloc_outputs()
        out_c, out_d = scene.alloc_outputs()
        for call in range(2):
            # second call: move everybody, so stale per-agent data in the shared array would show
            poses_np = s.poses.copy()
            if call == 1:
                poses_np[..., :2] += rng.uniform(-1.0, 1.0, size=poses_np[..., :2].shape).astype(np.float32)
                poses_np[..., 2] += 0.05
            poses = torch.from_numpy(poses_np).to(dev)
            scene.render(poses, dims, s.rig, active=active, out_class=ref_c, out_depth=ref_d)
            out_c.fill_(255); out_d.fill_(-1.0)
            torch.cuda.synchronize()
            free_before, _ = torch.cuda.mem_get_info(dev)
            pic.render_static(s.E, s.A, s.K, s.H, s.W, s.near, s.far, tri, cls, poses, dims, s.rig, out_c, out_d,
                              active=active)
            torch.cuda.synchronize()
            free_after, _ = torch.cuda.mem_get_info(dev)
            if call == 1:                     # the first call on a device may load the kernel image
                assert free_after == free_before, "pic_render_static changed the amount of free device memory"
            a, b = ref_c.cpu().numpy(), out_c.cpu().numpy()
            da, db = ref_d.cpu().numpy(), out_d.cpu().numpy()
            # same tolerance as the parity tests: at most 1e-4 of the pixels may differ in class
            # (the scene path pairs triangles into quads, which moves depths by an ulp at ties),
            # the binary16 depth elsewhere by at most one unit in the last place
            diff = a != b
            assert diff.mean() <= 1e-4, f"call {call}: {int(diff.sum())} class mismatches"
            assert _f16_ulps(da, db)[~diff].max() <= 1
            assert (b != 255).all()
        assert pic.static_status() == 0
    finally:
        scene.close()


def test_static_entry_point_against_the_oracle():
    """The acceptance rule of the parity tests, applied to pic_render_static's images of config 0 (the binary16
    depth plane is the only depth this entry point writes: it must equal the rounded oracle depth or be one
    unit in the last place off, and every class mismatch must sit on a pixel the oracle flags as ambiguous)."""
    import torch
    import oracle
    dev = torch.device("cuda", 0)
    s = make_config(0)
    cls, d16 = _static_render(s, dev)
    ref = oracle.render(s, np.arange(s.E * s.A * s.K))
    st = compare_images(ref.cls, ref.depth, ref.flag, cls, d16.astype(np.float32), d16, ref_kappa=ref.kappa, depth_rtol=1e-3)
    assert st["pixels"] == s.E * s.A * s.K * s.H * s.W


def test_static_entry_point_index_arithmetic_and_flags():
    """Two environments, three agents (one inactive), two cameras with different mounts, a ragged two-tile image
    and a handful of triangles: pic_render_static against the scene's exhaustive kernel (same arithmetic, so the
    images must be identical), then an empty map, then a NaN pose, which must be flagged and drawn as sky."""
    import torch
    import paper_2607_26005_b200 as pic
    from tests.gpu_util import CudaRun
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(11)
    tris = []
    for _ in range(24):
        c = np.array([rng.uniform(-30, 30), rng.uniform(-30, 30), rng.uniform(0.0, 3.0)])
        tris.append(c + rng.uniform(-4, 4, size=(3, 3)))
    tris = np.asarray(tris, np.float32)
    rig = make_rig((0.0, 110.0), 80.0, 60.0, 70, 100, mount=(1.0, 0.2, 1.4))
    rig[1, :3] = (-0.5, -0.3, 1.7)
    poses = rng.uniform(-10, 10, size=(2, 3, 3)).astype(np.float32)
    dims = np.tile(np.array(CAR, np.float32), (2, 3, 1))
    active = np.ones((2, 3), np.uint8); active[1, 2] = 0
    s = custom_scene(tris, rng.integers(2, 6, size=24).astype(np.uint8), poses, dims, rig, 70, 100, active=active)
    g = CudaRun(s)
    try:
        ref_c, ref_d, _ = g.render(brute=True, depth32=False)
    finally:
        g.close()
    cls, d16 = _static_render(s, dev)
    assert (cls == ref_c).all() and (d16.view(np.uint16) == ref_d.view(np.uint16)).all()
    assert (cls[5 * 2:] == 0).all()                     # the inactive agent's own images are sky
    # an empty map: only boxes, ground and sky
    s0 = custom_scene(np.zeros((0, 3, 3), np.float32), np.zeros(0, np.uint8), poses, dims, rig, 70, 100, active=active)
    g = CudaRun(s0)
    try:
        ref_c, ref_d, _ = g.render(brute=True, depth32=False)
    finally:
        g.close()
    cls, d16 = _static_render(s0, dev)
    assert (cls == ref_c).all() and (d16.view(np.uint16) == ref_d.view(np.uint16)).all() and set(np.unique(cls)) <= {0, 1, 4}
    assert pic.static_status() == 0
    bad = poses.copy(); bad[0, 1, 0] = np.nan
    cls, _ = _static_render(s0, dev, poses=bad)
    assert pic.static_status() & pic.FLAG_NONFINITE_POSE
    assert pic.static_status() == 0                     # reading clears it
    assert (cls[2:4] == 0).all()


def test_static_entry_point_rejects_oversized_batches():
    import torch
    import paper_2607_26005_b200 as pic
    dev = torch.device("cuda", 0)
    z = torch.zeros(16, dtype=torch.float32, device=dev)
    rig = np.array([[0, 0, 1.5, 0, 0, 32, 32]], np.float32)
    with pytest.raises(pic.PicError) as ei:
        pic.render_static(2048, 1, 1, 8, 8, 0.5, 100.0, None, None, torch.zeros(2048 * 3, device=dev),
                          torch.ones(2048 * 3, device=dev), rig, torch.zeros(2048 * 64, dtype=torch.uint8, device=dev),
                          torch.zeros(2048 * 64, dtype=torch.float16, device=dev))
    assert ei.value.status == 5 and "at most" in str(ei.value)
    with pytest.raises(pic.PicError) as ei:
        pic.render_static(1, 1, 1, 8, 1024, 0.5, 100.0, None, None, z[:3], z[:3] + 1, rig,
                          torch.zeros(8 * 1024, dtype=torch.uint8, device=dev),
                          torch.zeros(8 * 1024, dtype=torch.float16, device=dev))
    assert ei.value.status == 5
    # within every single limit, but far too much work for one launch: refused on the host, nothing runs
    n_tris, views, side = 60000, 64, 512
    with pytest.raises(pic.PicError) as ei:
        pic.render_static(1, views, 1, side, side, 0.5, 100.0, torch.zeros((n_tris, 3, 3), device=dev),
                          torch.zeros(n_tris, dtype=torch.uint8, device=dev), torch.zeros(views * 3, device=dev),
                          torch.ones(views * 3, device=dev), rig, torch.zeros(views * side * side, dtype=torch.uint8, device=dev),
                          torch.zeros(views * side * side, dtype=torch.float16, device=dev))
    assert ei.value.status == 5 and "tests" in str(ei.value)
