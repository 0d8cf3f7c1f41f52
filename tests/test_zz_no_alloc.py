"""pic_render_static -- the entry point for callers that may not allocate device memory (a locked
memory pool, a real-time loop, a host application that owns the heap).  It keeps its working
buffers in a fixed array inside the library, so this test checks that (a) it draws the same
images as the scene-based pic_render, on two calls in a row (the array is reused and must be
re-initialised by the call itself), and (b) the calls really allocate nothing.  Collected last so
that a failure here cannot hide the other tests' results."""
import numpy as np
import pytest

from scenes import make_config

pytestmark = pytest.mark.gpu


def _f16_ulps(a, b):
    return np.abs(a.view(np.uint16).astype(np.int32) - b.view(np.uint16).astype(np.int32))


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
    finally:
        scene.close()


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
