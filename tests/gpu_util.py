"""Helpers for the GPU parity tests: run a scenes.Scene through the CUDA library."""
from __future__ import annotations

import numpy as np


class CudaRun:
    """Creates the library scene for a scenes.Scene and renders it through the C ABI."""

    def __init__(self, scene, device: int = 0):
        import torch
        import paper_2607_26005_b200 as pic
        self.pic = pic
        self.torch = torch
        self.s = scene
        s = scene
        self.dev = torch.device("cuda", device)
        self.scene = pic.Scene(s.E, s.A, s.K, s.H, s.W, s.near, s.far, s.tri_xyz, s.tri_class,
                               map_tri_offset=s.map_tri_offset, env_map_id=s.env_map_id, agent_class=s.agent_class,
                               sky_class=s.sky_class, ground_class=s.ground_class, device=device,
                               tri_vis_cos=getattr(s, "tri_vis_cos", None))
        self.poses = torch.from_numpy(np.ascontiguousarray(s.poses)).to(self.dev)
        self.dims = torch.from_numpy(np.ascontiguousarray(s.dims)).to(self.dev)
        self.active = torch.from_numpy(np.ascontiguousarray(s.active)).to(self.dev)
        if getattr(s, "agent_classes", None) is not None:
            self.scene.set_agent_classes(torch.from_numpy(np.ascontiguousarray(s.agent_classes, dtype=np.uint8)).to(self.dev))

    def render(self, brute: bool = False, depth32: bool = True, poses=None, view_first: int = 0, view_count: int = 0,
               counters: bool = False, debug_flags: int = 0):
        """Returns (class u8 [V,H,W], depth f16 [V,H,W], depth32 f32 [V,H,W] or None[, counters]) as numpy."""
        torch, pic, s = self.torch, self.pic, self.s
        cls, dep = self.scene.alloc_outputs()
        cls.fill_(255)
        dep.fill_(-1.0)
        d32 = torch.full(self.scene.image_shape, -1.0, dtype=torch.float32, device=self.dev) if depth32 else None
        cnt = torch.zeros(16, dtype=torch.int64, device=self.dev) if counters else None
        self.scene.set_option(pic.OPT_BRUTE_FORCE, 1 if brute else 0)
        self.scene.set_option(pic.OPT_DEPTH32, d32 if depth32 else 0)
        self.scene.set_option(pic.OPT_COUNTERS, cnt if counters else 0)
        self.scene.set_option(pic.OPT_VIEW_FIRST, view_first)
        self.scene.set_option(pic.OPT_VIEW_COUNT, view_count)
        self.scene.set_option(pic.OPT_DEBUG_FLAGS, int(debug_flags))
        p = self.poses if poses is None else torch.from_numpy(np.ascontiguousarray(poses, dtype=np.float32)).to(self.dev)
        self.scene.render(p, self.dims, s.rig, active=self.active, out_class=cls, out_depth=dep)
        torch.cuda.synchronize()
        self.scene.set_option(pic.OPT_DEPTH32, 0)
        self.scene.set_option(pic.OPT_COUNTERS, 0)
        self.scene.set_option(pic.OPT_BRUTE_FORCE, 0)
        self.scene.set_option(pic.OPT_VIEW_FIRST, 0)
        self.scene.set_option(pic.OPT_VIEW_COUNT, 0)
        self.scene.set_option(pic.OPT_DEBUG_FLAGS, 0)
        V = s.E * s.A * s.K
        out = (cls.cpu().numpy().reshape(V, s.H, s.W), dep.cpu().numpy().reshape(V, s.H, s.W),
               d32.cpu().numpy().reshape(V, s.H, s.W) if depth32 else None)
        if counters:
            out = out + (cnt.cpu().numpy(),)
        return out

    def render_rgb(self, palette, antialias: bool, poses=None, view_first: int = 0, view_count: int = 0):
        """Colour images u8 [V,H,W,3] as numpy (sentinel 7 where nothing was written), and the status flags."""
        torch, pic, s = self.torch, self.pic, self.s
        rgb = torch.full(self.scene.image_shape + (3,), 7, dtype=torch.uint8, device=self.dev)
        self.scene.set_palette(palette)
        self.scene.set_option(pic.OPT_VIEW_FIRST, view_first)
        self.scene.set_option(pic.OPT_VIEW_COUNT, view_count)
        p = self.poses if poses is None else torch.from_numpy(np.ascontiguousarray(poses, dtype=np.float32)).to(self.dev)
        self.scene.render_rgb(p, self.dims, s.rig, active=self.active, out_rgb=rgb, antialias=antialias)
        torch.cuda.synchronize()
        self.scene.set_option(pic.OPT_VIEW_FIRST, 0)
        self.scene.set_option(pic.OPT_VIEW_COUNT, 0)
        return rgb.cpu().numpy().reshape(s.E * s.A * s.K, s.H, s.W, 3), self.scene.status()

    def close(self):
        self.scene.close()


def check_against_oracle(scene, view_ids=None, gpu: CudaRun = None, **kw):
    """Render `view_ids` with the oracle and all views with the CUDA path; apply the acceptance rule."""
    import oracle
    from tests.util import compare_images
    own = gpu is None
    if own:
        gpu = CudaRun(scene)
    try:
        cls, d16, d32 = gpu.render()
        # without the float32 depth image the kernels take their vector-store paths: same images
        cls_v, d16_v, _ = gpu.render(depth32=False)
        assert (cls_v == cls).all() and (d16_v.view(np.uint16) == d16.view(np.uint16)).all()
        if view_ids is None:
            view_ids = np.arange(scene.E * scene.A * scene.K)
        view_ids = np.asarray(view_ids, dtype=np.int64)
        ref = oracle.render(scene, view_ids)
        stats = compare_images(ref.cls, ref.depth, ref.flag, cls[view_ids], d32[view_ids], d16[view_ids],
                               ref_kappa=ref.kappa, **kw)
        stats["ref"] = ref
        stats["gpu"] = (cls, d16, d32)
        return stats
    finally:
        if own:
            gpu.close()
