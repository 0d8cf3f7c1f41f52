"""Thin ctypes binding of libpictura.so: argument marshalling only.

Every step of the rendering path runs inside the CUDA library; torch is used for device memory,
streams and nothing else.  There is no CPU fallback: if the library cannot be loaded, or no CUDA
device is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np

from . import build as _build

PIC_OK = 0
STATUS_NAMES = {0: "PIC_OK", 1: "PIC_ERR_INVALID_ARG", 2: "PIC_ERR_SHAPE", 3: "PIC_ERR_OOM", 4: "PIC_ERR_CUDA",
                5: "PIC_ERR_CAPACITY", 6: "PIC_ERR_NONFINITE"}
OPT_BRUTE_FORCE, OPT_DEPTH32, OPT_COUNTERS, OPT_VIEW_FIRST, OPT_VIEW_COUNT, OPT_TIMING, OPT_DEBUG_FLAGS, OPT_OUT_RELATIVE, OPT_OCCLUSION = 1, 2, 3, 4, 5, 6, 7, 8, 9
FLAG_NONFINITE_POSE = 1
FLAG_COLOUR_INCOMPLETE = 2
FLAG_COLOUR_FRAGMENTS = 4

EXPORTS = ["pic_scene_create", "pic_scene_destroy", "pic_render", "pic_render_host", "pic_set_state",
           "pic_get_state", "pic_set_agent_classes", "pic_set_palette", "pic_render_rgb", "pic_step_rgb", "pic_step", "pic_get_status", "pic_scene_set_option", "pic_get_kernel_times", "pic_map_stats", "pic_render_static", "pic_static_status", "pic_probe_fill", "pic_probe_ffma",
           "pic_last_error", "pic_version"]


class PicError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class pic_camera(C.Structure):
    _fields_ = [("mount_x", C.c_float), ("mount_y", C.c_float), ("mount_z", C.c_float), ("yaw", C.c_float),
                ("pitch", C.c_float), ("fx", C.c_float), ("fy", C.c_float)]


class pic_scene_desc(C.Structure):
    _fields_ = [("size", C.c_uint32), ("E", C.c_int32), ("A", C.c_int32), ("K", C.c_int32), ("H", C.c_int32),
                ("W", C.c_int32), ("near_z", C.c_float), ("far_z", C.c_float), ("num_maps", C.c_int32),
                ("env_map_id", C.c_void_p), ("map_tri_offset", C.c_void_p), ("tri_xyz", C.c_void_p),
                ("tri_class", C.c_void_p), ("agent_class", C.c_uint8), ("sky_class", C.c_uint8),
                ("ground_class", C.c_uint8), ("reserved", C.c_uint8), ("device", C.c_int32), ("tri_vis_cos", C.c_void_p)]


class pic_static_desc(C.Structure):
    _fields_ = [("size", C.c_uint32), ("E", C.c_int32), ("A", C.c_int32), ("K", C.c_int32), ("H", C.c_int32),
                ("W", C.c_int32), ("n_tris", C.c_int32), ("near_z", C.c_float), ("far_z", C.c_float),
                ("agent_class", C.c_uint8), ("sky_class", C.c_uint8), ("ground_class", C.c_uint8),
                ("reserved", C.c_uint8)]


_lib = None


def load(path: Optional[str] = None):
    """Load libpictura.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"CUDA library {path} is missing; run paper_2607_26005_b200.build.build()")
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.pic_scene_create.argtypes = [C.POINTER(pic_scene_desc), C.POINTER(vp)]
    lib.pic_scene_destroy.argtypes = [vp]
    lib.pic_render.argtypes = [vp, vp, vp, vp, C.POINTER(pic_camera), vp, vp, vp]
    lib.pic_render_host.argtypes = [vp, vp, vp, vp, C.POINTER(pic_camera), vp, vp, vp]
    lib.pic_set_state.argtypes = [vp, vp, vp, vp, vp]
    lib.pic_get_state.argtypes = [vp, vp, vp]
    lib.pic_set_agent_classes.argtypes = [vp, vp, vp]
    lib.pic_set_palette.argtypes = [vp, vp, vp]
    lib.pic_render_rgb.argtypes = [vp, vp, vp, vp, C.POINTER(pic_camera), C.c_int32, vp, vp]
    lib.pic_step_rgb.argtypes = [vp, vp, C.POINTER(pic_camera), C.c_int32, vp, vp]
    lib.pic_step.argtypes = [vp, vp, C.POINTER(pic_camera), vp, vp, vp]
    lib.pic_get_status.argtypes = [vp, C.POINTER(C.c_uint32), vp]
    lib.pic_scene_set_option.argtypes = [vp, C.c_int32, C.c_uint64]
    lib.pic_get_kernel_times.argtypes = [vp, C.POINTER(C.c_float), C.c_int32, C.POINTER(C.c_int32)]
    lib.pic_map_stats.argtypes = [C.POINTER(pic_scene_desc), C.POINTER(C.c_int64)]
    lib.pic_render_static.argtypes = [C.POINTER(pic_static_desc), vp, vp, vp, vp, vp, C.POINTER(pic_camera), vp, vp, vp]
    lib.pic_static_status.argtypes = [C.POINTER(C.c_uint32), vp]
    lib.pic_probe_fill.argtypes = [vp, C.c_uint64, vp]
    lib.pic_probe_ffma.argtypes = [vp, C.c_uint64, C.c_int32, C.POINTER(C.c_uint64), vp]
    for name in EXPORTS:
        getattr(lib, name).restype = C.c_int
    lib.pic_last_error.restype = C.c_char_p
    lib.pic_last_error.argtypes = []
    lib.pic_version.restype = C.c_int32
    lib.pic_version.argtypes = []
    _lib = lib
    return lib


def _check(lib, status: int):
    if status != PIC_OK:
        raise PicError(status, lib.pic_last_error().decode("utf-8", "replace"))


def _rig_array(rig) -> "C.Array":
    rig = np.asarray(rig, dtype=np.float32).reshape(-1, 7)
    arr = (pic_camera * rig.shape[0])()
    for k in range(rig.shape[0]):
        arr[k] = pic_camera(*[float(v) for v in rig[k]])
    return arr


def _dev_ptr(t, dtype, numel: Optional[int] = None) -> int:
    import torch
    if t is None:
        return 0
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("expected a CUDA torch tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"expected a contiguous {dtype} tensor, got {t.dtype}")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"expected {numel} elements, got {t.numel()}")
    return t.data_ptr()


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def map_stats(tri_xyz, tri_class, map_tri_offset=None, A: int = 0) -> dict:
    """Host-only statistics of the scene builder's map preprocessing (no GPU needed)."""
    lib = load()
    tri_xyz = np.ascontiguousarray(tri_xyz, dtype=np.float32).reshape(-1, 3, 3)
    tri_class = np.ascontiguousarray(tri_class, dtype=np.uint8).reshape(-1)
    if map_tri_offset is None:
        map_tri_offset = [0, tri_xyz.shape[0]]
    off = np.ascontiguousarray(map_tri_offset, dtype=np.int64)
    d = pic_scene_desc()
    d.size = C.sizeof(pic_scene_desc)
    d.A = int(A)
    d.num_maps = int(off.shape[0] - 1)
    d.map_tri_offset = off.ctypes.data
    d.tri_xyz = tri_xyz.ctypes.data
    d.tri_class = tri_class.ctypes.data
    out = (C.c_int64 * 8)()
    _check(lib, lib.pic_map_stats(C.byref(d), out))
    names = ["primitives", "quads", "leaves", "groups", "largest_leaf", "prims_outside_leaf", "leaves_outside_group",
             "triangles"]
    return dict(zip(names, [int(v) for v in out]))


def render_static(E: int, A: int, K: int, H: int, W: int, near: float, far: float, tri_xyz, tri_class, poses, dims,
                  rig, out_class, out_depth, active=None, agent_class: int = 4, sky_class: int = 0,
                  ground_class: int = 1, stream=None):
    """pic_render_static: render on the current device without a scene and without allocating.
    tri_xyz (f32 [N,3,3]), tri_class (u8 [N]), poses, dims, active and the outputs are CUDA tensors
    the caller already owns; nothing is allocated here either."""
    import torch
    lib = load()
    n, npx = E * A, E * A * K * H * W
    n_tris = 0 if tri_xyz is None else int(tri_xyz.shape[0])
    d = pic_static_desc()
    d.size = C.sizeof(pic_static_desc)
    d.E, d.A, d.K, d.H, d.W, d.n_tris = int(E), int(A), int(K), int(H), int(W), n_tris
    d.near_z, d.far_z = float(near), float(far)
    d.agent_class, d.sky_class, d.ground_class = int(agent_class), int(sky_class), int(ground_class)
    _check(lib, lib.pic_render_static(
        C.byref(d), _dev_ptr(tri_xyz, torch.float32, 9 * n_tris) if n_tris else None,
        _dev_ptr(tri_class, torch.uint8, n_tris) if n_tris else None, _dev_ptr(poses, torch.float32, 3 * n),
        _dev_ptr(dims, torch.float32, 3 * n), _dev_ptr(active, torch.uint8, n) if active is not None else None,
        _rig_array(rig), _dev_ptr(out_class, torch.uint8, npx), _dev_ptr(out_depth, torch.float16, npx),
        _stream_ptr(stream)))
    return out_class, out_depth


def probe_fill(dst, stream=None) -> int:
    """pic_probe_fill on a CUDA tensor (write-only stream, 128-bit stores); returns the bytes written."""
    lib = load()
    nbytes = dst.numel() * dst.element_size()
    _check(lib, lib.pic_probe_fill(C.c_void_p(dst.data_ptr()), nbytes, _stream_ptr(stream)))
    return nbytes


def probe_ffma(out, iters: int, stream=None) -> int:
    """pic_probe_ffma (register-only FFMA loop); `out` is a float32 CUDA tensor; returns the per-lane FMA count."""
    import torch
    lib = load()
    n = C.c_uint64(0)
    _check(lib, lib.pic_probe_ffma(_dev_ptr(out, torch.float32, out.numel()), out.numel(), int(iters), C.byref(n), _stream_ptr(stream)))
    return int(n.value)


def static_status(stream=None) -> int:
    """pic_static_status: read and clear the sticky flags of pic_render_static on the current device."""
    lib = load()
    flags = C.c_uint32(0)
    _check(lib, lib.pic_static_status(C.byref(flags), _stream_ptr(stream)))
    return int(flags.value)


class Scene:
    """Owner of one pic_scene.  Arrays follow include/pictura.h; device tensors are torch CUDA tensors."""

    def __init__(self, E: int, A: int, K: int, H: int, W: int, near: float, far: float, tri_xyz, tri_class,
                 map_tri_offset=None, env_map_id=None, agent_class: int = 4, sky_class: int = 0,
                 ground_class: int = 1, device: int = 0, tri_vis_cos=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the rasterizer has no CPU path")
        self._lib = load()
        tri_xyz = np.ascontiguousarray(tri_xyz, dtype=np.float32).reshape(-1, 3, 3)
        tri_class = np.ascontiguousarray(tri_class, dtype=np.uint8).reshape(-1)
        if map_tri_offset is None:
            map_tri_offset = [0, tri_xyz.shape[0]]
        off = np.ascontiguousarray(map_tri_offset, dtype=np.int64)
        emi = None if env_map_id is None else np.ascontiguousarray(env_map_id, dtype=np.int32)
        d = pic_scene_desc()
        d.size = C.sizeof(pic_scene_desc)
        d.E, d.A, d.K, d.H, d.W = int(E), int(A), int(K), int(H), int(W)
        d.near_z, d.far_z = float(near), float(far)
        d.num_maps = int(off.shape[0] - 1)
        d.env_map_id = None if emi is None else emi.ctypes.data
        d.map_tri_offset = off.ctypes.data
        d.tri_xyz = tri_xyz.ctypes.data
        d.tri_class = tri_class.ctypes.data
        d.agent_class, d.sky_class, d.ground_class = int(agent_class), int(sky_class), int(ground_class)
        d.device = int(device)
        vis = None if tri_vis_cos is None else np.ascontiguousarray(tri_vis_cos, dtype=np.float32).reshape(-1)
        if vis is not None and vis.shape[0] != tri_xyz.shape[0]:
            raise ValueError("tri_vis_cos needs one value per triangle")
        d.tri_vis_cos = None if vis is None else vis.ctypes.data
        handle = C.c_void_p()
        _check(self._lib, self._lib.pic_scene_create(C.byref(d), C.byref(handle)))
        self._h = handle
        self.E, self.A, self.K, self.H, self.W = int(E), int(A), int(K), int(H), int(W)
        self.device = torch.device("cuda", int(device))
        self._keep = []   # tensors referenced by options

    # -- shapes ---------------------------------------------------------------------------------
    @property
    def n_agents(self) -> int:
        return self.E * self.A

    @property
    def image_shape(self) -> Tuple[int, int, int, int, int]:
        return (self.E, self.A, self.K, self.H, self.W)

    def alloc_outputs(self):
        import torch
        cls = torch.empty(self.image_shape, dtype=torch.uint8, device=self.device)
        depth = torch.empty(self.image_shape, dtype=torch.float16, device=self.device)
        return cls, depth

    # -- calls ----------------------------------------------------------------------------------
    def render(self, poses, dims, rig, active=None, out_class=None, out_depth=None, stream=None):
        import torch
        if out_class is None or out_depth is None:
            out_class, out_depth = self.alloc_outputs()
        n, npx = self.n_agents, self.n_agents * self.K * self.H * self.W
        _check(self._lib, self._lib.pic_render(
            self._h, _dev_ptr(poses, torch.float32, 3 * n), _dev_ptr(dims, torch.float32, 3 * n),
            _dev_ptr(active, torch.uint8, n) if active is not None else None, _rig_array(rig),
            _dev_ptr(out_class, torch.uint8, npx), _dev_ptr(out_depth, torch.float16, npx), _stream_ptr(stream)))
        return out_class, out_depth

    def set_palette(self, palette, stream=None):
        """palette: numpy u8 [256,3], the RGB of every class id (colour output)."""
        pal = np.ascontiguousarray(palette, dtype=np.uint8)
        if pal.shape != (256, 3):
            raise ValueError("palette must be u8 [256,3]")
        _check(self._lib, self._lib.pic_set_palette(self._h, pal.ctypes.data_as(C.c_void_p), _stream_ptr(stream)))

    def render_rgb(self, poses, dims, rig, active=None, out_rgb=None, antialias=False, stream=None):
        """Colour images, u8 [E,A,K,H,W,3] (with OPT_OUT_RELATIVE: [views rendered,H,W,3], which the caller sizes);
        antialias: analytic coverage at one sample per pixel."""
        import torch
        if out_rgb is None:
            out_rgb = torch.empty(self.image_shape + (3,), dtype=torch.uint8, device=self.device)
        n, npx = self.n_agents, self.n_agents * self.K * self.H * self.W
        _check(self._lib, self._lib.pic_render_rgb(
            self._h, _dev_ptr(poses, torch.float32, 3 * n), _dev_ptr(dims, torch.float32, 3 * n),
            _dev_ptr(active, torch.uint8, n) if active is not None else None, _rig_array(rig),
            1 if antialias else 0, _dev_ptr(out_rgb, torch.uint8), _stream_ptr(stream)))
        return out_rgb

    def render_in_passes(self, poses, dims, rig, consume, max_bytes: int, active=None, stream=None) -> int:
        """Render all views in passes whose output fits `max_bytes` (class + depth bytes), into one pair of
        pass-sized buffers that is reused: after each pass `consume(first_view, n_views, class_u8, depth_f16)` is
        called with views of the buffers (shape [n_views, H, W]); the device is synchronised before it runs, and
        the next pass overwrites the buffers.  Returns the number of passes.  Argument marshalling only: every
        pass is one pic_render call with PIC_OPT_VIEW_FIRST / VIEW_COUNT / OUT_RELATIVE set."""
        import torch
        total = self.n_agents * self.K
        per_view = 3 * self.H * self.W
        n_pass_views = max(1, min(total, int(max_bytes) // per_view))
        out_c = torch.empty((n_pass_views, self.H, self.W), dtype=torch.uint8, device=self.device)
        out_d = torch.empty((n_pass_views, self.H, self.W), dtype=torch.float16, device=self.device)
        n, passes = self.n_agents, 0
        try:
            self.set_option(OPT_OUT_RELATIVE, 1)
            for first in range(0, total, n_pass_views):
                cnt = min(n_pass_views, total - first)
                self.set_option(OPT_VIEW_FIRST, first)
                self.set_option(OPT_VIEW_COUNT, cnt)
                _check(self._lib, self._lib.pic_render(
                    self._h, _dev_ptr(poses, torch.float32, 3 * n), _dev_ptr(dims, torch.float32, 3 * n),
                    _dev_ptr(active, torch.uint8, n) if active is not None else None, _rig_array(rig),
                    out_c.data_ptr(), out_d.data_ptr(), _stream_ptr(stream)))
                torch.cuda.synchronize(self.device)
                consume(first, cnt, out_c[:cnt], out_d[:cnt])
                passes += 1
        finally:
            self.set_option(OPT_VIEW_FIRST, 0)
            self.set_option(OPT_VIEW_COUNT, 0)
            self.set_option(OPT_OUT_RELATIVE, 0)
        return passes

    def render_host(self, poses: np.ndarray, dims: np.ndarray, rig, out_class: np.ndarray, out_depth: np.ndarray,
                    active: Optional[np.ndarray] = None, stream=None):
        """Host-buffer variant: numpy (or pinned torch CPU tensors viewed as numpy) in and out."""
        def hp(a, dtype, numel):
            if a is None:
                return None
            if a.dtype != dtype or not a.flags["C_CONTIGUOUS"] or a.size != numel:
                raise TypeError(f"expected contiguous {dtype} array of {numel} elements")
            return a.ctypes.data
        n, npx = self.n_agents, self.n_agents * self.K * self.H * self.W
        _check(self._lib, self._lib.pic_render_host(
            self._h, hp(poses, np.float32, 3 * n), hp(dims, np.float32, 3 * n), hp(active, np.uint8, n),
            _rig_array(rig), hp(out_class, np.uint8, npx), hp(out_depth, np.float16, npx), _stream_ptr(stream)))
        return out_class, out_depth

    def set_state(self, state, dims, active=None, stream=None):
        import torch
        n = self.n_agents
        _check(self._lib, self._lib.pic_set_state(
            self._h, _dev_ptr(state, torch.float32, 4 * n), _dev_ptr(dims, torch.float32, 3 * n),
            _dev_ptr(active, torch.uint8, n) if active is not None else None, _stream_ptr(stream)))

    def set_agent_classes(self, classes, stream=None):
        """classes: CUDA u8 tensor [E,A] (class of each agent's box), or None for the scene-wide agent class."""
        import torch
        _check(self._lib, self._lib.pic_set_agent_classes(
            self._h, _dev_ptr(classes, torch.uint8, self.n_agents) if classes is not None else None, _stream_ptr(stream)))

    def get_state(self, out=None, stream=None):
        import torch
        if out is None:
            out = torch.empty((self.E, self.A, 4), dtype=torch.float32, device=self.device)
        _check(self._lib, self._lib.pic_get_state(self._h, _dev_ptr(out, torch.float32, 4 * self.n_agents),
                                                  _stream_ptr(stream)))
        return out

    def step(self, actions, rig, out_class=None, out_depth=None, stream=None):
        import torch
        if out_class is None or out_depth is None:
            out_class, out_depth = self.alloc_outputs()
        n, npx = self.n_agents, self.n_agents * self.K * self.H * self.W
        _check(self._lib, self._lib.pic_step(
            self._h, _dev_ptr(actions, torch.float32, 2 * n), _rig_array(rig), _dev_ptr(out_class, torch.uint8, npx),
            _dev_ptr(out_depth, torch.float16, npx), _stream_ptr(stream)))
        return out_class, out_depth

    def step_rgb(self, actions, rig, out_rgb=None, antialias=False, stream=None):
        """One simulator step, then colour images u8 [E,A,K,H,W,3] from the new state."""
        import torch
        if out_rgb is None:
            out_rgb = torch.empty(self.image_shape + (3,), dtype=torch.uint8, device=self.device)
        _check(self._lib, self._lib.pic_step_rgb(
            self._h, _dev_ptr(actions, torch.float32, 2 * self.n_agents), _rig_array(rig), 1 if antialias else 0,
            _dev_ptr(out_rgb, torch.uint8), _stream_ptr(stream)))
        return out_rgb

    def status(self, stream=None) -> int:
        flags = C.c_uint32(0)
        _check(self._lib, self._lib.pic_get_status(self._h, C.byref(flags), _stream_ptr(stream)))
        return int(flags.value)

    def kernel_times(self) -> np.ndarray:
        """Milliseconds of each render-kernel launch since the last call (OPT_TIMING must be on)."""
        buf = (C.c_float * 1024)()
        n = C.c_int32(0)
        _check(self._lib, self._lib.pic_get_kernel_times(self._h, buf, 1024, C.byref(n)))
        return np.array(buf[:min(int(n.value), 1024)], dtype=np.float64)

    def set_option(self, option: int, value) -> None:
        import torch
        if isinstance(value, torch.Tensor):
            self._keep.append(value)
            value = value.data_ptr()
        _check(self._lib, self._lib.pic_scene_set_option(self._h, int(option), int(value)))

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.pic_scene_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
