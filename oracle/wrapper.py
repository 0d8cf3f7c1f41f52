"""ctypes loader for the C oracle (test infrastructure; see pic_oracle.c for the definition)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pic_oracle.c")
_LIB = os.path.join(_HERE, "libpic_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile pic_oracle.c into libpic_oracle.so next to it (gcc, -O2, OpenMP, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = C.CDLL(_LIB)
        p = C.c_void_p
        lib.pico_render.restype = C.c_int
        lib.pico_render.argtypes = [C.c_int] * 5 + [C.c_double] * 2 + [p] * 4 + [C.c_int] * 3 + [p] * 6 + \
                                   [C.c_int, p] + [p] * 7 + [C.c_int]
        lib.pico_render_rgb.restype = C.c_int
        lib.pico_render_rgb.argtypes = [C.c_int] * 5 + [C.c_double] * 2 + [p] * 4 + [C.c_int] * 3 + [p] * 6 + \
                                       [p, C.c_int] + [C.c_int, p] + [p] * 3 + [C.c_int]
        lib.pico_edge_coverage.restype = C.c_double
        lib.pico_edge_coverage.argtypes = [C.c_double] * 3
        lib.pico_pixel_coverage.restype = C.c_double
        lib.pico_pixel_coverage.argtypes = [C.c_int] + [p] * 3
        lib.pico_step.restype = None
        lib.pico_step.argtypes = [p, p, p, C.c_int64, C.c_double, C.c_double, C.c_double]
        lib.pico_f64_to_f16.restype = C.c_uint16
        lib.pico_f64_to_f16.argtypes = [C.c_double]
        lib.pico_max_threads.restype = C.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().pico_max_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


@dataclass
class OracleResult:
    view_ids: np.ndarray     # int64 [n]
    cls: np.ndarray          # u8  [n,H,W]
    depth: np.ndarray        # f64 [n,H,W]
    depth_f16: np.ndarray    # f16 [n,H,W]
    index: np.ndarray        # i32 [n,H,W]  winning primitive, -1 background
    flag: np.ndarray         # u8  [n,H,W]  ambiguity mask bits (1 edge, 2 depth, 4 near/far, 8 horizon, 16 grazing, 32 angular limit)
    kappa: np.ndarray        # f64 [n,H,W]  conditioning of the winner's depth (0 for background)
    counts: np.ndarray       # i64 [n,4]    in-frustum prims, prims with a kept fragment, kept fragments, flagged px


def render(scene, view_ids: Optional[Sequence[int]] = None, poses: Optional[np.ndarray] = None,
           n_threads: int = 0) -> OracleResult:
    """Render views of `scene` (a scenes.Scene).  view id = (e*A + a)*K + k; default: all views.
    `poses` overrides scene.poses (used when the state came from elsewhere)."""
    lib = _load()
    s = scene
    if view_ids is None:
        view_ids = np.arange(s.E * s.A * s.K, dtype=np.int64)
    view_ids = np.ascontiguousarray(view_ids, dtype=np.int64)
    n = int(view_ids.shape[0])
    poses = np.ascontiguousarray(s.poses if poses is None else poses, dtype=np.float32)
    dims = np.ascontiguousarray(s.dims, dtype=np.float32)
    active = np.ascontiguousarray(s.active, dtype=np.uint8)
    rig = np.ascontiguousarray(s.rig, dtype=np.float32)
    tri = np.ascontiguousarray(s.tri_xyz, dtype=np.float32)
    tcl = np.ascontiguousarray(s.tri_class, dtype=np.uint8)
    emi = np.ascontiguousarray(s.env_map_id, dtype=np.int32)
    off = np.ascontiguousarray(s.map_tri_offset, dtype=np.int64)
    acl = getattr(s, "agent_classes", None)
    acl = None if acl is None else np.ascontiguousarray(acl, dtype=np.uint8)
    vis = getattr(s, "tri_vis_cos", None)
    vis = None if vis is None else np.ascontiguousarray(vis, dtype=np.float32)
    cls = np.empty((n, s.H, s.W), np.uint8)
    depth = np.empty((n, s.H, s.W), np.float64)
    f16 = np.empty((n, s.H, s.W), np.uint16)
    index = np.empty((n, s.H, s.W), np.int32)
    flag = np.empty((n, s.H, s.W), np.uint8)
    kappa = np.empty((n, s.H, s.W), np.float64)
    counts = np.zeros((n, 4), np.int64)
    rc = lib.pico_render(s.E, s.A, s.K, s.H, s.W, float(s.near), float(s.far), _ptr(emi), _ptr(off), _ptr(tri),
                         _ptr(tcl), int(s.agent_class), int(s.sky_class), int(s.ground_class), _ptr(poses),
                         _ptr(dims), _ptr(active), _ptr(rig), _ptr(acl), _ptr(vis), n, _ptr(view_ids), _ptr(cls), _ptr(depth),
                         _ptr(f16), _ptr(index), _ptr(flag), _ptr(kappa), _ptr(counts), int(n_threads))
    if rc != 0:
        raise MemoryError("pico_render failed")
    return OracleResult(view_ids, cls, depth, f16.view(np.float16), index, flag, kappa, counts)


@dataclass
class OracleColour:
    view_ids: np.ndarray     # int64 [n]
    rgb: np.ndarray          # u8  [n,H,W,3]  rounded colour
    rgbf: np.ndarray         # f64 [n,H,W,3]  colour before rounding, 0..255
    flag: np.ndarray         # u8  [n,H,W]    ambiguity mask (see pico_render_rgb)


def render_rgb(scene, palette: np.ndarray, aa: bool, view_ids: Optional[Sequence[int]] = None,
               poses: Optional[np.ndarray] = None, n_threads: int = 0) -> OracleColour:
    """Colour images (O11) of views of `scene`, antialiased by analytic coverage (O12) if `aa`.
    palette: u8 [256,3], the RGB of every class."""
    lib = _load()
    s = scene
    if view_ids is None:
        view_ids = np.arange(s.E * s.A * s.K, dtype=np.int64)
    view_ids = np.ascontiguousarray(view_ids, dtype=np.int64)
    n = int(view_ids.shape[0])
    poses = np.ascontiguousarray(s.poses if poses is None else poses, dtype=np.float32)
    dims = np.ascontiguousarray(s.dims, dtype=np.float32)
    active = np.ascontiguousarray(s.active, dtype=np.uint8)
    rig = np.ascontiguousarray(s.rig, dtype=np.float32)
    tri = np.ascontiguousarray(s.tri_xyz, dtype=np.float32)
    tcl = np.ascontiguousarray(s.tri_class, dtype=np.uint8)
    emi = np.ascontiguousarray(s.env_map_id, dtype=np.int32)
    off = np.ascontiguousarray(s.map_tri_offset, dtype=np.int64)
    acl = getattr(s, "agent_classes", None)
    acl = None if acl is None else np.ascontiguousarray(acl, dtype=np.uint8)
    vis = getattr(s, "tri_vis_cos", None)
    vis = None if vis is None else np.ascontiguousarray(vis, dtype=np.float32)
    pal = np.ascontiguousarray(palette, dtype=np.uint8)
    assert pal.shape == (256, 3)
    rgb = np.empty((n, s.H, s.W, 3), np.uint8)
    rgbf = np.empty((n, s.H, s.W, 3), np.float64)
    flag = np.empty((n, s.H, s.W), np.uint8)
    rc = lib.pico_render_rgb(s.E, s.A, s.K, s.H, s.W, float(s.near), float(s.far), _ptr(emi), _ptr(off), _ptr(tri),
                             _ptr(tcl), int(s.agent_class), int(s.sky_class), int(s.ground_class), _ptr(poses),
                             _ptr(dims), _ptr(active), _ptr(rig), _ptr(acl), _ptr(vis), _ptr(pal), int(bool(aa)),
                             n, _ptr(view_ids), _ptr(rgb), _ptr(rgbf), _ptr(flag), int(n_threads))
    if rc != 0:
        raise MemoryError("pico_render_rgb failed")
    return OracleColour(view_ids, rgb, rgbf, flag)


def edge_coverage(e0: float, a: float, b: float) -> float:
    """O12: fraction of a pixel's unit square on which the linear function e0 + a x + b y is positive."""
    return float(_load().pico_edge_coverage(float(e0), float(a), float(b)))


def pixel_coverage(e, a, b) -> float:
    """O12: area of the part of a pixel's unit square on which the linear functions e[i] + a[i] x + b[i] y (at most 8) are >= 0."""
    e, a, b = (np.ascontiguousarray(x, dtype=np.float64) for x in (e, a, b))
    assert e.ndim == 1 and e.shape == a.shape == b.shape and len(e) <= 8
    return float(_load().pico_pixel_coverage(len(e), _ptr(e), _ptr(a), _ptr(b)))


def step(state: np.ndarray, actions: np.ndarray, active: Optional[np.ndarray], dt: float, wheelbase: float,
         v_max: float) -> np.ndarray:
    """One kinematic-bicycle step; state f64 [...,4] (copied), actions f32 [...,2]."""
    lib = _load()
    st = np.array(state, dtype=np.float64, order="C", copy=True)
    act = np.ascontiguousarray(actions, dtype=np.float32)
    n = st.size // 4
    assert act.size == 2 * n
    act_mask = None if active is None else np.ascontiguousarray(active, dtype=np.uint8)
    lib.pico_step(_ptr(st), _ptr(act), _ptr(act_mask), n, float(dt), float(wheelbase), float(v_max))
    return st


def f64_to_f16_bits(z: float) -> int:
    return int(_load().pico_f64_to_f16(float(z)))
