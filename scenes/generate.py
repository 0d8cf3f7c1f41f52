"""Seeded synthetic driving scenes: the inputs of the batched egocentric rasterizer.

This module only *draws inputs* (map triangles, agent poses and sizes, camera rigs, actions).
It holds none of the renderer's arithmetic: no projection, no coverage test, no depth.  Both the
CPU oracle's tests and the CUDA path's tests/benchmarks take their inputs from here, so the two
sides always see byte-identical float32 arrays.

The scenes stand in for the hand-authored town maps and logged layouts the paper trains on
(Sec. 3.1), which are not redistributable here.  Shapes, sizes and densities follow the five
benchmark workloads ("configs" 0..4):

  0  1 env  x  8 agents x 1 camera  64x64   3x3 grid map, 200 m blocks
  1  256    x 32        x 4         64x64   per-env 5x5 grid, 150 m blocks, jittered nodes
  2  1024   x 64        x 4         64x64   per-env 8x8 grid, 100 m blocks, curved connectors,
                                            platoons with 8-15 m headway (heavy occlusion)
  3  64     x 64        x 4         128x256 one shared 20x20 grid + roundabouts, 150 m far plane
  4  config 2 + initial speeds and per-step (accel, steer) actions for 100 steps

Conventions (Table "camera_rig" of the paper for the frames): world z up; agent frame x forward,
y left, z up; yaw counter-clockwise about z.  All arrays are float32 unless stated.

Seeds: maps 1000*cfg + map_id, agents 1000*cfg + 500000 + env, actions 1000*cfg + 900000 + step.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

CLASS_SKY = 0
CLASS_GROUND = 1
CLASS_ROAD = 2
CLASS_MARKING = 3
CLASS_VEHICLE = 4

CLASS_SIGNAL = 6
CLASS_CYCLIST = 7
CLASS_PEDESTRIAN = 8


def default_palette() -> np.ndarray:
    """An RGB triple per class id, u8 [256,3] (input of the colour output): sky, ground, road, markings, one hue per
    kind of road user, signals; every other class a grey that depends on its id."""
    pal = np.zeros((256, 3), np.uint8)
    for c in range(256):
        pal[c] = 40 + (c * 37) % 160
    pal[CLASS_SKY] = (135, 190, 235)
    pal[CLASS_GROUND] = (96, 124, 84)
    pal[CLASS_ROAD] = (72, 72, 76)
    pal[CLASS_MARKING] = (240, 240, 230)
    pal[CLASS_VEHICLE] = (40, 110, 220)
    pal[5] = (150, 120, 100)
    pal[CLASS_SIGNAL] = (230, 40, 40)
    pal[CLASS_CYCLIST] = (240, 150, 30)
    pal[CLASS_PEDESTRIAN] = (220, 50, 200)
    return pal


ROAD_WIDTH = 7.5          # two lanes
LANE_OFFSET = 1.875       # lane centre to road centre-line
DASH_WIDTH = 0.15
DASH_LENGTH = 3.0
DASH_PERIOD = 6.0
NODE_CLEARANCE = 5.0      # no dashes this close to an intersection node
MARKING_LIFT = 0.02       # markings float 2 cm above the road so depth never ties with it
NOMINAL_DIMS = (4.5, 1.9, 1.5)   # length, width, height
MOUNT = (2.25, 0.0, 1.5)  # camera mount in the agent frame: box front, 1.5 m high

DT = 0.1                  # s, step of the kinematic update
WHEELBASE = 2.8           # m
V_MAX = 30.0              # m/s


@dataclass
class Scene:
    """One batch of environments; everything the boundary calls need, as numpy arrays."""
    name: str
    E: int
    A: int
    K: int
    H: int
    W: int
    near: float
    far: float
    num_maps: int
    env_map_id: np.ndarray        # int32 [E]
    map_tri_offset: np.ndarray    # int64 [M+1]
    tri_xyz: np.ndarray           # f32 [N,3,3]
    tri_class: np.ndarray         # u8 [N]
    poses: np.ndarray             # f32 [E,A,3]  x, y, yaw
    dims: np.ndarray              # f32 [E,A,3]  length, width, height
    active: np.ndarray            # u8 [E,A]
    rig: np.ndarray               # f32 [K,7]    mount xyz, yaw, pitch, fx, fy
    speed: np.ndarray             # f32 [E,A]    initial speed (used by the stepping workload)
    agent_class: int = CLASS_VEHICLE
    sky_class: int = CLASS_SKY
    ground_class: int = CLASS_GROUND
    cfg: int = -1
    meta: dict = field(default_factory=dict)
    agent_classes: Optional[np.ndarray] = None   # u8 [E,A]: class of each agent's box (None: agent_class for all)
    tri_vis_cos: Optional[np.ndarray] = None     # f32 [N]: cos of the largest angle off its normal from which a triangle is
                                                 # drawn, front side only (0 or None: ordinary two-sided triangle)

    @property
    def n_views(self) -> int:
        return self.E * self.A * self.K

    def map_slice(self, env: int) -> Tuple[int, int]:
        m = int(self.env_map_id[env])
        return int(self.map_tri_offset[m]), int(self.map_tri_offset[m + 1])

    def state(self) -> np.ndarray:
        """Kinematic state [E,A,4] = x, y, yaw, v."""
        return np.concatenate([self.poses, self.speed[..., None]], axis=-1).astype(np.float32)


# ----------------------------------------------------------------------------------------------
# camera rigs
# ----------------------------------------------------------------------------------------------
def focal_px(size_px: int, fov_deg: float) -> float:
    """Pinhole focal length in pixels for a field of view across `size_px` pixels (the relation
    between the paper's 1545 px focal length and its 63.7 x 38.5 degree field of view)."""
    return (size_px / 2.0) / np.tan(np.deg2rad(fov_deg) / 2.0)


def make_rig(yaws_deg, hfov_deg: float, vfov_deg: float, W: int = 64, H: int = 64, mount=MOUNT,
             pitch_deg: float = 0.0) -> np.ndarray:
    """Rig rows: mount x, y, z (agent frame, m), yaw, pitch (rad), fx, fy (pixels)."""
    rig = np.zeros((len(yaws_deg), 7), dtype=np.float32)
    for k, y in enumerate(yaws_deg):
        rig[k] = (mount[0], mount[1], mount[2], np.deg2rad(y), np.deg2rad(pitch_deg),
                  focal_px(W, hfov_deg), focal_px(H, vfov_deg))
    return rig


# ----------------------------------------------------------------------------------------------
# maps
# ----------------------------------------------------------------------------------------------
def _quads_to_tris(p0, p1, p2, p3, z: float) -> np.ndarray:
    """[Q,2] corner arrays (counter-clockwise seen from above) -> [2Q,3,3] triangles at height z."""
    q = p0.shape[0]
    tri = np.empty((q, 2, 3, 3), dtype=np.float64)
    tri[:, 0, 0, :2], tri[:, 0, 1, :2], tri[:, 0, 2, :2] = p0, p1, p2
    tri[:, 1, 0, :2], tri[:, 1, 1, :2], tri[:, 1, 2, :2] = p0, p2, p3
    tri[..., 2] = z
    return tri.reshape(2 * q, 3, 3)


def _strip_quads(a, b, half_width: float, z: float) -> np.ndarray:
    """Quads of the given half width around the segments a->b ([S,2] each)."""
    t = b - a
    ln = np.linalg.norm(t, axis=1, keepdims=True)
    t = t / ln
    n = np.stack([-t[:, 1], t[:, 0]], axis=1)           # left normal
    w = half_width
    return _quads_to_tris(a - w * n, b - w * n, b + w * n, a + w * n, z)


def _ring_quads(centre, r_in: float, r_out: float, t0: float, t1: float, nq: int, z: float) -> np.ndarray:
    """nq quads of an annulus sector around `centre` from angle t0 to t1."""
    t = np.linspace(t0, t1, nq + 1)
    c, s = np.cos(t), np.sin(t)
    inner = centre[None, :] + r_in * np.stack([c, s], axis=1)
    outer = centre[None, :] + r_out * np.stack([c, s], axis=1)
    return _quads_to_tris(inner[:-1], outer[:-1], outer[1:], inner[1:], z)


@dataclass
class GridMap:
    tri_xyz: np.ndarray       # f32 [N,3,3]
    tri_class: np.ndarray     # u8 [N]
    nodes: np.ndarray         # f64 [n,n,2]


def grid_map(seed: int, n: int, block: float, jitter: float = 0.0, arcs: bool = False,
             roundabouts: int = 0, dash_period: float = DASH_PERIOD) -> GridMap:
    """n x n intersection nodes `block` metres apart, centred on the origin.

    Triangle order: all road quads, then all centre-line dashes, then connector arcs, then
    roundabouts.  Road quads overlap at intersections (same class, so harmless).
    """
    rng = np.random.default_rng(seed)
    ax = (np.arange(n) - (n - 1) / 2.0) * block
    nodes = np.stack(np.meshgrid(ax, ax, indexing="ij"), axis=-1).astype(np.float64)  # [i,j] -> (x=ax[i], y=ax[j])
    if jitter > 0:
        nodes = nodes + rng.uniform(-jitter, jitter, size=nodes.shape)
    seg_a = np.concatenate([nodes[:-1, :].reshape(-1, 2), nodes[:, :-1].reshape(-1, 2)])
    seg_b = np.concatenate([nodes[1:, :].reshape(-1, 2), nodes[:, 1:].reshape(-1, 2)])
    parts = [_strip_quads(seg_a, seg_b, ROAD_WIDTH / 2, 0.0)]
    classes = [np.full(parts[0].shape[0], CLASS_ROAD, np.uint8)]

    # dashes: [NODE_CLEARANCE + period*i, +DASH_LENGTH] while they end NODE_CLEARANCE before the far node
    t = seg_b - seg_a
    ln = np.linalg.norm(t, axis=1)
    t = t / ln[:, None]
    max_nd = int(np.floor((ln.max() - 2 * NODE_CLEARANCE - DASH_LENGTH) / dash_period)) + 1
    if max_nd > 0:
        start = NODE_CLEARANCE + dash_period * np.arange(max_nd)                     # [D]
        ok = (start[None, :] + DASH_LENGTH) <= (ln[:, None] - NODE_CLEARANCE)        # [S,D]
        si, di = np.nonzero(ok)
        da = seg_a[si] + t[si] * start[di][:, None]
        db = da + t[si] * DASH_LENGTH
        dash = _strip_quads(da, db, DASH_WIDTH / 2, MARKING_LIFT)
        parts.append(dash)
        classes.append(np.full(dash.shape[0], CLASS_MARKING, np.uint8))

    if arcs:
        # one quarter-circle connector per node (radius 20 m, 16 quads), in a seeded quadrant
        quad = rng.integers(0, 4, size=n * n)
        flat = nodes.reshape(-1, 2)
        r = 20.0
        arc_parts = []
        for idx in range(n * n):
            sx, sy = ((1, 1), (-1, 1), (-1, -1), (1, -1))[quad[idx]]
            centre = flat[idx] + np.array([sx * r, sy * r])
            # the arc runs from the point on the node's y-road to the point on its x-road
            a0 = np.arctan2(0.0, -sx)          # direction centre -> (node.x, node.y + sy*r)
            a1 = np.arctan2(-sy, 0.0)          # direction centre -> (node.x + sx*r, node.y)
            d = (a1 - a0 + np.pi) % (2 * np.pi) - np.pi
            arc_parts.append(_ring_quads(centre, r - ROAD_WIDTH / 2, r + ROAD_WIDTH / 2, a0, a0 + d, 16, 0.0))
        arc = np.concatenate(arc_parts)
        parts.append(arc)
        classes.append(np.full(arc.shape[0], CLASS_ROAD, np.uint8))

    if roundabouts > 0:
        pick = rng.choice(n * n, size=roundabouts, replace=False)
        flat = nodes.reshape(-1, 2)
        rb = np.concatenate([_ring_quads(flat[p], 12.0, 19.5, 0.0, 2 * np.pi, 32, 0.0) for p in pick])
        parts.append(rb)
        classes.append(np.full(rb.shape[0], CLASS_ROAD, np.uint8))

    return GridMap(np.concatenate(parts).astype(np.float32), np.concatenate(classes), nodes)


# ----------------------------------------------------------------------------------------------
# agents
# ----------------------------------------------------------------------------------------------
def _agents_on_centrelines(rng, gm: GridMap, A: int, min_sep: float = 6.0):
    """Uniform positions along the road centre-lines, yaw = road heading (either way) + N(0, 0.1)."""
    nodes = gm.nodes
    seg_a = np.concatenate([nodes[:-1, :].reshape(-1, 2), nodes[:, :-1].reshape(-1, 2)])
    seg_b = np.concatenate([nodes[1:, :].reshape(-1, 2), nodes[:, 1:].reshape(-1, 2)])
    ln = np.linalg.norm(seg_b - seg_a, axis=1)
    prob = ln / ln.sum()
    pos = np.zeros((A, 2))
    yaw = np.zeros(A)
    count = 0
    tries = 0
    while count < A:
        tries += 1
        s = rng.choice(len(ln), p=prob)
        u = rng.uniform(0.0, 1.0)
        p = seg_a[s] + u * (seg_b[s] - seg_a[s])
        heading = np.arctan2(seg_b[s, 1] - seg_a[s, 1], seg_b[s, 0] - seg_a[s, 0])
        if rng.uniform() < 0.5:
            heading += np.pi
        noise = rng.normal(0.0, 0.1)
        if count and tries < 10000 and np.min(np.linalg.norm(pos[:count] - p, axis=1)) < min_sep:
            continue
        pos[count] = p
        yaw[count] = heading + noise
        count += 1
    yaw = (yaw + np.pi) % (2 * np.pi) - np.pi
    return pos, yaw


def _polyline_point(pts: np.ndarray, s: np.ndarray):
    """Point and heading at arc length s along the polyline pts [P,2]."""
    seg = pts[1:] - pts[:-1]
    ln = np.linalg.norm(seg, axis=1)
    cum = np.concatenate([[0.0], np.cumsum(ln)])
    i = np.clip(np.searchsorted(cum, s, side="right") - 1, 0, len(ln) - 1)
    u = (s - cum[i]) / ln[i]
    p = pts[i] + u[:, None] * seg[i]
    heading = np.arctan2(seg[i, 1], seg[i, 0])
    return p, heading, cum[-1]


def _agents_in_platoons(rng, gm: GridMap, A: int, per_platoon: int = 8, span: int = 3,
                        headway=(8.0, 15.0), min_sep: float = 5.0):
    """Platoons on lane centres of a span x span node neighbourhood, right-hand traffic."""
    n = gm.nodes.shape[0]
    span = min(span, n)
    i0 = rng.integers(0, n - span + 1)
    j0 = rng.integers(0, n - span + 1)
    lanes = []
    for r in range(span):
        row = gm.nodes[i0:i0 + span, j0 + r]          # varies along x
        col = gm.nodes[i0 + r, j0:j0 + span]          # varies along y
        lanes += [row, row[::-1], col, col[::-1]]
    n_platoons = (A + per_platoon - 1) // per_platoon
    order = rng.permutation(len(lanes))
    pos = np.zeros((A, 2))
    yaw = np.zeros(A)
    count = 0
    for pl in range(n_platoons):
        m = min(per_platoon, A - count)
        pts = lanes[order[pl % len(lanes)]]
        best = None
        for attempt in range(20):
            gaps = rng.uniform(headway[0], headway[1], size=m - 1) if m > 1 else np.zeros(0)
            rel = np.concatenate([[0.0], np.cumsum(gaps)])
            total = _polyline_point(pts, np.zeros(1))[2]
            s0 = rng.uniform(2.0, max(2.0 + 1e-6, total - rel[-1] - 2.0))
            p, heading, _ = _polyline_point(pts, s0 + rel)
            right = np.stack([np.sin(heading), -np.cos(heading)], axis=1)
            p = p + LANE_OFFSET * right
            best = (p, heading)
            if count == 0 or np.min(np.linalg.norm(pos[:count, None, :] - p[None, :, :], axis=2)) >= min_sep:
                break
        p, heading = best
        pos[count:count + m] = p
        yaw[count:count + m] = heading + rng.normal(0.0, 0.03, size=m)
        count += m
    yaw = (yaw + np.pi) % (2 * np.pi) - np.pi
    return pos, yaw


def _dims(rng, A: int, jitter: float) -> np.ndarray:
    d = np.tile(np.asarray(NOMINAL_DIMS, dtype=np.float64), (A, 1))
    if jitter > 0:
        d = d * rng.uniform(1.0 - jitter, 1.0 + jitter, size=d.shape)
    return d


# ----------------------------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------------------------
_CFG = {
    #      E     A   n  block jitter arcs  rb   H    W   far   hfov vfov yaws                platoons dimjit
    0: dict(E=1, A=8, n=3, block=200.0, jitter=0.0, arcs=False, rb=0, H=64, W=64, far=100.0,
            hfov=90.0, vfov=90.0, yaws=(0.0,), platoons=False, dimjit=0.0, shared=False),
    1: dict(E=256, A=32, n=5, block=150.0, jitter=10.0, arcs=False, rb=0, H=64, W=64, far=100.0,
            hfov=90.0, vfov=90.0, yaws=(0.0, 90.0, 180.0, 270.0), platoons=False, dimjit=0.1, shared=False),
    2: dict(E=1024, A=64, n=8, block=100.0, jitter=10.0, arcs=True, rb=0, H=64, W=64, far=100.0,
            hfov=90.0, vfov=90.0, yaws=(0.0, 90.0, 180.0, 270.0), platoons=True, dimjit=0.1, shared=False),
    3: dict(E=64, A=64, n=20, block=150.0, jitter=0.0, arcs=False, rb=16, H=128, W=256, far=150.0,
            hfov=96.0, vfov=40.0, yaws=(0.0, 90.0, 180.0, 270.0), platoons=True, dimjit=0.1, shared=True),
}
_CFG[4] = dict(_CFG[2])


def make_config(cfg: int, E: Optional[int] = None, A: Optional[int] = None, env_offset: int = 0) -> Scene:
    """Build workload `cfg` (0..4).  `E`/`A` shrink it for tests; `env_offset` selects which envs
    of the full workload are generated (env e of the result is env env_offset+e of the workload,
    drawn from the same per-env seeds)."""
    c = _CFG[cfg]
    E = c["E"] if E is None else int(E)
    A = c["A"] if A is None else int(A)
    base = 1000 * cfg
    maps: List[GridMap] = []
    if c["shared"]:
        maps.append(grid_map(base, c["n"], c["block"], c["jitter"], c["arcs"], c["rb"]))
        env_map_id = np.zeros(E, dtype=np.int32)
    else:
        for e in range(E):
            maps.append(grid_map(base + env_offset + e, c["n"], c["block"], c["jitter"], c["arcs"], c["rb"]))
        env_map_id = np.arange(E, dtype=np.int32)
    counts = np.array([m.tri_xyz.shape[0] for m in maps], dtype=np.int64)
    offset = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    tri_xyz = np.concatenate([m.tri_xyz for m in maps]).astype(np.float32)
    tri_class = np.concatenate([m.tri_class for m in maps]).astype(np.uint8)

    poses = np.zeros((E, A, 3), dtype=np.float32)
    dims = np.zeros((E, A, 3), dtype=np.float32)
    speed = np.zeros((E, A), dtype=np.float32)
    for e in range(E):
        rng = np.random.default_rng(base + 500000 + env_offset + e)
        gm = maps[int(env_map_id[e])]
        if c["platoons"]:
            pos, yaw = _agents_in_platoons(rng, gm, A)
        else:
            pos, yaw = _agents_on_centrelines(rng, gm, A)
        poses[e, :, :2] = pos
        poses[e, :, 2] = yaw
        dims[e] = _dims(rng, A, c["dimjit"])
        speed[e] = rng.uniform(5.0, 15.0, size=A)
    rig = make_rig(c["yaws"], c["hfov"], c["vfov"], c["W"], c["H"])
    return Scene(name=f"cfg{cfg}", E=E, A=A, K=rig.shape[0], H=c["H"], W=c["W"], near=0.5, far=c["far"],
                 num_maps=len(maps), env_map_id=env_map_id, map_tri_offset=offset, tri_xyz=tri_xyz,
                 tri_class=tri_class, poses=poses, dims=dims, active=np.ones((E, A), dtype=np.uint8),
                 rig=rig, speed=speed, cfg=cfg,
                 meta=dict(tris_per_map=counts.tolist() if len(counts) <= 8 else
                           dict(min=int(counts.min()), max=int(counts.max()), mean=float(counts.mean()))))


# ----------------------------------------------------------------------------------------------
# the paper's own workload shape: its four-camera rig at 16:9, variable agent counts, ego chunks
# ----------------------------------------------------------------------------------------------
# Table "Camera rig": per-camera mounts (ego frame, metres) and yaws; one 1545 px focal length on a
# 1920 x 1080 sensor, rendered at 96 x 54 by default (32 x 18 ... 384 x 216 in the resolution sweep).
PAPER_RIG_MOUNTS = ((1.66, -0.01, 1.49, 0.0), (1.63, 0.12, 1.48, 55.0), (1.62, -0.16, 1.49, -55.0), (-0.47, 0.02, 1.43, 180.0))
PAPER_FOCAL_PX, PAPER_SENSOR_W, PAPER_SENSOR_H = 1545.0, 1920, 1080
PAPER_SEED = 7000


def make_paper_rig(W: int = 96, H: int = 54) -> np.ndarray:
    """The paper's rig at render size W x H: front, front-left (+55 deg), front-right (-55 deg), back.  The four
    cameras have different mounts, so they do not share an origin."""
    rig = np.zeros((4, 7), dtype=np.float32)
    for k, (x, y, z, yaw) in enumerate(PAPER_RIG_MOUNTS):
        rig[k] = (x, y, z, np.deg2rad(yaw), 0.0, PAPER_FOCAL_PX * W / PAPER_SENSOR_W, PAPER_FOCAL_PX * H / PAPER_SENSOR_H)
    return rig


def make_paper_workload(W: int = 96, H: int = 54, egos: int = 2048, slots: int = 120, E: Optional[int] = None,
                        far: float = 100.0, env_offset: int = 0) -> Scene:
    """One chunk of about `egos` egos in the paper's shape (Appendix, hyper-parameter table and Sec. "Renderer
    memory usage"): map instances with a number of agents drawn from U{1, slots} each -- A = slots agent slots
    per environment, the surplus marked inactive -- rendered by the four-camera rig at 16:9.  Environments are
    added until the active agents reach `egos` (or exactly E environments if E is given).  Maps are the
    8 x 8 grids with curved connectors of workload 2 (stand-ins for the town maps); agents sit on road
    centre-lines.  Seeds: PAPER_SEED + env for maps, PAPER_SEED + 500000 + env for agents."""
    maps: List[GridMap] = []
    poses_l, dims_l, active_l = [], [], []
    n_active, e = 0, 0
    while (E is None and n_active < egos) or (E is not None and e < E):
        gm = grid_map(PAPER_SEED + env_offset + e, 8, 100.0, 10.0, True, 0)
        rng = np.random.default_rng(PAPER_SEED + 500000 + env_offset + e)
        n = int(rng.integers(1, slots + 1))
        if E is None:
            n = min(n, egos - n_active)
        pos, yaw = _agents_on_centrelines(rng, gm, slots)
        p = np.zeros((slots, 3), np.float32)
        p[:, :2] = pos
        p[:, 2] = yaw
        a = np.zeros(slots, np.uint8)
        a[:n] = 1
        maps.append(gm); poses_l.append(p); dims_l.append(_dims(rng, slots, 0.1)); active_l.append(a)
        n_active += n
        e += 1
    n_env = len(maps)
    counts = np.array([m.tri_xyz.shape[0] for m in maps], dtype=np.int64)
    return Scene(name=f"paper{W}x{H}", E=n_env, A=slots, K=4, H=H, W=W, near=0.5, far=far, num_maps=n_env,
                 env_map_id=np.arange(n_env, dtype=np.int32), map_tri_offset=np.concatenate([[0], np.cumsum(counts)]).astype(np.int64),
                 tri_xyz=np.concatenate([m.tri_xyz for m in maps]).astype(np.float32),
                 tri_class=np.concatenate([m.tri_class for m in maps]).astype(np.uint8),
                 poses=np.stack(poses_l).astype(np.float32), dims=np.stack(dims_l).astype(np.float32),
                 active=np.stack(active_l), rig=make_paper_rig(W, H), speed=np.zeros((n_env, slots), np.float32),
                 meta=dict(active_agents=int(n_active)))


def make_actions(cfg: int, step: int, E: int, A: int) -> np.ndarray:
    """Actions of one step, f32 [E,A,2]: accel ~ U[-3,2] m/s^2, steer ~ U[-0.3,0.3] rad."""
    rng = np.random.default_rng(1000 * cfg + 900000 + step)
    a = np.empty((E, A, 2), dtype=np.float32)
    a[..., 0] = rng.uniform(-3.0, 2.0, size=(E, A))
    a[..., 1] = rng.uniform(-0.3, 0.3, size=(E, A))
    return a


def disk_triangles(centre, normal, radius: float, n: int = 12) -> np.ndarray:
    """A traffic-light disk as a fan of n triangles around its centre (a regular n-gon), wound counter-clockwise
    when seen from the side its `normal` points to; f32 [n,3,3]."""
    c = np.asarray(centre, np.float64); nz = np.asarray(normal, np.float64); nz = nz / np.linalg.norm(nz)
    a = np.cross(nz, [0.0, 0.0, 1.0] if abs(nz[2]) < 0.9 else [1.0, 0.0, 0.0]); a /= np.linalg.norm(a)
    b = np.cross(nz, a)
    ang = 2 * np.pi * np.arange(n + 1) / n
    rim = c + radius * (np.cos(ang)[:, None] * a + np.sin(ang)[:, None] * b)
    return np.stack([np.stack([c, rim[i], rim[i + 1]]) for i in range(n)]).astype(np.float32)


def custom_scene(tri_xyz, tri_class, poses, dims, rig, H: int, W: int, near: float = 0.5, far: float = 100.0,
                 active=None, env_map_id=None, map_tri_offset=None, name: str = "custom", agent_classes=None,
                 tri_vis_cos=None) -> Scene:
    """Wrap hand-made arrays (tests) in a Scene.  poses/dims are [E,A,3]; one map unless offsets are given."""
    tri_xyz = np.asarray(tri_xyz, dtype=np.float32).reshape(-1, 3, 3)
    tri_class = np.asarray(tri_class, dtype=np.uint8).reshape(-1)
    poses = np.asarray(poses, dtype=np.float32)
    dims = np.asarray(dims, dtype=np.float32)
    E, A = poses.shape[:2]
    if map_tri_offset is None:
        map_tri_offset = np.array([0, tri_xyz.shape[0]], dtype=np.int64)
    map_tri_offset = np.asarray(map_tri_offset, dtype=np.int64)
    M = len(map_tri_offset) - 1
    if env_map_id is None:
        env_map_id = np.arange(E, dtype=np.int32) if M == E and M > 1 else np.zeros(E, dtype=np.int32)
    rig = np.asarray(rig, dtype=np.float32).reshape(-1, 7)
    if active is None:
        active = np.ones((E, A), dtype=np.uint8)
    return Scene(name=name, E=E, A=A, K=rig.shape[0], H=H, W=W, near=near, far=far, num_maps=M,
                 env_map_id=np.asarray(env_map_id, dtype=np.int32), map_tri_offset=map_tri_offset,
                 tri_xyz=tri_xyz, tri_class=tri_class, poses=poses, dims=dims,
                 active=np.asarray(active, dtype=np.uint8), rig=rig,
                 speed=np.zeros((E, A), dtype=np.float32),
                 agent_classes=None if agent_classes is None else np.asarray(agent_classes, np.uint8).reshape(E, A),
                 tri_vis_cos=None if tri_vis_cos is None else np.asarray(tri_vis_cos, np.float32).reshape(-1))
