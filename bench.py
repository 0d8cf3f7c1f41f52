#!/usr/bin/env python
"""Benchmark of the batched egocentric rasterizer: agent-steps/s and images/s on B200.

Default workload (the headline): a step is one pic_step over one batch of synthetic environments --
kinematic bicycle update of every agent, then every agent's K camera views (class u8 + depth f16)
-- on the 1024 env x 64 agent x 4 camera x 64x64 configuration (heavy-occlusion platoons on an 8x8
grid with curved connectors), driven by seeded actions.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--envs E] [--workload NAME]

--workload configs2     (default) the stepping workload above
--workload paper96x54   one chunk of 2048 egos in the paper's own shape: its four-camera rig with four
                        different mounts at 96 x 54, U{1,120} active agents per map instance; a step is
                        one pic_render of the chunk (L2 flushed between calls)

N > 1: one rank per GPU under torchrun (started here if the script was not launched by it); every
rank renders its own E environments (different seeds), there is no collective on the data path
(weak scaling).  `--impl reference` times the CPU oracle (plain C, double precision, brute force) on
the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import glob
import json
import os
import re
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

CFG = 2                       # scene of the stepping workload
ALU_LANES_PER_SM = 128        # FP32 lanes per SM
FALLBACK_HBM_GBS = 6650.0
KERNELS_PER_CALL = 5          # rig, agent, cull, render, cooperative


def _affinity_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured", float(p.get("sm_max_mhz", 1965.0))
    return FALLBACK_HBM_GBS, "fallback", 1965.0


def dram_bytes_per_view(workload: str):
    """DRAM traffic of the render path per view from the tracked ncu summary of this workload: a line
    `dram_bytes_per_view: N` in profiles/*<workload>*dram*.md (dram__bytes_read.sum + dram__bytes_write.sum of
    the cull, render and cooperative kernels of ONE call on a slice whose images exceed L2 several times, divided by
    its views).  None if no such summary is tracked."""
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", f"*{workload}*dram*.md"))):
        m = re.search(r"^dram_bytes_per_view:\s*([0-9.]+)", open(path).read(), re.M)
        if m:
            return float(m.group(1)), os.path.relpath(path, ROOT)
    return None, None


def env_offset(rank: int, envs_per_rank: int) -> int:
    """First environment of the full (weak-scaled) workload rendered by `rank`: ranks take disjoint,
    consecutive slices; there is no exchange between them."""
    return rank * envs_per_rank


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of a list of floats over all ranks (timing rule: slowest rank counts)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def _oracle_sample(scene, n_views: int, seed: int = 0, active_only: bool = False):
    """Time the oracle on a seeded sample of views; returns (seconds, views, counts[n,4])."""
    import oracle
    rng = np.random.default_rng(seed)
    total = scene.E * scene.A * scene.K
    pool = np.flatnonzero(np.repeat(scene.active.reshape(-1), scene.K)) if active_only else np.arange(total)
    views = np.sort(rng.choice(pool, size=min(n_views, len(pool)), replace=False))
    oracle.render(scene, views[:2])            # build / page in the library
    t0 = time.perf_counter()
    r = oracle.render(scene, views)
    return time.perf_counter() - t0, views, r.counts


class ClockSampler:
    """nvidia-smi in the background during the timed region (read-only queries)."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="pic_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                t = [x.strip() for x in line.split(",")]
                if len(t) < 9:
                    continue
                try:
                    sm.append(float(t[1])); mx.append(float(t[2]))
                except ValueError:
                    continue
                for name, val in zip(names, t[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            res.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(np.max(mx)), samples=len(sm))
        res["reasons"] = sorted(reasons)
        return res


def _workload_scene(args, rank: int):
    from scenes import make_config, make_paper_workload
    if args.workload == "paper96x54":
        return make_paper_workload(96, 54, egos=2048, E=args.envs, env_offset=env_offset(rank, 64))
    E = 1024 if args.envs is None else args.envs
    return make_config(CFG, E=E, env_offset=env_offset(rank, E))


def _workload_text(args, s) -> str:
    if args.workload == "paper96x54":
        return ("paper-shaped chunk rendered with pic_render: the paper's four-camera rig (four different mounts, 1545 px "
                f"focal length on 1920x1080) at {s.W}x{s.H}, {s.E} map instances (8x8 grid maps with curved connectors) x {s.A} "
                f"agent slots with U{{1,{s.A}}} active agents each = {int(s.active.sum())} egos")
    return ("configs[2] scene stepped with pic_step (configs[4] protocol): per-env 8x8 grid maps with curved connectors, "
            "8 platoons of 8, 4 cameras 64x64")


def run_reference(args, rank: int, world: int) -> None:
    """The oracle as it stands, on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    from scenes import make_config, make_paper_workload
    paper = args.workload == "paper96x54"
    scene = make_paper_workload(96, 54, E=2) if paper else make_config(CFG, E=4)
    cores = _affinity_cores()
    per_step = max(8, 2 * cores)
    for w in range(args.warmup):
        _oracle_sample(scene, 4, seed=1000 + w, active_only=paper)
    t_total, n_views = 0.0, 0
    for k in range(args.steps):
        dt, views, _ = _oracle_sample(scene, per_step, seed=k, active_only=paper)
        t_total += dt
        n_views += len(views)
    agent_steps = n_views / scene.K
    value = agent_steps / t_total
    line = {
        "impl": "reference", "metric": "agent_steps_per_s", "value": value, "unit": "agent-steps/s",
        "images_per_s": n_views / t_total, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * t_total / max(1, args.steps), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": _workload_text(args, scene) + f"; each step = {per_step} seeded views of a "
                               f"{scene.E}-environment slice, extrapolated per view",
                   "A": scene.A, "K": scene.K, "H": scene.H, "W": scene.W},
        "cpu_baseline": {"value": value, "unit": "agent-steps/s", "cores": min(cores, 64), "kind": "oracle",
                         "sample": f"{n_views} views in {args.steps} steps"},
        "e2e": {"value": value, "unit": "agent-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _series(ms) -> dict:
    ms = np.asarray(ms, dtype=np.float64)
    if not len(ms):
        return {}
    return {"first": float(ms[0]), "median": float(np.median(ms)), "last": float(ms[-1]), "min": float(ms.min()),
            "max": float(ms.max()), "mean": float(ms.mean()), "n": int(len(ms))}


def run_cuda(args, rank: int, world: int, local_rank: int) -> None:
    import torch
    import paper_2607_26005_b200 as pic
    from scenes import make_actions

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    paper = args.workload == "paper96x54"
    t_gen = time.perf_counter()
    s = _workload_scene(args, rank)
    t_gen = time.perf_counter() - t_gen
    scene = pic.Scene(s.E, s.A, s.K, s.H, s.W, s.near, s.far, s.tri_xyz, s.tri_class, map_tri_offset=s.map_tri_offset,
                      env_map_id=s.env_map_id, agent_class=s.agent_class, sky_class=s.sky_class,
                      ground_class=s.ground_class, device=local_rank)
    poses0 = torch.from_numpy(s.poses).to(dev)
    dims = torch.from_numpy(s.dims).to(dev)
    active = torch.from_numpy(s.active).to(dev)
    out_cls, out_dep = scene.alloc_outputs()
    out_bytes = out_cls.numel() + 2 * out_dep.numel()
    stream = torch.cuda.current_stream()
    # images smaller than a few L2 sizes: a 512 MB buffer is overwritten between timed calls
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device=dev) if out_bytes < 4 * 126e6 else None

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def static_calls(n: int, warm: int):
        """n pic_render calls on the initial poses, each timed by the library's own event pair around its render
        kernels; L2 flushed between calls when the images would fit it."""
        scene.set_option(pic.OPT_TIMING, 1)
        for _ in range(warm):
            scene.render(poses0, dims, s.rig, active=active, out_class=out_cls, out_depth=out_dep)
        torch.cuda.synchronize()
        scene.kernel_times()
        for _ in range(n):
            if flush is not None:
                pic.probe_fill(flush)
            scene.render(poses0, dims, s.rig, active=active, out_class=out_cls, out_depth=out_dep)
        torch.cuda.synchronize()
        kt = scene.kernel_times()
        scene.set_option(pic.OPT_TIMING, 0)
        return kt

    def colour_calls(n: int, warm: int, antialias: bool):
        """n pic_render_rgb calls (the paper's output format), timed like static_calls."""
        from scenes import default_palette
        out_rgb = torch.empty(scene.image_shape + (3,), dtype=torch.uint8, device=dev)
        scene.set_palette(default_palette())
        scene.set_option(pic.OPT_TIMING, 1)
        for _ in range(warm):
            scene.render_rgb(poses0, dims, s.rig, active=active, out_rgb=out_rgb, antialias=antialias)
        torch.cuda.synchronize()
        scene.kernel_times()
        for _ in range(n):
            if flush is not None:
                pic.probe_fill(flush)
            scene.render_rgb(poses0, dims, s.rig, active=active, out_rgb=out_rgb, antialias=antialias)
        torch.cuda.synchronize()
        kt = scene.kernel_times()
        scene.set_option(pic.OPT_TIMING, 0)
        return kt, scene.status()

    sampler = ClockSampler(local_rank)
    colour = None
    if paper:
        # ---- a step = one pic_render of the chunk; each call between its own events (L2 flushed in between)
        static_calls(0, args.warmup)
        if rank == 0:
            sampler.start()
        barrier()
        step_ms = []
        for _ in range(args.steps):
            if flush is not None:
                pic.probe_fill(flush)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            scene.render(poses0, dims, s.rig, active=active, out_class=out_cls, out_depth=out_dep)
            e1.record(stream)
            step_ms.append((e0, e1))
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        step_ms = [a.elapsed_time(b) for a, b in step_ms]
        ms_total = float(np.sum(step_ms))
        kt = static_calls(max(20, args.steps), 0)
        kt_static = kt
        if rank == 0:       # outside the timed region: the same chunk as colour images, plain and antialiased
            colour = {aa: colour_calls(20, 3, aa) for aa in (False, True)}
    else:
        # ---- the stepping workload: K consecutive pic_step calls between one pair of events
        state0 = torch.from_numpy(s.state()).to(dev)
        n_act = args.warmup + args.steps
        actions = [torch.from_numpy(make_actions(4, 1 + i, s.E, s.A)).to(dev) for i in range(n_act)]
        scene.set_state(state0, dims, active)
        scene.set_option(pic.OPT_TIMING, 1)
        for i in range(args.warmup):
            scene.step(actions[i], s.rig, out_cls, out_dep)
        torch.cuda.synchronize()
        scene.kernel_times()
        if rank == 0:
            sampler.start()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(args.steps):
            scene.step(actions[args.warmup + i], s.rig, out_cls, out_dep)
        ev1.record(stream)
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        ms_total = ev0.elapsed_time(ev1)
        kt = scene.kernel_times()
        scene.set_option(pic.OPT_TIMING, 0)
        # the same scene rendered statically from its initial poses (no drift of the geometry in view)
        kt_static = static_calls(20, 3)
    flags = scene.status()

    # ---- the roofline's denominators measured here: a write-only stream with 128-bit stores over the output
    # tensors, and a register-only FFMA loop (library microbenchmarks)
    barrier()
    pic.probe_fill(out_dep); pic.probe_fill(out_cls)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps_fill = max(3, int(2e9 // max(1, out_bytes)))
    f0.record(stream)
    for _ in range(reps_fill):
        pic.probe_fill(out_dep); pic.probe_fill(out_cls)
    f1.record(stream)
    torch.cuda.synchronize()
    fill_gbs = reps_fill * out_bytes / (f0.elapsed_time(f1) * 1e-3) / 1e9
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    ffma_out = torch.empty(sms * 2048, dtype=torch.float32, device=dev)
    pic.probe_ffma(ffma_out, 1000)
    f0.record(stream)
    n_fma = pic.probe_ffma(ffma_out, 40000)
    f1.record(stream)
    torch.cuda.synchronize()
    ffma_lane_ops = n_fma / (f0.elapsed_time(f1) * 1e-3)

    # ---- end to end through the host-buffer entry point (pinned host memory)
    n_e2e = max(1, min(args.steps, 3))
    h_poses = torch.from_numpy(s.poses.copy()).pin_memory()
    h_dims = torch.from_numpy(s.dims.copy()).pin_memory()
    h_active = torch.from_numpy(s.active.copy()).pin_memory()
    h_cls = torch.empty(scene.image_shape, dtype=torch.uint8).pin_memory()
    h_dep = torch.empty(scene.image_shape, dtype=torch.float16).pin_memory()
    args_host = (h_poses.numpy(), h_dims.numpy(), s.rig, h_cls.numpy(), h_dep.numpy())
    scene.render_host(*args_host, active=h_active.numpy())          # allocates the staging buffers
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(n_e2e):
        scene.render_host(*args_host, active=h_active.numpy())
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], world, dev)

    if rank == 0:
        n_active = int(s.active.sum())
        agents = n_active * world                       # agent-steps count active agents (all of them in configs[2])
        views_all = s.E * s.A * s.K * world
        ms_step = ms_total / args.steps
        value = agents / (ms_step * 1e-3)
        e2e_value = agents / (ms_e2e / n_e2e * 1e-3)
        hbm_peak, peak_kind, sm_max = _peaks()
        # algorithmic bytes of one render call on one GPU: 3 B per pixel written (every slot's images are
        # written, inactive ones as sky) + every map once (36 B of vertices + 1 B class per triangle) + poses,
        # sizes and activity of every agent
        px = s.E * s.A * s.K * s.H * s.W
        alg_bytes = 3 * px + 37 * int(s.tri_xyz.shape[0]) + 25 * s.E * s.A
        k_ms = float(np.mean(kt)) if len(kt) else ms_step
        achieved = alg_bytes / (k_ms * 1e-3) / 1e9
        # CPU baseline on this host: the oracle on a bounded sample of the same workload
        cores = _affinity_cores()
        n_sample = 32 * min(cores, 64)
        t_or, or_views, counts = _oracle_sample(s, n_sample, seed=12345, active_only=paper)
        cpu_value = (len(or_views) / s.K) / t_or
        # FP32-issue ceiling from the oracle's counts: 100 ops per in-frustum triangle, 8 per kept fragment,
        # 3 per pixel, over the views of active agents; peak = the FFMA loop measured above
        n_alg_view = 100.0 * counts[:, 0].mean() + 8.0 * counts[:, 2].mean() + 3.0 * s.H * s.W
        n_alg = n_alg_view * n_active * s.K + 3.0 * s.H * s.W * (s.E * s.A - n_active) * s.K
        alu_derived = sms * ALU_LANES_PER_SM * sm_max * 1e6
        t_alu = n_alg / ffma_lane_ops
        t_hbm = alg_bytes / (hbm_peak * 1e9)
        if t_hbm >= t_alu:
            roof = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                    "frac": achieved / hbm_peak, "peak_kind": peak_kind}
        else:
            ach = n_alg / (k_ms * 1e-3) / 1e12
            roof = {"bound": "alu", "achieved": ach, "peak": ffma_lane_ops / 1e12, "unit": "Tlane-op/s",
                    "frac": ach / (ffma_lane_ops / 1e12), "peak_kind": "measured: register-only FFMA loop (pic_probe_ffma)"}
        per_view, src = dram_bytes_per_view("paper96x54" if paper else "configs2")
        roof.update({
            "traffic": None if per_view is None else per_view * s.E * s.A * s.K, "traffic_source": src,
            # kernel_ms: the library's event pair around the render kernels of a call (cull_kernel, the render
            # kernel, and the cooperative kernel for tiles whose lists overflow), i.e. all the render work of a step;
            # their shares are in profiles/
            "kernel": "cull_kernel + " + ("render_kernel" if paper else "render_full_kernel") + " (+ cooperative_kernel)",
            "kernel_ms": k_ms, "kernel_ms_series": _series(kt), "kernel_launches_timed": int(len(kt)),
            "algorithmic_bytes": alg_bytes, "t_hbm_ms": 1e3 * t_hbm, "t_alu_ms": 1e3 * t_alu,
            "alg_lane_ops_per_view": float(n_alg_view), "write_only_fill_gbs": fill_gbs,
            "ffma_tlane_ops": ffma_lane_ops / 1e12, "ffma_tlane_ops_derived": alu_derived / 1e12})
        ks = np.asarray(kt_static, dtype=np.float64)
        roof_static = None
        if len(ks):
            med, mn = float(np.median(ks)), float(ks.min())
            roof_static = {"entry": "pic_render on the initial poses", "calls": int(len(ks)), "kernel_ms_median": med,
                           "kernel_ms_min": mn, "achieved_median": alg_bytes / (med * 1e-3) / 1e9, "unit": "GB/s",
                           "frac_median": alg_bytes / (med * 1e-3) / 1e9 / hbm_peak, "frac_best": alg_bytes / (mn * 1e-3) / 1e9 / hbm_peak,
                           "agent_steps_per_s_median": n_active / (med * 1e-3)}
        l2_policy = ("outputs (%.1f GB per step per GPU) exceed L2; no flush needed" % (out_bytes / 1e9)) if flush is None else \
            ("outputs are %.0f MB per call: a 512 MB buffer is overwritten between timed calls" % (out_bytes / 1e6))
        line = {
            "metric": "agent_steps_per_s", "value": value, "unit": "agent-steps/s",
            "images_per_s": agents * s.K / (ms_step * 1e-3), "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": _workload_text(args, s), "E_per_gpu": s.E, "A": s.A, "K": s.K, "H": s.H, "W": s.W,
                       "active_agents_per_gpu": n_active, "views_written": views_all, "map_triangles": int(s.tri_xyz.shape[0]),
                       "l2_policy": l2_policy, "scene_gen_s": round(t_gen, 1)},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "agent-steps/s", "h2d_bytes_per_step": 25 * s.E * s.A,
                    "d2h_bytes_per_step": 3 * px, "steps": n_e2e, "entry": "pic_render_host, pinned host buffers"},
            "gpu_launches": KERNELS_PER_CALL * args.steps,   # rig, agent, cull, render and cooperative kernels per step
            "roofline": roof,
            "roofline_static": roof_static,
            "cpu_baseline": {"value": cpu_value, "unit": "agent-steps/s", "cores": min(cores, 64), "kind": "oracle",
                             "sample": f"{len(or_views)} seeded views of this workload in {t_or:.1f} s"},
            "colour": None if colour is None else {
                "entry": "pic_render_rgb (u8 RGB, 3 B per pixel) on the same chunk; cull_kernel + colour_kernel between the library's events",
                **{("antialiased" if aa else "plain"): {
                    "kernel_ms_median": float(np.median(k)), "kernel_ms_min": float(np.min(k)), "calls": int(len(k)),
                    "agent_steps_per_s": n_active / (float(np.median(k)) * 1e-3), "images_per_s": n_active * s.K / (float(np.median(k)) * 1e-3),
                    "achieved_gbs": alg_bytes / (float(np.median(k)) * 1e-3) / 1e9, "frac": alg_bytes / (float(np.median(k)) * 1e-3) / 1e9 / hbm_peak,
                    "status_flags": int(st)} for aa, (k, st) in colour.items()}},
            "paper_context": "paper reports up to 500K agent-steps/s (2M images/s) on one H100, RGB+AA output",
            "status_flags": flags,
        }
        print(json.dumps(line), flush=True)
    scene.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def _free_port() -> int:
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100, help="timed steps (the stepping workload is defined over 100 consecutive steps)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--envs", type=int, default=None, help="environments per GPU (default: 1024 = the benchmark workload; "
                                                          "paper96x54: as many map instances as 2048 egos need)")
    ap.add_argument("--workload", default="configs2", choices=["configs2", "paper96x54"])
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else max(args.warmup, 0)
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # not started by torchrun: start the N ranks here (one process per GPU, rendezvous on the loopback)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_cuda(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
