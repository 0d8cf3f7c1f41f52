"""CPU-only checks of the product side: the C-ABI library builds, loads and exports every entry
point the header declares; the host-side map preprocessing keeps its invariants; the multi-rank
plumbing of the benchmark works over gloo.  No compute call touches a GPU here."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "pictura.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pic_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_entry_point():
    import paper_2607_26005_b200 as pic
    lib = pic.load()
    declared = _declared_functions()
    assert len(declared) >= 12 and "pic_scene_create" in declared and "pic_render" in declared and "pic_step" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/pictura.h but not exported"
    assert set(pic.EXPORTS) <= set(declared)
    assert lib.pic_version() >= 100
    assert isinstance(lib.pic_last_error(), bytes)


def test_no_cpu_fallback():
    import torch
    import paper_2607_26005_b200 as pic
    if torch.cuda.is_available():
        pytest.skip("only meaningful on a machine without a GPU")
    with pytest.raises(RuntimeError):
        pic.Scene(1, 1, 1, 8, 8, 0.5, 100.0, [], [])


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_26005_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2607_26005_b200" not in text and "pictura" not in text


def test_map_preprocessing_invariants():
    import paper_2607_26005_b200 as pic
    from scenes import make_config
    for cfg, E in ((0, 1), (1, 2), (2, 2), (3, 1)):
        s = make_config(cfg, E=E)
        st = pic.map_stats(s.tri_xyz, s.tri_class, s.map_tri_offset, A=s.A)
        n = int(s.tri_xyz.shape[0])
        assert st["triangles"] == n
        # every map of the benchmark workloads is made of quads given as consecutive triangle pairs
        assert st["quads"] == n // 2 and st["primitives"] == n // 2
        assert st["largest_leaf"] <= 8
        assert st["prims_outside_leaf"] == 0 and st["leaves_outside_group"] == 0
        assert st["leaves"] * 8 >= st["primitives"] and st["groups"] * 32 >= st["leaves"]


def test_quad_pairing_rules():
    import paper_2607_26005_b200 as pic
    sq = [[(0, 0, 0), (1, 0, 0), (1, 1, 0)], [(0, 0, 0), (1, 1, 0), (0, 1, 0)]]
    assert pic.map_stats(sq, [2, 2])["quads"] == 1
    assert pic.map_stats(sq, [2, 3])["quads"] == 0                      # classes differ
    bent = [[(0, 0, 0), (1, 0, 0), (1, 1, 0)], [(0, 0, 0), (1, 1, 0), (0, 1, 0.5)]]
    assert pic.map_stats(bent, [2, 2])["quads"] == 0                    # not planar
    concave = [[(0, 0, 0), (2, 0, 0), (2, 2, 0)], [(0, 0, 0), (2, 2, 0), (1.8, 0.5, 0)]]
    assert pic.map_stats(concave, [2, 2])["quads"] == 0                 # fold-over: not convex
    apart = [[(0, 0, 0), (1, 0, 0), (1, 1, 0)], [(5, 0, 0), (6, 1, 0), (5, 1, 0)]]
    assert pic.map_stats(apart, [2, 2])["quads"] == 0                   # no shared edge
    other_winding = [[(0, 0, 0), (1, 0, 0), (1, 1, 0)], [(0, 1, 0), (1, 1, 0), (0, 0, 0)]]
    assert pic.map_stats(other_winding, [2, 2])["quads"] == 1
    three = sq + [[(5, 5, 0), (6, 5, 0), (6, 6, 0)]]
    st = pic.map_stats(three, [2, 2, 2])
    assert st["quads"] == 1 and st["primitives"] == 2 and st["triangles"] == 3
    empty = pic.map_stats(np.zeros((0, 3, 3)), [])
    assert empty["primitives"] == 0 and empty["groups"] == 0


_GLOO_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import numpy as np
import bench
from scenes import make_config
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# every rank renders its own environments: the shards are disjoint slices of the full workload
E = 2
mine = make_config(2, E=E, A=8, env_offset=bench.env_offset(rank, E))
full = make_config(2, E=E * world, A=8)
assert np.array_equal(mine.poses, full.poses[rank * E:(rank + 1) * E])
lo, hi = full.map_tri_offset[rank * E], full.map_tri_offset[(rank + 1) * E]
assert np.array_equal(mine.tri_xyz, full.tri_xyz[lo:hi])
# timing is the maximum over ranks
t = bench.max_over_ranks([10.0 + rank, 1.0], world, torch.device("cpu"))
assert t == [10.0 + world - 1, 1.0], t
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_two_rank_sharding_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617")
    procs = []
    for rank in range(2):
        procs.append(subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(rank), WORLD_SIZE="2"),
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for p, out in zip(procs, outs):
        assert p.returncode == 0, out
        assert "ok" in out
