"""The paper's own workload shape (table "Camera rig", hyper-parameter table, App. "Renderer memory usage"):
the four-camera rig with four different mounts at 16:9 resolutions, a number of agents per map instance drawn
from U{1,120} (the other slots inactive), chunks of about 2048 egos, and a batch streamed in passes through
buffers bounded by a byte budget.  Images whose size is not a multiple of the 64-pixel tile take the general
kernels (ragged tiles, two tiles per 96-pixel row)."""
import numpy as np
import pytest

from scenes import make_paper_workload, make_paper_rig
from tests.util import compare_images, assert_same_as_exhaustive

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


def test_paper_rig_values():
    rig = make_paper_rig(96, 54)
    assert rig.shape == (4, 7) and np.allclose(rig[:, 5], 77.25) and np.allclose(rig[:, 6], 77.25)
    assert np.allclose(np.degrees(rig[:, 3]), [0, 55, -55, 180]) and len({tuple(r[:3]) for r in rig}) == 4


def _check(gu, s, n_oracle, n_brute, seed):
    import oracle
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        cls, d16, d32 = g.render()
        assert (cls != 255).all()
        rng = np.random.default_rng(seed)
        act_views = np.flatnonzero(np.repeat(s.active.reshape(-1), s.K))
        views = np.union1d(rng.choice(act_views, size=min(n_oracle, len(act_views)), replace=False), rng.choice(V, size=8, replace=False))
        ref = oracle.render(s, views)
        st = compare_images(ref.cls, ref.depth, ref.flag, cls[views], d32[views], d16[views])
        # inactive slots: sky class, far depth, and nobody sees them (the oracle agrees above)
        off = np.flatnonzero(np.repeat(1 - s.active.reshape(-1), s.K))
        if len(off):
            assert (cls[off] == s.sky_class).all() and (d16[off] == np.float16(s.far)).all()
        first = int(rng.integers(0, V - n_brute))
        a = g.render(view_first=first, view_count=n_brute)
        b = g.render(brute=True, view_first=first, view_count=n_brute)
        assert_same_as_exhaustive(a, b, slice(first, first + n_brute))
        return st, (cls, d16)
    finally:
        g.close()


def test_paper_rig_96x54_three_map_instances(gu):
    s = make_paper_workload(96, 54, E=3)
    assert s.K == 4 and 0 < s.active.sum() < s.E * s.A
    st, _ = _check(gu, s, n_oracle=160, n_brute=240, seed=1)
    print("paper 96x54, 3 instances:", st)


def test_paper_rig_384x216(gu):
    s = make_paper_workload(384, 216, E=1, slots=24)
    st, _ = _check(gu, s, n_oracle=10, n_brute=8, seed=2)
    print("paper 384x216:", st)


def test_paper_chunk_of_2048_egos_and_streaming_in_passes(gu):
    """The full chunk (about 31 map instances x 120 slots x 4 cameras at 96 x 54) in one call against the oracle
    on sampled views, then streamed in passes through buffers of at most 24 MB: the streamed images must equal
    the one-shot images bit for bit, the pass count must follow from the byte budget."""
    import torch
    s = make_paper_workload(96, 54)
    assert s.meta["active_agents"] == 2048
    st, (cls, d16) = _check(gu, s, n_oracle=128, n_brute=256, seed=3)
    print("paper chunk:", st)
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        budget = 24 * 1000 * 1000
        per_pass = budget // (3 * s.H * s.W)
        got_c = np.full((V, s.H, s.W), 255, np.uint8)
        got_d = np.zeros((V, s.H, s.W), np.float16)
        seen = []

        def consume(first, n, c, d):
            assert c.shape == (n, s.H, s.W) and n <= per_pass
            got_c[first:first + n] = c.cpu().numpy()
            got_d[first:first + n] = d.cpu().numpy()
            seen.append((first, n))

        passes = g.scene.render_in_passes(g.poses, g.dims, s.rig, consume, budget, active=g.active)
        assert passes == -(-V // per_pass) == len(seen) and passes > 1
        assert sum(n for _, n in seen) == V and seen[-1][1] == V - per_pass * (passes - 1)
        assert (got_c == cls).all() and (got_d.view(np.uint16) == d16.view(np.uint16)).all()
        # the options are back to their defaults: an ordinary call renders everything again
        c2, d2, _ = g.render(depth32=False)
        assert (c2 == cls).all()
    finally:
        g.close()
