"""Per-road-user occlusion counts (PIC_OPT_OCCLUSION) against the oracle: for a view and another agent b, the
pixels of the image won by b's box and the pixels b's box covers when drawn alone.  Integer counts: they must equal
the oracle's except by the number of pixels the oracle itself flags as ambiguous for that pair (the band around
b's silhouette, near/far plane contacts, depth ties) -- and on most pairs that number is zero."""
import numpy as np
import pytest

from scenes import make_config, make_paper_workload
from tests.util import single_env

pytestmark = pytest.mark.gpu
CAR = (4.5, 1.9, 1.5)


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from tests import gpu_util
    return gpu_util


def _gpu_counts(gu, s, brute=False, debug_flags=0, view_first=0, view_count=0):
    import torch
    import paper_2607_26005_b200 as pic
    g = gu.CudaRun(s)
    try:
        V = s.E * s.A * s.K
        occ = torch.full((V, s.A, 2), 12345, dtype=torch.int32, device=g.dev)
        g.scene.set_option(pic.OPT_OCCLUSION, occ)
        try:
            out = g.render(depth32=False, brute=brute, debug_flags=debug_flags, view_first=view_first, view_count=view_count)
        finally:
            g.scene.set_option(pic.OPT_OCCLUSION, 0)
        return occ.cpu().numpy().astype(np.int64), out
    finally:
        g.close()


def _compare(s, occ, views):
    import oracle
    vis, un, slack_v, slack_u = oracle.occlusion_counts(s, views)
    got = occ[np.asarray(views)]
    dv, du = np.abs(got[..., 0] - vis), np.abs(got[..., 1] - un)
    assert (dv <= slack_v).all(), f"visible counts off beyond the ambiguous pixels: {np.argwhere(dv > slack_v)[:5].tolist()}"
    assert (du <= slack_u).all(), f"unoccluded counts off beyond the ambiguous pixels: {np.argwhere(du > slack_u)[:5].tolist()}"
    exact = (slack_v == 0) & (slack_u == 0)
    return dict(pairs=int(vis.size), seen=int((un > 0).sum()), exact_pairs=int(exact.sum()), differing=int(((dv > 0) | (du > 0)).sum()),
                partly_hidden=int(((vis < un) & (vis > 0)).sum()), hidden=int(((un > 0) & (vis == 0)).sum()))


def test_occlusion_hand_counted(gu):
    # the oracle's closed forms: a car 12.5 m ahead = 48 pixels; half of it behind a wall that ends on the optical axis
    car = (12.5, 0.0, 0.0) + CAR
    half = [[(6.0, 0.0, -5), (6.0, 40, -5), (6.0, 40, 30)], [(6.0, 0.0, -5), (6.0, 40, 30), (6.0, 0.0, 30)]]
    s = single_env(half, [5, 5], [(0, 0, 0) + CAR, car, (20.0, 0.0, 0.0) + CAR, (30.0, 20.0, 0.0) + CAR], active=[1, 1, 1, 0])
    occ, _ = _gpu_counts(gu, s)
    assert occ[0].tolist() == [[0, 0], [24, 48], [0, 12], [0, 0]]
    assert occ[1, 0].tolist() == [0, 0] or occ[1, 0, 1] >= occ[1, 0, 0]      # view of the second car: the ego is behind it
    assert (occ[3] == 0).all()                                              # an inactive ego counts nothing
    _compare(s, occ, np.arange(4))


def test_occlusion_on_the_occluded_platoons(gu):
    s = make_config(2, E=2)
    occ, (cls, *_ ) = _gpu_counts(gu, s)
    views = np.arange(0, s.E * s.A * s.K, 7)
    st = _compare(s, occ, views)
    print("occlusion, platoons:", st)
    assert st["partly_hidden"] > 0 and st["hidden"] > 0 and st["exact_pairs"] > 0.9 * st["pairs"]
    # the visible counts of a view add up to its vehicle-class pixels
    assert (occ[..., 0].sum(1) == (cls == s.agent_class).reshape(len(cls), -1).sum(1)).all()
    # the same counts from the exhaustive kernel, from the cooperative kernel alone, and for a view sub-range
    # (the exhaustive kernel also draws the box faces turned away from the camera, which own a silhouette pixel
    # now and then where the facing face does not: a few visible counts may differ by a pixel or two)
    occ_b, _ = _gpu_counts(gu, s, brute=True)
    assert (occ_b[..., 1] == occ[..., 1]).all()
    d = np.abs(occ_b[..., 0] - occ[..., 0])
    print("exhaustive vs production visible counts: pairs differing", int((d > 0).sum()), "pixels", int(d.sum()))
    assert d.max() <= 3 and d.sum() <= 1e-3 * occ[..., 0].sum()
    occ_c, _ = _gpu_counts(gu, s, debug_flags=4)
    assert (occ_c == occ).all()
    occ_r, _ = _gpu_counts(gu, s, view_first=100, view_count=50)
    assert (occ_r[100:150] == occ[100:150]).all() and (occ_r[:100] == 12345).all() and (occ_r[150:] == 12345).all()


def test_occlusion_ragged_multi_tile_images(gu):
    s = make_paper_workload(96, 54, E=1, slots=40)
    occ, _ = _gpu_counts(gu, s)
    act = np.flatnonzero(np.repeat(s.active.reshape(-1), s.K))
    st = _compare(s, occ, act[::3])
    print("occlusion, paper rig 96x54:", st)
    assert st["seen"] > 0
