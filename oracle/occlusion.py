"""Occlusion of road users, as the renderer sees it -- TEST INFRASTRUCTURE, not product code.

The paper reads "the road user's occlusion percentage from the renderer" (Sec. 5.2, counterfactual
probes) without defining it.  The reading taken here: for one view and one other agent b,

    unoccluded(b) = pixels at which b's box, rendered ALONE (no map, no other agent), leaves a kept
                    fragment (steps O4, O5 of pic_oracle.c: covered, near <= z <= far),
    visible(b)    = pixels of the full render whose winning primitive (step O6) is one of b's 12
                    box triangles,
    occlusion percentage = 100 * (1 - visible / unoccluded)      (undefined where unoccluded is 0).

Both counts are written out as that definition, with the oracle's own renderer as the only step:
`visible` counts the winner indices of one render of the full scene, `unoccluded` renders a scene
that holds only the ego and b.  The ego and inactive agents have both counts 0.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import numpy as np

from .wrapper import render


def occlusion_counts(scene, view_ids: Optional[Sequence[int]] = None, poses: Optional[np.ndarray] = None
                     ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """(visible, unoccluded, slack_visible, slack_unoccluded) of the listed views, int64 [n, A] each.  The two
    slacks say by how many pixels a float32 renderer may legitimately differ: slack_unoccluded counts the pixels
    that the render of b alone flags as ambiguous (O8: on the band of its silhouette, or at the near / far plane);
    slack_visible counts the pixels flagged in the full render that b covers or whose band b's silhouette touches."""
    from scenes import custom_scene
    s = scene
    if view_ids is None:
        view_ids = np.arange(s.E * s.A * s.K, dtype=np.int64)
    view_ids = np.asarray(view_ids, dtype=np.int64)
    P = np.asarray(s.poses if poses is None else poses, dtype=np.float32)
    full = render(s, view_ids, poses=P)
    n = len(view_ids)
    visible = np.zeros((n, s.A), np.int64)
    unocc = np.zeros((n, s.A), np.int64)
    slack_v = np.zeros((n, s.A), np.int64)
    slack_u = np.zeros((n, s.A), np.int64)
    no_map = np.zeros((0, 3, 3), np.float32)
    for i, v in enumerate(view_ids):
        k, a, e = int(v % s.K), int((v // s.K) % s.A), int(v // (s.K * s.A))
        if not s.active[e, a]:
            continue
        t0, t1 = s.map_slice(e)
        n_map = t1 - t0
        idx = full.index[i]
        owner = np.where(idx >= n_map, (idx - n_map) // 12, -1)
        flagged = (full.flag[i] & 47) != 0
        for b in range(s.A):
            if b == a or not s.active[e, b]:
                continue
            visible[i, b] = int((owner == b).sum())
            alone = custom_scene(no_map, np.zeros(0, np.uint8), P[e][None, [a, b]], s.dims[e][None, [a, b]], s.rig[k:k + 1],
                                 s.H, s.W, s.near, s.far)
            r = render(alone, [0])
            cov = r.index[0] >= 0
            edge = (r.flag[0] & 5) != 0
            unocc[i, b] = int(cov.sum())
            slack_u[i, b] = int(edge.sum())
            slack_v[i, b] = int((flagged & (cov | edge)).sum())
    return visible, unocc, slack_v, slack_u
