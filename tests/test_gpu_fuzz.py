"""Seeded random scenes through both sides: the CUDA path must match the oracle under the
acceptance rule and the exhaustive kernel bit for bit.  The seeds include the ones on which an
earlier sweep found depth differences above 1e-4 on planes grazing the camera centre (the tolerance
now widens with the reported conditioning) and a one-ulp depth difference on a box silhouette."""
import numpy as np
import pytest

from tests.util import compare_images, random_scene, assert_same_as_exhaustive

pytestmark = pytest.mark.gpu

SEEDS = [143, 209, 226, 294, 434, 640, 661, 904, 1236, 2306] + list(range(1000, 1050))


def test_fuzz_scenes_match_oracle_and_exhaustive_kernel():
    import torch
    import oracle
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from tests.gpu_util import CudaRun
    pixels = flagged = 0
    for i, seed in enumerate(SEEDS):
        s = random_scene(seed, full_tiles=(i % 3 == 2))
        g = CudaRun(s)
        try:
            cls, d16, d32 = g.render()
            b = g.render(brute=True)
            assert_same_as_exhaustive((cls, d16, d32), b)
            # without the float32 depth image the kernels take their vector-store paths and, for
            # images made of full tiles, their full-tile instantiations: the same images
            cls_v, d16_v, _ = g.render(depth32=False)
            assert (cls_v == cls).all() and (d16_v.view(np.uint16) == d16.view(np.uint16)).all()
            ref = oracle.render(s)
            # tiny images: allow a handful of flagged mismatches rather than a fraction
            st = compare_images(ref.cls, ref.depth, ref.flag, cls, d32, d16, max_mismatch_frac=2e-3, ref_kappa=ref.kappa)
            pixels += st["pixels"]; flagged += st["flagged"]
        except AssertionError as ex:
            raise AssertionError(f"seed {seed}: {ex}") from ex
        finally:
            g.close()
    assert flagged < 0.02 * pixels
