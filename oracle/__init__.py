"""CPU oracle of the batched egocentric rasterizer -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``pic_oracle.c`` (plain C, double precision, brute force).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the product
package never does, and this package never imports the product.
"""
from .wrapper import build, render, render_rgb, edge_coverage, pixel_coverage, step, f64_to_f16_bits, max_threads, OracleResult, OracleColour
from .occlusion import occlusion_counts

__all__ = ["build", "render", "render_rgb", "edge_coverage", "pixel_coverage", "OracleColour", "step", "f64_to_f16_bits", "max_threads", "OracleResult", "occlusion_counts"]
