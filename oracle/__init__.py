"""CPU oracle for the quantized-matmul error probe. TEST INFRASTRUCTURE ONLY.

This package is a plain, slow, obviously-correct restatement of what the probe
computes (Eq. 1 scale and quantizer, the 8-bit format rules of the Methodology
section, the descaled 8-bit matmul, and the backward error of Eq. 3), written
from the paper in numpy/fp64.  It shares no code, table or constant with the
CUDA library and must never be imported by the product path: only the tests,
the smoke check and the benchmark's CPU-baseline leg may use it.

Pins (see tests/test_oracle_*.py): printed maxima 448 / 57344 / 127, grid
cardinalities, tie enumeration, closed-form SQNR, brute-force triple loops,
on-grid zero error, scale invariance, a hand-computed 2x2x2 case; for the tensor statistics
and the Eq. 2 split (stats.py): closed-form moments of small integer arrays and of uniform /
exponential laws, scipy's skew and kurtosis, hand-worked INT8 / E4M3 examples, the half-ulp
bound on rounding RE, the class identities (counts and squared errors add up); for stochastic
rounding (rng.py, probe._quantize_stochastic): the published known-answer vectors of
Philox4x32-10, round-up frequency = distance fraction, unbiasedness, grid values fixed.
Parity unpinned: the paper prints no numeric value of Eq. 3 for any input, so
the metric is pinned only by those mathematical checks, not by a paper value.
"""
from .formats import FORMATS, decode_table, positive_grid, qmax
from .probe import (scale, quantize, dequantize, gemm_lp, gemm_ref, gemm_den,
                    metric, probe, derived, relative_error)
from .stats import tensor_stats, quantize_error

__all__ = ["FORMATS", "decode_table", "positive_grid", "qmax", "scale", "quantize",
           "dequantize", "gemm_lp", "gemm_ref", "gemm_den", "metric", "probe",
           "derived", "relative_error", "tensor_stats", "quantize_error"]
