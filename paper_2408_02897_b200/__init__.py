"""Quantized-matmul error probe for B200: Python binding over the C-ABI library libqm.so.

The binding only marshals arguments; every step of the probe runs in the CUDA kernels.
Importing the package does not load the library; the first call does, and fails loudly if
the library has not been built (python -m paper_2408_02897_b200.build).
"""
from .binding import (FMT, GRAN, REF, QmError, MetricResult, lib, qm_code_ld, qm_scale, qm_scale_shared, qm_quantize, qm_quantize_formats,
                      qm_gemm, qm_gemm_ref, qm_metric, qm_tensor_stats, qm_quantize_error, TensorStats, QuantError, qm_metric_noalloc, qm_probe_layer, qm_probe_layer2, ProbePlan2, qm_probe_layer_host,
                      qm_workspace_bytes, operand_of, ProbePlan, ProbeBatch, HostProbeBatch,
                      kernel_launches,
                      profile_enable, profile_read, profile_samples)

__all__ = ["FMT", "GRAN", "REF", "QmError", "MetricResult", "lib", "qm_code_ld", "qm_scale", "qm_scale_shared",
           "qm_quantize", "qm_quantize_formats", "qm_gemm", "qm_gemm_ref", "qm_metric", "qm_tensor_stats", "qm_quantize_error",
           "TensorStats", "QuantError", "qm_metric_noalloc", "qm_probe_layer",
           "qm_probe_layer_host", "qm_probe_layer2", "ProbePlan2", "qm_workspace_bytes", "operand_of", "ProbePlan", "ProbeBatch",
           "HostProbeBatch", "kernel_launches",
           "profile_enable", "profile_read", "profile_samples"]
