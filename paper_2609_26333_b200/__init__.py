"""B200-native format-disaggregated quantized linear layer (arXiv 2609.26333).

Thin ctypes binding over the C ABI in ``include/dq.h``; every step of the path
runs in the CUDA kernels of ``libdq.so``.  There is no CPU fallback: the import
of :mod:`binding` fails loudly when the library is missing.
"""
from .binding import (DQError, prefill_rmsnorm_quantize, prefill_silu_mul_quantize, prefill_gemm_silu_mul_quantize, gate_up_row_order, test_silu, rmsnorm_quantize_activations, silu_mul_quantize_activations, bench_gemm_mma_only, bench_gemm_clocks, bench_stream_read, alloc_workspace, DQWeights, FMT_LUT2, FMT_LUT3, FMT_NVFP4, FMT_NVFP4_FROM_LUT3, decode_linear, decode_linear_host, decode_linear_lut2, decode_linear_nvfp4, test_decode_linear, prefill_host_staging_bytes, prefill_linear_host,
                      export_canonical, get_status, import_canonical, import_canonical_lut2, lib, pack_weights, packed_bytes, prefill_gemm, prefill_linear, prefill_linear_static, prefill_quantize,
                      prefill_workspace_bytes, quantize_activations, status_string, version)

__all__ = ["DQError", "prefill_rmsnorm_quantize", "prefill_silu_mul_quantize", "prefill_gemm_silu_mul_quantize", "gate_up_row_order", "test_silu", "rmsnorm_quantize_activations", "silu_mul_quantize_activations", "bench_gemm_mma_only", "bench_gemm_clocks", "bench_stream_read", "alloc_workspace", "DQWeights", "FMT_LUT2", "FMT_LUT3", "FMT_NVFP4", "FMT_NVFP4_FROM_LUT3", "decode_linear", "decode_linear_host", "decode_linear_lut2", "decode_linear_nvfp4", "test_decode_linear", "prefill_host_staging_bytes", "prefill_linear_host",
           "export_canonical", "get_status", "import_canonical", "import_canonical_lut2", "lib", "pack_weights", "packed_bytes", "prefill_gemm", "prefill_linear", "prefill_linear_static", "prefill_quantize",
           "prefill_workspace_bytes", "quantize_activations", "status_string", "version"]
