"""MX+ (MXFP4+) block quantization and GEMM for NVIDIA B200 (sm_100a).

The product is the CUDA library ``libmxp.so`` (C ABI in ``include/mxp.h``); ``binding``
marshals torch tensors into it.  Nothing here computes on the CPU.
"""
from .binding import (BF16, F32, MODE_MXFP4, MODE_MXFP4_PLUS, MODE_MXFP4_PP, MODE_MXFP6, MODE_MXFP6_PLUS, MODE_MXFP8, MODE_MXFP8_PLUS, MxpError, Packed, alloc_packed,  # noqa: F401
                      mxp_dequantize, mxp_quantize_reordered, mxp_channel_order, mxp_nvfp4_quantize, mxp_nvfp4_dequantize, mxp_gemm, mxp_gemm_noalloc, mxp_gemm_decode_chained, mxp_gemm_decode_prepack, mxp_gemm_decode_prepacked, mxp_gemm_decode_workspace_bytes, DecodeWeights, mxp_gemm_status, mxp_gemm_clock_stamp, mxp_gemm_workspace_bytes, mxp_gemm_min_workspace_bytes,
                      mxp_gemm_prepack, mxp_gemm_prepack_form, PREPACK_PLAIN, PREPACK_WIDE, PREPACK_SPLIT, PREPACK_WIDE8, PREPACK_WIDE_X2, PREPACK_WIDE8_X3, mxp_gemm_prepacked, mxp_gemm_dense_prepacked, mxp_quantize_gemm_ready, mxp_gemm_ready, mxp_wait_selftest,
                      mxp_quantize, mxp_tensor_peak_probe, mxp_debug_override, KNOB_INPLACE_KERNEL, KNOB_STREAM_HALVES, KNOB_WEIGHT_ONLY_KERNEL, KNOB_ONE_SIDED, status_string, version)
