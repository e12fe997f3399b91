"""MX+ (MXFP4+) block quantization and GEMM for NVIDIA B200 (sm_100a)."""
