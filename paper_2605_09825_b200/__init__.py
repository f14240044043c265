"""B200-native MXFP4 quantize + block-scaled GEMM library (Python binding over a C ABI)."""
