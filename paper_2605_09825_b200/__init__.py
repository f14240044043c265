"""B200-native MXFP4 quantize + block-scaled GEMM library (Python binding over a C ABI).

``paper_2605_09825_b200.api``   ctypes binding of ``include/mxfp4.h`` (needs torch + the built .so)
``paper_2605_09825_b200.build`` in-tree nvcc build of ``libmxfp4.so`` for sm_100a
``paper_2605_09825_b200.synth`` seeded synthetic inputs (numpy only)
"""
