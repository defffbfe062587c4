"""B200-native BCR sparse multiply (GEMV / GEMM / implicit-im2col conv / GRU) behind a C ABI.

`paper_2108_11033_b200.binding` loads the in-tree shared library and mirrors its entry points;
`paper_2108_11033_b200.build.build_library()` compiles it with nvcc for sm_100a.
"""
