"""Structured contraction ops (matmul, conv_1d_nwc_wcf, conv_2d_nhwc_hwcf) on NVIDIA B200.

The compute lives in libsg.so (hand-written CUDA for sm_100a behind the C ABI
of include/sg.h); `binding` marshals torch tensors into it, `inputs` holds the
seeded synthetic input generators, `build` compiles the library in-tree.
"""
