"""B200-native offloaded sparse-MoE decode step with prediction-guided expert prefetch.

The product is libspm.so (CUDA kernels for sm_100a + host runtime behind the C ABI of
include/spm.h); `binding` exposes the same entry points to Python and `model` sets up buffers.
"""
