"""Causal linear attention with a causal depthwise-convolution branch: CUDA kernels for
sm_100a behind a C-ABI library, plus the Python binding that marshals arguments."""
