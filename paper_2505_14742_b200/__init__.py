"""B200-native (sm_100a) hot path of the Quaff quantized linear layer (arxiv 2505.14742).

``synth``    seeded synthetic workloads (numpy only)
``build``    builds libquaff.so in-tree with nvcc
``binding``  ctypes binding with the C ABI's names (needs torch + a CUDA device to run)
``layer``    per-layer buffer owner that chains the entry points into one training step (+ CUDA graph of a step)
``dist``     multi-GPU plumbing of the benchmark (token-sharded replicas, no data-path collective)
"""
__all__ = ["synth", "build", "binding", "layer", "dist"]
