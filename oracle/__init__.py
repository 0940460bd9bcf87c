"""CPU oracle of the SIMD-structured sparse convolution (pointwise and general k x k) and of its storage format.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only tests, the smoke
check and the benchmark's CPU-baseline leg do.  It shares no code with the CUDA path.
"""
from .conv import bf16_decode, conv1x1, conv1x1_ex, conv1x1_points, conv2d, conv2d_points, num_threads
from . import latency
from .storage import flatten, pack, unpack

__all__ = ["bf16_decode", "conv1x1", "conv1x1_ex", "conv1x1_points", "conv2d", "conv2d_points", "num_threads", "latency", "pack", "unpack", "flatten"]
