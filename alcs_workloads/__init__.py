"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA path's tests and benchmark.

Holds input generators only; none of the method's arithmetic lives here.
"""
from .layers import (LayerSpec, config_layers, make_bias, make_mask, make_weights, make_x,
                     mobilenet_stack, resnet50_stack, single_layer, sweep, uniform_block_mask,
                     with_batch, zipf_block_mask)

from .conv2d import (Conv2dSpec, make_bias2d, make_mask2d, make_weights2d, make_x2d,
                     resnet18_3x3_stack)

__all__ = ["Conv2dSpec", "make_bias2d", "make_mask2d", "make_weights2d", "make_x2d", "resnet18_3x3_stack",
           "LayerSpec", "config_layers", "make_bias", "make_mask", "make_weights", "make_x",
           "mobilenet_stack", "resnet50_stack", "single_layer", "sweep", "uniform_block_mask",
           "with_batch", "zipf_block_mask"]
