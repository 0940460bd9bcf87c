"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA path's tests and benchmark.

Holds input generators only; none of the method's arithmetic lives here.
"""
from .layers import (LayerSpec, config_layers, make_bias, make_mask, make_weights, make_x,
                     mobilenet_stack, resnet50_stack, single_layer, sweep, uniform_block_mask,
                     with_batch, zipf_block_mask)

__all__ = ["LayerSpec", "config_layers", "make_bias", "make_mask", "make_weights", "make_x",
           "mobilenet_stack", "resnet50_stack", "single_layer", "sweep", "uniform_block_mask",
           "with_batch", "zipf_block_mask"]
