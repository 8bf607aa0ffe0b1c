"""Seeded synthetic workloads: layer stacks, weights and videos for the RRM hot path.

This module only *describes* networks (shapes, topology) and *draws random inputs*.
It holds none of the method's arithmetic: no convolution, no delta, no quantised
inference.  Both the CPU oracle's tests and the CUDA path's tests/bench take their
inputs from here, so the two sides see byte-identical tensors.

All draws use numpy's counter-based Philox generator keyed by an integer seed.
"""
from .nets import (LayerSpec, single_conv_f32, fc6_i8, fc6_i8_pruned, alexnet_convs, resnet18_convs,
                   xnor_alexnet_convs, alexnet_full, vgg16_convs, out_hw, tensor_shapes, dense_macs,
                   with_explicit_bn, fold_bn_f32)
from .video import (block_redraw_sequence, fc_run_sequence, moving_rect_video)

__all__ = [
    "LayerSpec", "single_conv_f32", "fc6_i8", "fc6_i8_pruned", "alexnet_convs", "resnet18_convs",
    "xnor_alexnet_convs", "alexnet_full", "vgg16_convs", "out_hw", "tensor_shapes", "dense_macs",
    "with_explicit_bn", "fold_bn_f32",
    "block_redraw_sequence", "fc_run_sequence", "moving_rect_video",
]
