"""Seeded synthetic workloads: layer-shape lists and input generators.

This package holds no convolution, Winograd, packing or selection arithmetic.
It only describes layer shapes and draws seeded random tensors, and it is the
one module both the CPU oracle's tests and the CUDA path's tests import.
"""
from .configs import (  # noqa: F401
    OP_CONV, OP_MAXPOOL, OP_GAVGPOOL, ACT_NONE, ACT_RELU, ACT_RELU6,
    cfg1, cfg2_resnet18, cfg3_mobilenetv2, cfg4_resnet50, cfg5_vgg16,
    CONFIGS, out_hw, conv_layers, weight_count, tiny_net,
)
from .gen import make_weights, make_input, weight_blob  # noqa: F401
