"""Seeded synthetic workloads shared by the CPU oracle's tests and the CUDA library's tests.

This package holds no arithmetic of the method: it only describes networks as
op lists (plain tuples) and draws seeded inputs of the stated shapes.
"""
from .resnet_spec import (CONV, BNRELU, ADD, MAXPOOL, HEAD, BN, RELU, Op, resnet_v2_cifar, resnet_v2_imagenet, resnet_v1_cifar, vgg16_cifar,
                          default_cuts, CONFIGS, config, conv_sweep_shapes)
from .inputs import draw_inputs, draw_params, tensor_shapes, param_offsets
