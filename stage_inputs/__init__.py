"""Seeded synthetic inputs for the stage training step.

This package only *describes* and *draws* inputs: layer lists of the workloads,
random tensors, initial parameter values.  It contains none of the arithmetic
of the training step itself, so both the CPU oracle and the CUDA library can be
fed from it without sharing any of the method's code.
"""
from .rng import uniform, normal, labels, tensor_key        # noqa: F401
from .nets import (Layer, OPS, inverted_residual, block_net, stage_net_mbv2_4blocks,   # noqa: F401
                   mobilenetv2_net, resnet50_c2c3_net, mobilenetv2_units,
                   partition_units, out_shape, bnfree_net, bottleneck_net,
                   small_mobilenet, forward_macs, single_unit_net, head_net, mbconv_net,
                   efficientnet_b1_stage_net)
from .params import param_layout, init_params, param_count, randomize_bn   # noqa: F401
from .bf16 import round_to_bf16, f32_to_bf16_bits, bf16_bits_to_f32   # noqa: F401
from .planner_cases import synthetic_problem   # noqa: F401
