"""Seeded synthetic workloads: architecture tables and random tensors.

This package only *describes* networks (plain lists of layer dictionaries) and
draws random arrays.  It holds none of the method's arithmetic (no folding, no
quantizer, no convolution, no arithmetic-intensity formula), so both the CPU
oracle's tests and the CUDA library's binding may consume its output as data.
"""
from .archs import (resnet20, mobilenet_v2, conv_layer_indices, tiny_net,  # noqa: F401
                    heavy_early_resnet20, plain_convnet20, depthwise_stack,
                    pointwise_stack, inverted_residual_stack)
from .gen import (  # noqa: F401
    gen_model,
    gen_images,
    gen_random_scheme,
    one_layer_lowered_schemes,
    coordinate_step_schemes,
    mixed_int4_int8_scheme,
    gen_linear_case,
)
