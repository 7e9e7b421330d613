"""Seeded synthetic inputs for the SPARQ hot path.

This module only draws random tensors and lists workload shapes.  It holds
none of the method's arithmetic (no window selection, no rounding, no
matrix product), so both the CPU oracle's tests and the CUDA path's tests
may use it without sharing anything that is under test.

Value recipe (stands in for post-ReLU ResNet activations quantized to 8 bits
with a symmetric min-max scheme, Section 5 of the paper):

* activations: exact zeros with probability ``zero_frac``; the rest are a
  discrete half-normal ``clip(round(|N(0,1)| * 40), 1, 255)``;
* weights: ``clip(round(N(0,1) * 30), -127, 127)`` (signed, symmetric);
* per-output-channel scale: ``U(0.001, 0.01)``, bias: ``U(-1, 1)``.
"""
from .generators import (  # noqa: F401
    activations,
    weights,
    scales,
    bias,
    ConvShape,
    resnet50_conv_layers,
    conv_out_hw,
    inv_out_scale,
    sparse24_weights,
    sparse24_dense,
)
