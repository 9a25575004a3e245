"""Seeded synthetic workloads shared by the tests, the CPU oracle harness and the GPU path.

This module only *draws numbers* and *describes workloads* (tensor shapes, layer lists).
It contains none of the arithmetic of the ops themselves: no convolution, no matmul, no
padding or output-shape formula.  Both the oracle and the CUDA library are handed the same
bytes produced here, so parity never depends on how the numbers were drawn.

Generator: a counter-based 64-bit integer mixer (the SplitMix64 output function applied to
``key + (i+1) * golden_ratio_odd``), so element ``i`` of stream ``s`` of seed ``k`` is a pure
function of ``(k, s, i)`` and tensors can be produced in any order or in slices.
  * uniform[a, b): the top 24 bits of the mixed word fill a fraction in [0, 1).
  * normal: Box-Muller in float64 from two 53-bit fractions, then scaled and cast to fp32.
"""
from __future__ import annotations

import numpy as np

from .generator import mix64, uniform, normal, small_integers
from .workloads import (
    Layer,
    mobilenet_v1_layers,
    layer_channels,
    make_model_weights,
    config_matmul,
    config_separable_block,
    config_mobilenet,
    config_mobilenet_atrous,
    CONFIG_SEEDS,
)

__all__ = [
    "mix64",
    "uniform",
    "normal",
    "small_integers",
    "Layer",
    "mobilenet_v1_layers",
    "layer_channels",
    "make_model_weights",
    "config_matmul",
    "config_separable_block",
    "config_mobilenet",
    "config_mobilenet_atrous",
    "CONFIG_SEEDS",
]
