"""Seeded synthetic inputs and the point sets named by the workloads.

This package holds data only: random tensors of the stated shapes and
distributions, and the interpolation point sets printed in the paper.  It
contains none of the method's arithmetic, so both the CPU oracle and the CUDA
path may draw their inputs from it without sharing code.
"""
from .points import POINT_SETS, point_set, pow2_range_scales  # noqa: F401
from .inputs import (  # noqa: F401
    ConvCase, CONFIGS, make_conv_inputs, make_vgg_inputs, VGG16_LAYERS,
)
