"""Seeded synthetic inputs for the ROCKET transform: series and kernel parameters.

This module is the only code that both the CUDA path's tests and the CPU oracle's
tests consume.  It holds input generation only (random series, random kernel
parameters drawn by the rules of Section 3.1); none of the transform's arithmetic
(convolution, pooling, gradients) lives here.
"""
from .rng import counter_u64, counter_uniform
from .kernels import KernelParams, generate_kernels, kernels_from_lists
from .minirocket import MiniParams, generate_minirocket
from .series import (random_walk_series, ar1_spike_series, normal_array, intensity_series_u8,
                     channel_statistics)

__all__ = [
    "counter_u64", "counter_uniform", "KernelParams", "generate_kernels",
    "kernels_from_lists", "random_walk_series", "ar1_spike_series", "normal_array",
    "intensity_series_u8", "channel_statistics", "MiniParams", "generate_minirocket",
]
