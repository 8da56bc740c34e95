"""B200-native ROCKET transform: thin Python binding over the C-ABI CUDA library.

The binding only marshals arguments; every step of the transform runs in the CUDA kernels
of librocket_b200.so.  There is no CPU fallback: importing works without a GPU (so the build
can be checked), but every compute call needs a CUDA device and the compiled library.
"""
from .binding import (MiniRocket, PASS_BACKWARD, PASS_HARD, PASS_SOFT, PASS_U8_INPUT, RocketError, RocketParams, device_alloc_count,
                      kernel_launch_count, library_path, load_library,
                      rocket_ridge_fit, rocket_ridge_predict,
                      rocket_transform, rocket_transform_f16, rocket_transform_soft, rocket_transform_soft_backward, rocket_transform_soft_u8,
                      rocket_transform_u8)

__all__ = ["MiniRocket", "PASS_BACKWARD", "PASS_HARD", "PASS_SOFT", "PASS_U8_INPUT", "RocketError", "RocketParams",
           "device_alloc_count", "kernel_launch_count", "library_path", "load_library",
           "rocket_ridge_fit", "rocket_ridge_predict",
           "rocket_transform", "rocket_transform_f16", "rocket_transform_soft", "rocket_transform_soft_backward", "rocket_transform_soft_u8",
           "rocket_transform_u8"]
