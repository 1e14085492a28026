"""B200-native W4A4 linear path of QuantVGGT's Dual-Smoothed Fine-Grained Quantization.

CUDA kernels (sm_100a) behind a C ABI (include/qvggt.h) plus this thin binding.
"""
from .binding import (EXPORTS, rotate_smooth_quantize_c8_expand, w4a4_linear_c8_expanded, rotate_smooth_quantize_c8_grouped, w4a4_linear_c8_grouped, w4a4_linear_c8_packed_weights, gelu, gelu_rotate_smooth_quantize_c8, rotate_smooth_quantize_tc, debug_starved_linear_c8, layernorm, layernorm_rotate_smooth_quantize_c8, QvggtError, Weights, calibrate_smooth, lib, prepare_weights,
                      quantize_weights_static, rotate_smooth_quantize, rotate_smooth_quantize_c8, rotate_smooth_quantize_static_c8, w4a4_linear,
                      w4a4_linear_c8)
from .buildlib import build

__all__ = ["EXPORTS", "QvggtError", "Weights", "calibrate_smooth", "lib", "prepare_weights",
           "rotate_smooth_quantize", "w4a4_linear", "build", "quantize_weights_static",
           "rotate_smooth_quantize_c8", "w4a4_linear_c8", "rotate_smooth_quantize_static_c8", "layernorm", "layernorm_rotate_smooth_quantize_c8", "debug_starved_linear_c8", "rotate_smooth_quantize_tc", "gelu", "gelu_rotate_smooth_quantize_c8", "w4a4_linear_c8_packed_weights", "rotate_smooth_quantize_c8_grouped", "w4a4_linear_c8_grouped", "rotate_smooth_quantize_c8_expand", "w4a4_linear_c8_expanded"]
