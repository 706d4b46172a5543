"""B200-native hierarchical fine-tuning (HiFT) training step.

Thin ctypes binding over libhift.so (see include/hift.h).  Every step of the
path runs in the library's CUDA kernels; Python only marshals arguments.
"""
from .binding import (HiFT, HiftError, lib, load_library, opt_step, k_linear, k_attention_fwd,
                      k_attention_bwd, k_attention_fwd_drop, k_attention_bwd_drop, k_linear_rope, k_linear_swiglu, k_linear_dx_swiglu_bwd, k_linear_gelu, k_linear_dx_gelu_bwd, k_norm_fwd, k_norm_bwd, k_norm_bwd_static, k_cross_entropy, tc_error_flag, adafactor_step,
                      code_path_switch, KERNEL_CLASSES)

__all__ = ["HiFT", "HiftError", "lib", "load_library", "opt_step", "k_linear", "k_attention_fwd",
           "k_attention_bwd", "k_attention_fwd_drop", "k_attention_bwd_drop", "k_linear_rope", "k_linear_swiglu", "k_linear_dx_swiglu_bwd", "k_linear_gelu", "k_linear_dx_gelu_bwd", "k_norm_fwd", "k_norm_bwd", "k_norm_bwd_static", "k_cross_entropy", "tc_error_flag", "adafactor_step", "code_path_switch", "KERNEL_CLASSES"]
