"""B200-native SQuant weight quantization (progressive CASE solver).

`binding` wraps the C ABI of include/squant.h; `workloads` holds seeded synthetic inputs.
The CUDA library is loaded on first use and there is no fallback when it is missing.
"""
from .binding import (FLAG_NARROW_RANGE, FLAG_PACK_INT4, NOALLOC_MAX_CTAS, MODE_C, MODE_E, MODE_EKC, MODE_K, LayerBuffers, ModelCall,
                      SquantError, alloc_outputs, load_library, squant_device_status, squant_launch_count,
                      squant_plan_info, squant_quantize_layer, squant_quantize_layer_noalloc,
                      squant_quantize_model,
                      squant_quantize_model_host, squant_selfcheck_division, squant_shutdown,
                      squant_debug_set_status, squant_debug_wait_expires, squant_debug_violations, use_library)

__all__ = ["FLAG_NARROW_RANGE", "FLAG_PACK_INT4", "NOALLOC_MAX_CTAS", "MODE_C", "MODE_E", "MODE_EKC", "MODE_K", "LayerBuffers",
           "ModelCall", "SquantError", "alloc_outputs", "load_library", "squant_device_status", "squant_launch_count",
           "squant_plan_info", "squant_quantize_layer", "squant_quantize_layer_noalloc",
           "squant_quantize_model",
           "squant_quantize_model_host", "squant_selfcheck_division", "squant_shutdown",
           "squant_debug_set_status", "squant_debug_wait_expires", "squant_debug_violations", "use_library"]
