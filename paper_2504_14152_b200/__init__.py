"""B200-native FGMP linear layer: thin Python binding over the C-ABI library libfgmp.so.

Every step of the path runs in the CUDA kernels of the library; this package only
marshals arguments (torch tensors give device memory and streams).
"""
from .binding import (  # noqa: F401
    FgmpError, PackedTensor, OP_QUANTIZE_WEIGHTS, OP_QUANTIZE_ACTIVATIONS, OP_LINEAR, OP_CALIBRATE_TAU, OP_GLOBAL_TAU,
    OP_LINEAR_QUANTIZE, OP_LINEAR_FUSED, OP_LINEAR_CLASSES, SCORE_LP_ERROR, SCORE_HP_TO_LP, CLIP_NONE, CLIP_SW_BRUTE,
    acts_bytes, weights_bytes, workspace_bytes, workspace_init, alloc_workspace, quantize_weights, quantize_activations,
    calibrate_tau, activation_scores, weight_scores, global_tau, channel_mean_sq, linear_quantize, linear, linear_classes, linear_fused, check, unpack, version, status_string, library_path,
    profile_begin, profile_end, kernel_names, linear_static, STATIC_SCRATCH_BYTES, tensor_peak, selftest_wait_timeout,
)
