// Host-side helpers shared by the translation units of libfgmp.
#pragma once
#include <cuda_runtime.h>
#include "fgmp.h"

// FGMP_OK iff the current device is compute capability 10.x (cached per device)
fgmp_status fgmp_require_sm100();
// turns the last launch error into a status
fgmp_status fgmp_launch_status();
// number of SMs of the current device (cached)
int fgmp_sm_count();
// workspace sizes of the individual operations
size_t fgmp_ws_quantize_weights(int64_t N, int64_t K);
size_t fgmp_ws_calibrate(int64_t M, int64_t K);
size_t fgmp_ws_linear(int64_t M, int64_t N, int64_t K);
size_t fgmp_ws_linear_quantize(int64_t M, int64_t N, int64_t K);
size_t fgmp_ws_linear_fused(int64_t M, int64_t N, int64_t K);
size_t fgmp_ws_linear_classes(int64_t M, int64_t N, int64_t K);
size_t fgmp_ws_global_tau(int64_t total_scores);
// weight-streaming kernel for M <= 16 tokens and K % 256 == 0
bool fgmp_decode_supported(int64_t M, int64_t N, int64_t K);
size_t fgmp_ws_decode(int64_t M, int64_t N, int64_t K);
fgmp_status fgmp_linear_decode(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                               int64_t M, int64_t N, int64_t K, void* workspace, bool clear_first, cudaStream_t s);

// all-NVFP4 prefill GEMM (fgmp_gemm4.cu): decides on the device whether it applies, answer in status[2]
fgmp_status fgmp_launch_gemm_nvfp4(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                                   int64_t M, int64_t N, int64_t K, int* status, cudaStream_t s);

// ---- the FP8 tensor scale of a call (fgmp_scales): given on its own, or scale_fp4 * 2^ratio ----
#include <math.h>
inline bool fgmp_scales_valid(const fgmp_scales& sc)
{
    return sc.fp8_log2_ratio >= -7 && sc.fp8_log2_ratio <= 7 && sc.scale_fp8 >= 0.f && isfinite(sc.scale_fp8);
}
inline bool fgmp_fp8_free(const fgmp_scales& sc) { return sc.scale_fp8 > 0.f; }
inline float fgmp_fp8_scale(const fgmp_scales& sc) { return sc.scale_fp8 > 0.f ? sc.scale_fp8 : ldexpf(sc.scale_fp4, sc.fp8_log2_ratio); }

// ---- launch accounting (see fgmp_profile_begin in fgmp.h) ----
enum FgmpKernelId {
    FGMP_K_ACT_QUANT = 0, FGMP_K_ACT_AUX, FGMP_K_UNPACK, FGMP_K_EXPAND_A, FGMP_K_EXPAND_W, FGMP_K_GEMM_BF16,
    FGMP_K_W_AMAX, FGMP_K_W_SCORE, FGMP_K_SELECT, FGMP_K_W_MASK, FGMP_K_SCAN, FGMP_K_W_EMIT, FGMP_K_W_AUX,
    FGMP_K_ACT_SCORES, FGMP_K_DECODE, FGMP_K_GEMM_NVFP4, FGMP_K_COUNT
};
// Brackets one kernel launch: counts it and, when event timing of this kernel id is on,
// records a CUDA event before and after it on the launch stream.
struct FgmpLaunchScope {
    int id; cudaStream_t s; cudaEvent_t stop;
    FgmpLaunchScope(int id, cudaStream_t s);
    ~FgmpLaunchScope();
};
#define FGMP_LAUNCH(id, stream, ...) do { FgmpLaunchScope fgmp_scope_(id, stream); __VA_ARGS__; } while (0)
