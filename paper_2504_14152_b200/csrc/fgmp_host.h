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
