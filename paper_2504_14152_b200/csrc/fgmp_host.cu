// Host utilities: device capability check, status strings, size queries.
#include "fgmp_common.cuh"
#include "fgmp_host.h"

namespace {
struct DevInfo { int checked; int major; int sms; };
DevInfo g_dev[64];
DevInfo* cur_dev()
{
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= 64) return nullptr;
    DevInfo* i = &g_dev[d];
    if (!i->checked) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, d) != cudaSuccess) return nullptr;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, d) != cudaSuccess) return nullptr;
        i->major = major; i->sms = sms; i->checked = 1;
    }
    return i;
}
}  // namespace

fgmp_status fgmp_require_sm100()
{
    DevInfo* i = cur_dev();
    if (!i) return FGMP_ERR_CUDA;
    return i->major == 10 ? FGMP_OK : FGMP_ERR_ARCH;
}

int fgmp_sm_count()
{
    DevInfo* i = cur_dev();
    return i ? i->sms : 148;
}

fgmp_status fgmp_launch_status()
{
    return cudaGetLastError() == cudaSuccess ? FGMP_OK : FGMP_ERR_CUDA;
}

extern "C" const char* fgmp_status_string(fgmp_status s)
{
    switch (s) {
        case FGMP_OK: return "ok";
        case FGMP_ERR_INVALID_ARG: return "invalid argument";
        case FGMP_ERR_SHAPE: return "unsupported shape, leading dimension or alignment";
        case FGMP_ERR_WORKSPACE: return "workspace or output buffer too small";
        case FGMP_ERR_CUDA: return "CUDA call failed";
        case FGMP_ERR_ARCH: return "device is not sm_100";
        case FGMP_ERR_TIMEOUT: return "device-side wait timed out";
        case FGMP_ERR_CAPACITY: return "more FP8 blocks than the packed buffer can hold";
    }
    return "unknown status";
}

extern "C" int fgmp_version(void) { return 1; }

extern "C" size_t fgmp_weights_bytes(int64_t N, int64_t K, int64_t max_fp8_blocks)
{
    if (N < 1 || K < 64 || (K % 64) != 0 || max_fp8_blocks < 0 || max_fp8_blocks > N * (K / 16)) return 0;
    return fgmp_layout(N, K, 1, max_fp8_blocks).total;
}

extern "C" size_t fgmp_acts_bytes(int64_t M, int64_t K)
{
    if (M < 1 || K < 64 || (K % 64) != 0) return 0;
    return fgmp_layout(M, K, 0, 0).total;
}
