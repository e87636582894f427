// Host utilities: device capability check, status strings, size queries.
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include <vector>
#include <mutex>

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

// ------------------------------------------------------------------ launch accounting
namespace {
struct ProfRec { int id; cudaEvent_t a, b; };
std::mutex g_prof_mu;
bool g_prof_on = false;
unsigned g_prof_mask = 0;
long long g_prof_count[FGMP_K_COUNT];
std::vector<ProfRec> g_prof_recs;
std::vector<cudaEvent_t> g_event_pool;
const char* const g_kernel_names[FGMP_K_COUNT] = {
    "quant_act", "act_aux", "unpack", "expand_acts", "expand_weights", "gemm_bf16_tcgen05",
    "w_amax", "w_score_clip", "select", "w_mask", "scan", "w_emit", "w_aux", "act_scores", "decode_gemm", "gemm_nvfp4_tcgen05"};
cudaEvent_t get_event()
{
    if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}
}  // namespace

FgmpLaunchScope::FgmpLaunchScope(int id_, cudaStream_t s_) : id(id_), s(s_), stop(nullptr)
{
    if (!g_prof_on) return;
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_count[id]++;
    if (g_prof_mask & (1u << id)) {
        ProfRec r{id, get_event(), get_event()};
        if (r.a && r.b) {
            cudaEventRecord(r.a, s);
            stop = r.b;
            g_prof_recs.push_back(r);
        }
    }
}

FgmpLaunchScope::~FgmpLaunchScope()
{
    if (stop) cudaEventRecord(stop, s);
}

extern "C" int fgmp_profile_begin(unsigned timed_kernel_mask)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    for (int i = 0; i < FGMP_K_COUNT; ++i) g_prof_count[i] = 0;
    for (auto& r : g_prof_recs) { g_event_pool.push_back(r.a); g_event_pool.push_back(r.b); }
    g_prof_recs.clear();
    g_prof_mask = timed_kernel_mask;
    g_prof_on = true;
    return FGMP_K_COUNT;
}

extern "C" int fgmp_profile_end(int n, long long* launches, float* ms_total)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = false;
    for (int i = 0; i < n && i < FGMP_K_COUNT; ++i) { launches[i] = g_prof_count[i]; ms_total[i] = 0.f; }
    for (auto& r : g_prof_recs) {
        float ms = 0.f;
        if (cudaEventSynchronize(r.b) == cudaSuccess && cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess && r.id < n)
            ms_total[r.id] += ms;
        g_event_pool.push_back(r.a); g_event_pool.push_back(r.b);
    }
    g_prof_recs.clear();
    return FGMP_K_COUNT;
}

extern "C" const char* fgmp_kernel_name(int id)
{
    return (id >= 0 && id < FGMP_K_COUNT) ? g_kernel_names[id] : "";
}
