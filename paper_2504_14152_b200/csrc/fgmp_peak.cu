// Tensor-core rate of this GPU for the three operand kinds the mixed GEMM's rooflines are stated
// in: an MMA-only loop (operands resident in shared memory, nothing loaded or stored), one CTA per
// SM, M = 128, N = 256 per instruction.  Gives the denominators P4 (NVFP4 with block scales), P8
// (E4M3) and P16 (bf16) of the blended roofline (Section 4.1's four block-pair products run at
// the rate of their formats at best).
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <mutex>

namespace {

constexpr int PK_THREADS = 128;
constexpr uint32_t PK_A_BYTES = 128 * 128;      // 128 rows x 128 bytes, 128-byte swizzle: four MMA K steps of 32 bytes
constexpr uint32_t PK_B_BYTES = 256 * 128;
constexpr size_t PK_SMEM = PK_A_BYTES + PK_B_BYTES + 1024 + 64;
constexpr uint32_t PK_N = 256;
constexpr uint32_t PK_SF_COL0 = 256;            // scale columns behind the accumulator (block-scaled kind only)

constexpr uint32_t PK_SW128_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
constexpr uint32_t PK_IDESC_NM = ((uint32_t)(PK_N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
constexpr uint32_t PK_IDESC_BF16 = (1u << 4) | (1u << 7) | (1u << 10) | PK_IDESC_NM;   // f32 accumulate, bf16 x bf16
constexpr uint32_t PK_IDESC_E4M3 = (1u << 4) | (0u << 7) | (0u << 10) | PK_IDESC_NM;   // f32 accumulate, E4M3 x E4M3
constexpr uint32_t PK_IDESC_NVF4 = (1u << 7) | (1u << 10) | PK_IDESC_NM;               // E2M1 x E2M1, UE4M3 scales

__device__ __forceinline__ void umma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// kind: 0 = bf16 (K = 16 per instruction), 1 = E4M3 (K = 32), 2 = NVFP4 (K = 64)
__global__ void __launch_bounds__(PK_THREADS, 1)
tensor_peak_kernel(int kind, int64_t n_mma, int* status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // offset from the array: stays known as shared memory
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + PK_A_BYTES + PK_B_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t done = smem_u32(bar);

    // operands: a fixed bit pattern of finite, mostly non-zero values in every format
    // (bf16 0x3c3b / 0xbc45 ..., E4M3 bytes with exponent field 6-8, E2M1 codes 1-7 and 9-15)
    {
        uint32_t* w = reinterpret_cast<uint32_t*>(smem);
        for (uint32_t i = threadIdx.x; i < (PK_A_BYTES + PK_B_BYTES) / 4; i += PK_THREADS) {
            uint32_t h = i * 2654435761u; h ^= h >> 15;
            uint32_t v;
            if (kind == 0)      v = 0x3c003c00u | (h & 0x807f807fu);                 // +-(1 .. 1.5) in bf16
            else if (kind == 1) v = 0x38383838u | (h & 0x87078707u) | ((h >> 3) & 0x00080008u);   // +-(1 .. 30) in E4M3
            else                v = (h & 0x77777777u) | 0x11111111u | ((h >> 7) & 0x88888888u);   // no zeros in E2M1
            w[i] = v;
        }
    }
    if (threadIdx.x == 0) {
        mbar_init(done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), 512);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (kind == 2) {
        // every block scale = 1.0 (E4M3 0x38): 16 columns for the 128 rows of A, 32 for the 256 rows of B
        uint32_t r[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = 0x38383838u;
        const uint32_t t = tmem_base + ((uint32_t)(warp * 32) << 16) + PK_SF_COL0;
        tmem_st16(t, r); tmem_st16(t + 16, r); tmem_st16(t + 32, r);
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp == 0) {
        const uint32_t a_lo = (smem_u32(smem) >> 4) | (1u << 16), b_lo = (smem_u32(smem + PK_A_BYTES) >> 4) | (1u << 16);
        if (lane == 0) {
            for (int64_t i = 0; i < n_mma; ++i) {
                const uint32_t k = (uint32_t)(i & 3) * 2u;          // 32 bytes further along K
                uint64_t ad, bd;
                asm("mov.b64 %0, {%1, %2};" : "=l"(ad) : "r"(a_lo + k), "r"(PK_SW128_HI));
                asm("mov.b64 %0, {%1, %2};" : "=l"(bd) : "r"(b_lo + k), "r"(PK_SW128_HI));
                const uint32_t acc = i ? 1u : 0u;
                if (kind == 0)      umma_f16(tmem_base, ad, bd, PK_IDESC_BF16, acc);
                else if (kind == 1) umma_f8(tmem_base, ad, bd, PK_IDESC_E4M3, acc);
                else                umma_nvf4(tmem_base, ad, bd, PK_IDESC_NVF4, tmem_base + PK_SF_COL0 + 4 * (k >> 1),
                                              tmem_base + PK_SF_COL0 + 16 + 8 * (k >> 1), acc);
            }
            umma_commit(done);
        }
        __syncwarp();
        mbar_wait(done, 0, abort_flag, status, 20);
        tc_fence_after();
    }
    __syncthreads();
    if (*abort_flag) {                                  // MMAs may still be in flight: let them drain before the tensor memory goes back
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}


// The same loop on CTA pairs: tcgen05.mma cta_group::2, M = 256 (128 rows of A per CTA), N = 256 (128 rows of B per
// CTA), issued by the pair's leader; each CTA's tensor memory holds its 128 rows of the accumulator (and, for the
// block-scaled kind, the scales of its rows of A and of all rows of B).
__device__ __forceinline__ void umma_f8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

constexpr uint32_t PKP_B_BYTES = 128 * 128;
constexpr size_t PKP_SMEM = PK_A_BYTES + PKP_B_BYTES + 1024 + 64;
constexpr uint32_t PKP_IDESC_NM = ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PK_THREADS, 1)
tensor_peak_pair_kernel(int kind, int64_t n_mma, int* status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + PK_A_BYTES + PKP_B_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t done = smem_u32(bar);
    {
        uint32_t* w = reinterpret_cast<uint32_t*>(smem);
        for (uint32_t i = threadIdx.x; i < (PK_A_BYTES + PKP_B_BYTES) / 4; i += PK_THREADS) {
            uint32_t h = (i + 7919u * rank) * 2654435761u; h ^= h >> 15;
            uint32_t v;
            if (kind == 0)      v = 0x3c003c00u | (h & 0x807f807fu);
            else if (kind == 1) v = 0x38383838u | (h & 0x87078707u) | ((h >> 3) & 0x00080008u);
            else                v = (h & 0x77777777u) | 0x11111111u | ((h >> 7) & 0x88888888u);
            w[i] = v;
        }
    }
    if (threadIdx.x == 0) {
        mbar_init(done, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_pair(smem_u32(tmem_slot), 512);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (kind == 2) {
        uint32_t r[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) r[i] = 0x38383838u;
        const uint32_t t = tmem_base + ((uint32_t)(warp * 32) << 16) + PK_SF_COL0;
        tmem_st16(t, r); tmem_st16(t + 16, r); tmem_st16(t + 32, r);
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                                     // both CTAs' operands and scales are in place
    tc_fence_after();

    if (warp == 0) {
        if (rank == 0) {
            const uint32_t a_lo = (smem_u32(smem) >> 4) | (1u << 16), b_lo = (smem_u32(smem + PK_A_BYTES) >> 4) | (1u << 16);
            if (lane == 0) {
                for (int64_t i = 0; i < n_mma; ++i) {
                    const uint32_t k = (uint32_t)(i & 3) * 2u;
                    uint64_t ad, bd;
                    asm("mov.b64 %0, {%1, %2};" : "=l"(ad) : "r"(a_lo + k), "r"(PK_SW128_HI));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(bd) : "r"(b_lo + k), "r"(PK_SW128_HI));
                    const uint32_t acc = i ? 1u : 0u;
                    if (kind == 0)      umma_f16_pair(tmem_base, ad, bd, (1u << 4) | (1u << 7) | (1u << 10) | PKP_IDESC_NM, acc);
                    else if (kind == 1) umma_f8_pair(tmem_base, ad, bd, (1u << 4) | PKP_IDESC_NM, acc);
                    else                umma_nvf4_pair(tmem_base, ad, bd, (1u << 7) | (1u << 10) | PKP_IDESC_NM,
                                                       tmem_base + PK_SF_COL0 + 4 * (k >> 1), tmem_base + PK_SF_COL0 + 16 + 8 * (k >> 1), acc);
                }
                umma_commit_pair(done, 3);
            }
            __syncwarp();
        }
        mbar_wait(done, 0, abort_flag, status, 21);     // both CTAs wait for the leader's last MMA
        tc_fence_after();
    }
    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync();
    if (warp == 0) tmem_dealloc_pair(tmem_base, 512);
}

// One CTA waits, with the library's bounded wait, for a barrier that nothing completes: the wait runs out
// after limit_ns, FGMP_ERR_TIMEOUT goes into the status word like in the GEMM kernels, and the kernel returns.
__global__ void __launch_bounds__(32, 1) wait_selftest_kernel(unsigned long long limit_ns, int* status)
{
    __shared__ uint64_t bar;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, abort_flag, status, 30, limit_ns);
    __syncwarp();
}

}  // namespace

extern "C" fgmp_status fgmp_tensor_peak(int kind, int64_t mma_per_cta, void* workspace, size_t ws_bytes, void* cuda_stream)
{
    // (at about 0.1 us per instruction 2^21 of them stay far inside the bounded wait at the end of the loop)
    const bool pair = kind >= 4;
    if (pair) kind -= 4;
    if (kind < 0 || kind > 2 || mma_per_cta < 1 || mma_per_cta > (int64_t)1 << 21 || !workspace || ws_bytes < 256 ||
        ((uintptr_t)workspace & 255)) return FGMP_ERR_INVALID_ARG;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    static std::mutex mu;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return FGMP_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lk(mu);
        if (!attr_set[dev]) {
            if (cudaFuncSetAttribute(tensor_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PK_SMEM) != cudaSuccess ||
                cudaFuncSetAttribute(tensor_peak_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PKP_SMEM) != cudaSuccess)
                return FGMP_ERR_CUDA;
            attr_set[dev] = true;
        }
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (pair) {
        tensor_peak_pair_kernel<<<(fgmp_sm_count() / 2) * 2, PK_THREADS, PKP_SMEM, s>>>(kind, mma_per_cta, reinterpret_cast<int*>(workspace));
        return fgmp_launch_status();
    }
    tensor_peak_kernel<<<fgmp_sm_count(), PK_THREADS, PK_SMEM, s>>>(kind, mma_per_cta, reinterpret_cast<int*>(workspace));
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_selftest_wait_timeout(void* workspace, size_t ws_bytes, int64_t limit_ns, void* cuda_stream)
{
    if (!workspace || ws_bytes < 256 || ((uintptr_t)workspace & 255)) return FGMP_ERR_INVALID_ARG;
    if (limit_ns < 1000 || limit_ns > 100000000) return FGMP_ERR_INVALID_ARG;      // 1 us .. 0.1 s
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>((unsigned long long)limit_ns, reinterpret_cast<int*>(workspace));
    return fgmp_launch_status();
}
