// fgmp_linear: the mixed-precision GEMM (Section 4.1 of the paper).
//
// General path ("common container"): every block of both operands, whatever its format, is
// an exact bf16 number once its microscale is folded in (E2M1 x E4M3 scale has at most 6
// significant bits, E4M3 has 4).  A streaming pass expands the packed operands into bf16
// planes, and a persistent tcgen05 kernel multiplies them with FP32 accumulation in TMEM;
// the two FP32 tensor scales are applied in the epilogue.  All four block-pair products of
// the paper's datapath (FP4xFP4, FP4xFP8, FP8xFP4, FP8xFP8) are therefore exact products.
//
// Kernel structure (one CTA per SM, 192 threads):
//   warp 0    : TMA producer   (global -> 128B-swizzled shared tiles, mbarrier complete_tx)
//   warp 1    : MMA issuer     (tcgen05.mma kind::f16, accumulators in TMEM, double buffered)
//   warps 2-5 : epilogue       (tcgen05.ld -> scale -> global), overlapped with the next tile
// Every wait on an mbarrier is bounded; on expiry the CTA records FGMP_ERR_TIMEOUT and leaves.
#include <cuda.h>
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <mutex>

namespace {

// ------------------------------------------------------------------ expand to bf16 planes
// plane[r, k] = e2m1 * e4m3scale (NVFP4 block) or e4m3 * 2^ratio (FP8 block); exact in bf16.
__device__ __forceinline__ void e4m3x16_scaled(const uint4& c, float r8, float (&v)[16])
{
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 a = e4m3x2_to_f32x2(w[i] & 0xffff), bb = e4m3x2_to_f32x2(w[i] >> 16);
        v[4 * i] = a.x * r8; v[4 * i + 1] = a.y * r8; v[4 * i + 2] = bb.x * r8; v[4 * i + 3] = bb.y * r8;
    }
}

__device__ __forceinline__ void store_256(void* dst, const uint32_t (&o)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
}

// 16 values that are exact in bf16 (the low 16 bits of every float are zero) -> 32 bytes
__device__ __forceinline__ void store_bf16x16(uint4* dst, const float (&v)[16])
{
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
        o[i] = (__float_as_uint(v[2 * i]) >> 16) | (__float_as_uint(v[2 * i + 1]) & 0xffff0000u);
    store_256(dst, o);        // one 32-byte store (the planes are 32-byte aligned and a block is 32 bytes): whole sectors per lane
}

__device__ __forceinline__ void nvfp4x16_scaled(const uint2& c, uint32_t scale_code, float (&v)[16])
{
    const float d = e4m3_to_f32(scale_code);
    const uint32_t w[2] = {c.x, c.y};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float2 q = e2m1x2_to_f32x2((w[i >> 2] >> ((i & 3) * 8)) & 0xff);
        v[2 * i] = q.x * d; v[2 * i + 1] = q.y * d;
    }
}

// A packed tensor is read only if its header describes the tensor the call was given; otherwise the
// status word of the workspace says so and the kernel leaves.
// cls: 0 = every block on the NVFP4 tensor scale (needs the power-of-two tie of the two scales), 1 / 2 = only the
// NVFP4 / only the FP8 blocks, each over its own tensor scale (the per-class passes of fgmp_linear_classes)
__device__ __forceinline__ bool header_matches(const fgmp_packed_header* h, int64_t rows, int64_t K, uint32_t kind, int* status, int where, int cls = 0)
{
    const bool ok = h->magic == FGMP_MAGIC && h->version == 7u && h->rows == rows && h->K == K && h->kind == kind && h->error == 0 &&
                    (cls != 0 || h->fp8_scale_free == 0);
    if (!ok && threadIdx.x == 0) { atomicCAS(status, 0, (int)FGMP_ERR_INVALID_ARG); atomicExch(status + 1, where); }
    return ok;
}

// packed activations -> bf16 plane; one thread per block
__global__ void __launch_bounds__(256) expand_kernel(const uint8_t* blob, int64_t rows, int64_t K, uint4* plane, int* status, int cls)
{
    if (status[2]) return;                              // the all-NVFP4 GEMM has produced the result already
    const fgmp_packed_header* h = reinterpret_cast<const fgmp_packed_header*>(blob);
    if (!header_matches(h, rows, K, 0u, status, 11, cls)) return;
    const PackedLayout L = fgmp_layout(rows, K, 0, 0);
    const uint32_t* pmask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const float r8 = cls ? 1.0f : __int_as_float((127 + h->fp8_log2_ratio) << 23);
    const int64_t nblk = rows * L.KB;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblk; b += (int64_t)gridDim.x * blockDim.x) {
        int64_t r = b / L.KB, kb = b % L.KB;
        uint32_t word = pmask[r * L.MW + (kb >> 5)];
        bool is8 = (word >> (kb & 31)) & 1;
        float v[16];
        if (is8) e4m3x16_scaled(*reinterpret_cast<const uint4*>(blob + L.off_codes8 + (size_t)(r * K + kb * 16)), r8, v);
        else nvfp4x16_scaled(*reinterpret_cast<const uint2*>(blob + L.off_codes4 + (r * K) / 2 + kb * 8),
                             blob[L.off_sf + fgmp_sf_offset(r, kb, K)], v);
        if (cls && (is8 != (cls == 2))) {               // a block of the other class
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
        }
        store_bf16x16(plane + (r * K) / 8 + kb * 2, v);
    }
}

// packed weights -> bf16 plane; one CTA of 128 threads per unit record, consecutive threads on
// consecutive blocks of one row, four blocks per thread in flight at a time
__global__ void __launch_bounds__(128) expand_w_kernel(const uint8_t* __restrict__ blob, int64_t rows, int64_t K, uint4* __restrict__ plane, int* status, int cls)
{
    __shared__ UnitScratch sc;
    if (status[2]) return;                              // the all-NVFP4 GEMM has produced the result already
    const fgmp_packed_header* h = reinterpret_cast<const fgmp_packed_header*>(blob);
    if (!header_matches(h, rows, K, 1u, status, 12, cls)) return;
    const PackedLayout L = fgmp_layout(rows, K, 1, 0);
    const float r8 = cls ? 1.0f : __int_as_float((127 + h->fp8_log2_ratio) << 23);
    const int64_t unit = blockIdx.x, tile = unit / L.chunks, c = unit % L.chunks;
    const uint32_t* mask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const uint32_t m16 = fgmp_chunk_mask(mask, L, tile * 128 + threadIdx.x, c);
    const uint32_t cnt = fgmp_unit_positions(m16, sc.warp, sc.pos, sc.cnt);
    const uint8_t* rec = blob + L.off_rec + (size_t)unit * REC_BYTES;
    const uint8_t* halves = blob + L.off_ovf + (size_t)reinterpret_cast<const uint32_t*>(blob + L.off_uptr)[unit] * 16 + fgmp_list_halves_offset(cnt);
    const int j = threadIdx.x & 15;
    const int64_t kb = c * 16 + j;
    if (kb >= L.KB) return;
#pragma unroll 1
    for (int i0 = 0; i0 < 16; i0 += 4) {
        uint2 slot[4], hi[4];
        uint32_t sfb[4], pos[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = (threadIdx.x >> 4) + 8 * (i0 + i);
            pos[i] = sc.pos[row * 16 + j];
            slot[i] = __ldg(reinterpret_cast<const uint2*>(rec + REC_W4 + fgmp_rec_w4_offset(row, j)));
            sfb[i] = __ldg(rec + REC_SF + fgmp_rec_sf_offset(row, j));
            hi[i] = make_uint2(0u, 0u);
            if (pos[i] != 0xffffu) hi[i] = __ldg(reinterpret_cast<const uint2*>(halves + (size_t)pos[i] * 8));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = (threadIdx.x >> 4) + 8 * (i0 + i);
            const int64_t r = tile * 128 + row;
            if (r >= L.rows) continue;
            float v[16];
            if (pos[i] != 0xffffu) e4m3x16_scaled(make_uint4(slot[i].x, slot[i].y, hi[i].x, hi[i].y), r8, v);
            else nvfp4x16_scaled(slot[i], sfb[i], v);
            if (cls && ((pos[i] != 0xffffu) != (cls == 2))) {
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = 0.f;
            }
            store_bf16x16(plane + (r * K) / 8 + kb * 2, v);
        }
    }
}

// ------------------------------------------------------------------ bf16 tcgen05 GEMM on CTA pairs
// Two CTAs of a cluster share one 256 x 256 output tile: each loads its 128 rows of A and its half
// (128 rows) of B, the pair's leader issues tcgen05.mma cta_group::2 (M = 256), which reads both
// halves of B from the two shared memories, and each CTA's TMEM holds the accumulators of its own
// 128 rows.  B is fetched once per pair: a stage is 32 KiB per CTA for 256 x 256 x 64 of math (a single
// CTA with a 128 x 256 tile needs 48 KiB for half of that), which is what the L2 -> shared-memory path can
// sustain.  No TMA multicast.  Persistent: warp 0 = TMA producer, warp 1 = MMA issuer (leader CTA
// only) and TMEM owner, warps 2-5 = epilogue; two accumulator buffers of 256 TMEM columns.
constexpr int BK = 64;                              // BK bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int GEMM_THREADS = 192;
constexpr int P_BM = 256, P_BN = 256;               // per pair
constexpr int P_STAGES = 6;
constexpr uint32_t P_A_BYTES = 128 * BK * 2, P_B_BYTES = 128 * BK * 2, P_STAGE_BYTES = P_A_BYTES + P_B_BYTES;
constexpr uint32_t TMEM_COLS = 2 * P_BN;            // two accumulator buffers
constexpr size_t PAIR_SMEM = (size_t)P_STAGES * P_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
// instruction descriptor, kind::f16: D=f32, A=B=bf16, both K-major, N=256, M=256
constexpr uint32_t IDESC_BF16_PAIR = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P_BN >> 3) << 17) | ((uint32_t)(P_BM >> 4) << 24);

// Tile order: bands of P_RASTER_M tile rows, all tile columns of a band before the next band, tile rows
// fastest inside a band.  The pairs that run together then share few A and B panels, which the
// 126 MB L2 keeps between their reads.
constexpr int P_RASTER_M = 4;
__device__ __forceinline__ void pair_tile_coords(int64_t t, int64_t tiles_m, int64_t tiles_n, int64_t& tm, int64_t& tn)
{
    const int64_t per_band = (int64_t)P_RASTER_M * tiles_n;
    const int64_t band = t / per_band, r = t % per_band;
    const int64_t rows = min((int64_t)P_RASTER_M, tiles_m - band * P_RASTER_M);
    tm = band * P_RASTER_M + r % rows;
    tn = r / rows;
}

// The activation quantizer of the NEXT layer, run on the accumulators in the epilogue (Section 4.2:
// the post-processing unit quantizes each output block to FP4 or FP8 from the FP32 partial sums).
// codes4 == nullptr: off.  The output row of length N is the next layer's K.
struct QuantNext {
    const float* fisher;                 // [N] per-channel sensitivity of the next layer's input
    float s4, k6, s8, inv8, tau;
    int mode, ratio, free8;
    uint8_t* codes4; uint8_t* sf; uint32_t* mask; uint8_t* codes8;
    fgmp_packed_header* header;
    int64_t MW;                          // mask words per output row
};

struct GemmParams {
    void* Y; int64_t ldy; int y_is_bf16;
    int64_t M, N, K;
    const fgmp_packed_header* ha; const fgmp_packed_header* hw;
    int* status;
    QuantNext q;
    int cls_a, cls_w;       // 0, or the class of each operand's plane (1 = NVFP4 blocks, 2 = FP8 blocks): picks the tensor scales
    int accumulate;         // add to Y (fp32) instead of storing
};

// One row of 32 accumulator columns = two blocks of the next layer's activations: round to bf16 (what an
// unfused fgmp_linear would have stored), then the quantizer's steps in its order.  Returns the two mask bits.
__device__ __forceinline__ uint32_t quantize_chunk32(const GemmParams& p, int64_t row, int64_t col0, const uint32_t (&r)[32], float alpha)
{
    const QuantNext& q = p.q;
    uint32_t bits = 0;
    if (row >= p.M) return 0u;
#pragma unroll
    for (int hb = 0; hb < 2; ++hb) {
        const int64_t col = col0 + 16 * hb;
        if (col + 16 > p.N) break;
        const int64_t kb = col >> 4;
        float v[16], f[16], dq4[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __bfloat162float(__float2bfloat16_rn(__uint_as_float(r[16 * hb + i]) * alpha));
        const float4* fp = reinterpret_cast<const float4*>(q.fisher + col);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 t = __ldg(fp + i);
            f[4 * i] = t.x; f[4 * i + 1] = t.y; f[4 * i + 2] = t.z; f[4 * i + 3] = t.w;
        }
        uint32_t sc = block_dynamic_scale(v, q.k6);
        uint32_t c4[2], c8[4];
        block_nvfp4(v, sc, q.s4, c4, dq4);
        float score;
        if (q.mode == 0) {
            score = weighted_sq_sum(v, dq4, f);
        } else {
            float dq8[16];
            block_fp8(v, q.inv8, q.s8, c8, dq8);
            score = weighted_sq_sum(dq4, dq8, f);
        }
        if (score > q.tau) {
            if (q.mode == 0) {
                float dq8[16];
                block_fp8(v, q.inv8, q.s8, c8, dq8);
            }
            *reinterpret_cast<uint4*>(q.codes8 + row * p.N + kb * 16) = make_uint4(c8[0], c8[1], c8[2], c8[3]);
            c4[0] = 0; c4[1] = 0; sc = 0;
            bits |= 1u << hb;
        }
        *reinterpret_cast<uint2*>(q.codes4 + (row * p.N) / 2 + kb * 8) = make_uint2(c4[0], c4[1]);
        q.sf[fgmp_sf_offset(row, kb, p.N)] = (uint8_t)sc;
    }
    return bits;
}

// one row of 32 accumulator columns -> Y (scaled by the product of the tensor scales)
__device__ __forceinline__ void store_chunk32(const GemmParams& p, int64_t row, int64_t col0, const uint32_t (&r)[32], float alpha)
{
    if (row >= p.M) return;
    // Y and its row pitch 32-byte aligned: a lane writes whole 32-byte sectors
    const bool wide = !p.accumulate && ((uintptr_t)p.Y & 31) == 0 && ((p.ldy * (p.y_is_bf16 ? 2 : 4)) % 32) == 0 && col0 + 32 <= p.N;
    if (wide) {
        if (p.y_is_bf16) {
            __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.Y) + row * p.ldy + col0;
#pragma unroll
            for (int j = 0; j < 32; j += 16) {
                uint32_t o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[j + 2 * u]) * alpha, __uint_as_float(r[j + 2 * u + 1]) * alpha);
                    o[u] = *reinterpret_cast<uint32_t*>(&h);
                }
                store_256(y + j, o);
            }
        } else {
            float* y = reinterpret_cast<float*>(p.Y) + row * p.ldy + col0;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
                uint32_t o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) o[u] = __float_as_uint(__uint_as_float(r[j + u]) * alpha);
                store_256(y + j, o);
            }
        }
        return;
    }
    if (p.y_is_bf16) {
        __nv_bfloat16* y = reinterpret_cast<__nv_bfloat16*>(p.Y) + row * p.ldy + col0;
        if (col0 + 32 <= p.N && (p.ldy % 8) == 0) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
                uint32_t o[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[j + 2 * u]) * alpha,
                                                             __uint_as_float(r[j + 2 * u + 1]) * alpha);
                    o[u] = *reinterpret_cast<uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(y + j) = make_uint4(o[0], o[1], o[2], o[3]);
            }
        } else {
            for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) y[j] = __float2bfloat16_rn(__uint_as_float(r[j]) * alpha);
        }
    } else {
        float* y = reinterpret_cast<float*>(p.Y) + row * p.ldy + col0;
        if (p.accumulate) {
            for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) y[j] = __fadd_rn(y[j], __fmul_rn(__uint_as_float(r[j]), alpha));
        } else if (col0 + 32 <= p.N && (p.ldy % 4) == 0) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(y + j) = make_float4(__uint_as_float(r[j]) * alpha, __uint_as_float(r[j + 1]) * alpha,
                                                                __uint_as_float(r[j + 2]) * alpha, __uint_as_float(r[j + 3]) * alpha);
        } else {
            for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) y[j] = __uint_as_float(r[j]) * alpha;
        }
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmParams p)
{
    if (p.status[2]) return;                            // the all-NVFP4 GEMM has produced the result already (every thread of every CTA sees the same word)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // offset from the array: stays known as shared memory
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)P_STAGES * P_STAGE_BYTES);
    // bars[0..S) full (used in the leader), [S..2S) empty, [2S..2S+2) acc_full, [2S+2..2S+4) acc_empty (leader)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * P_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0 = leader
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + P_STAGES);
    const uint32_t accf0 = smem_u32(bars + 2 * P_STAGES), acce0 = smem_u32(bars + 2 * P_STAGES + 2);

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 8); }   // 4 epilogue warps x 2 CTAs
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync();                                     // the other CTA's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (p.q.codes4 && blockIdx.x == 0 && threadIdx.x == 0) {
        fgmp_packed_header* h = p.q.header;
        h->magic = FGMP_MAGIC; h->version = 7; h->rows = p.M; h->K = p.N; h->scale_fp4 = p.q.s4;
        h->fp8_log2_ratio = p.q.ratio; h->n_fp8 = (p.q.tau == INFINITY) ? 0 : -1; h->tau_eff = 0.f; h->kind = 0; h->capacity = 0;
        h->error = 0; h->scale_fp8 = p.q.s8; h->fp8_scale_free = p.q.free8;
    }
    const int64_t tiles_m = (p.M + P_BM - 1) / P_BM, tiles_n = (p.N + P_BN - 1) / P_BN;
    const int64_t num_tiles = tiles_m * tiles_n;
    const int64_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_kb = (int)(p.K / BK);

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            for (int64_t t = pair; t < num_tiles && ok; t += num_pairs) {
                int64_t tm, tn;
                pair_tile_coords(t, tiles_m, tiles_n, tm, tn);
                const int32_t m0 = (int32_t)(tm * P_BM + 128 * rank), n0 = (int32_t)(tn * P_BN + 128 * rank);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1))) break;
                    // the leader's barrier counts the bytes of both CTAs
                    if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * P_STAGE_BYTES);
                    const uint32_t fb = cluster_map(full0 + 8 * stage, 0);
                    const uint32_t sa = smem_u32(smem + (size_t)stage * P_STAGE_BYTES);
                    tma_load_2d_pair(sa, &tmA, kb * BK, m0, fb);
                    tma_load_2d_pair(sa + P_A_BYTES, &tmB, kb * BK, n0, fb);
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int64_t it = 0;
            for (int64_t t = pair; t < num_tiles && ok; t += num_pairs, ++it) {
                const int acc = (int)(it & 1); const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
                if (!(ok = mbar_wait(acce0 + 8 * acc, acc_phase ^ 1, abort_flag, p.status, 2))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * P_BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 3))) break;
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)stage * P_STAGE_BYTES);
                    const uint64_t adesc = smem_desc_sw128(sa), bdesc = smem_desc_sw128(sa + P_A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_f16_pair(d_tmem, adesc + (uint64_t)(k * UMMA_K * 2 / 16), bdesc + (uint64_t)(k * UMMA_K * 2 / 16),
                                      IDESC_BF16_PAIR, (kb | k) ? 1u : 0u);
                    umma_commit_pair(empty0 + 8 * stage, 3);          // the stage is free in both CTAs
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit_pair(accf0 + 8 * acc, 3);         // both epilogues may read their halves
            }
        }
    } else {
        const int q = warp & 3;                        // TMEM lane quadrant this warp may read
        const float alpha = __fmul_rn(p.cls_a == 2 ? p.ha->scale_fp8 : p.ha->scale_fp4, p.cls_w == 2 ? p.hw->scale_fp8 : p.hw->scale_fp4);
        bool ok = true;
        int64_t it = 0;
        for (int64_t t = pair; t < num_tiles && ok; t += num_pairs, ++it) {
            const int acc = (int)(it & 1); const uint32_t acc_phase = (uint32_t)((it >> 1) & 1);
            int64_t tm, tn;
            pair_tile_coords(t, tiles_m, tiles_n, tm, tn);
            const int64_t m0 = tm * P_BM + 128 * rank, n0 = tn * P_BN;
            if (!(ok = mbar_wait(accf0 + 8 * acc, acc_phase, abort_flag, p.status, 4))) break;
            tc_fence_after();
            const int64_t row = m0 + q * 32 + lane;
            uint32_t mbits = 0;                        // FP8 flags of this row's 16 output blocks in the tile
#pragma unroll 1
            for (int c = 0; c < P_BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * P_BN + c * 32), r);
                if (p.q.codes4) mbits |= quantize_chunk32(p, row, n0 + c * 32, r, alpha) << (2 * c);
                else store_chunk32(p, row, n0 + c * 32, r, alpha);
            }
            if (p.q.codes4 && row < p.M) {
                // a 256-column tile is half a mask word of the row
                uint16_t* mw = reinterpret_cast<uint16_t*>(p.q.mask + row * p.q.MW + (tn >> 1));
                mw[tn & 1] = (uint16_t)mbits;
                if ((tn & 1) == 0 && (tn + 1) * P_BN >= p.N) mw[1] = 0;      // no tile behind this one
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(cluster_map(acce0 + 8 * acc, 0));
        }
    }

    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync();                                     // neither CTA leaves while the other may still read its memory
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 row-major [rows, K] tensor, box = [box_rows, 64 elements], 128-byte swizzle
bool make_tmap_bf16(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int box_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t fgmp_ws_linear_quantize(int64_t M, int64_t N, int64_t K)
{
    return fgmp_ws_linear(M, N, K) + (fgmp_decode_supported(M, N, K) ? fgmp_align1k((size_t)M * N * 2) : 0);
}

size_t fgmp_ws_linear(int64_t M, int64_t N, int64_t K)
{
    if (fgmp_decode_supported(M, N, K)) return fgmp_ws_decode(M, N, K);
    return (size_t)FGMP_WS_CONTROL_BYTES + fgmp_align1k((size_t)M * K * 2) + fgmp_align1k((size_t)N * K * 2);
}

// CTA pairs that can be resident at once on this device (a pair needs two SMs of one cluster domain)
static fgmp_status resident_pairs(int* pairs)
{
    static std::mutex mu;
    static int pairs_of_device[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return FGMP_ERR_CUDA;
    std::lock_guard<std::mutex> lk(mu);
    if (!pairs_of_device[dev]) {
        if (cudaFuncSetAttribute(gemm_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PAIR_SMEM) != cudaSuccess)
            return FGMP_ERR_CUDA;
        cudaLaunchConfig_t qc = {};
        qc.gridDim = dim3((unsigned)(fgmp_sm_count() & ~1)); qc.blockDim = dim3(GEMM_THREADS); qc.dynamicSmemBytes = PAIR_SMEM;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_bf16_pair_kernel, &qc) != cudaSuccess || n < 1) return FGMP_ERR_CUDA;
        pairs_of_device[dev] = n;
    }
    *pairs = pairs_of_device[dev];
    return FGMP_OK;
}

// expand both operands and run the pair GEMM (M > 16 or a shape the weight-streaming kernel does not take)
static fgmp_status launch_prefill(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                                  int64_t M, int64_t N, int64_t K, void* workspace, const QuantNext& qn, cudaStream_t s)
{
    uint8_t* ws = (uint8_t*)workspace;
    int* status = reinterpret_cast<int*>(ws);
    uint8_t* planeA = ws + FGMP_WS_CONTROL_BYTES;       // the control area stays as the decode-sized calls need it
    uint8_t* planeW = planeA + fgmp_align1k((size_t)M * K * 2);

    int pairs_avail = 0;
    fgmp_status stp = resident_pairs(&pairs_avail);
    if (stp != FGMP_OK) return stp;
    CUtensorMap tmA, tmB;
    if (!make_tmap_bf16(&tmA, planeA, M, K, 128) || !make_tmap_bf16(&tmB, planeW, N, K, 128)) return FGMP_ERR_CUDA;

    if (cudaMemsetAsync(status, 0, 256, s) != cudaSuccess) return FGMP_ERR_CUDA;
    // Operands without any FP8 block go through the NVFP4 tensor-core kind straight from the packed form; whether
    // that is the case is written in the two headers, so the kernel looks itself and leaves word 2 of the status
    // area at 1 if it has done the work.  (The variant with the next layer's quantizer in the epilogue has the
    // general path only.)
    if (!qn.codes4) {
        const fgmp_status st4 = fgmp_launch_gemm_nvfp4(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, status, s);
        if (st4 != FGMP_OK) return st4;
    }
    const int sms = fgmp_sm_count();
    {
        const int64_t nb = M * (K / 16);
        const int g = (int)((nb + 255) / 256 < (int64_t)sms * 8 ? (nb + 255) / 256 : (int64_t)sms * 8);
        FGMP_LAUNCH(FGMP_K_EXPAND_A, s, expand_kernel<<<g, 256, 0, s>>>((const uint8_t*)packed_acts, M, K, reinterpret_cast<uint4*>(planeA), status, 0));
        const PackedLayout LW = fgmp_layout(N, K, 1, 0);
        FGMP_LAUNCH(FGMP_K_EXPAND_W, s, expand_w_kernel<<<(unsigned)LW.units, 128, 0, s>>>((const uint8_t*)packed_weights, N, K, reinterpret_cast<uint4*>(planeW), status, 0));
    }
    GemmParams p;
    p.Y = Y; p.ldy = ldy; p.y_is_bf16 = y_is_bf16; p.M = M; p.N = N; p.K = K;
    p.ha = reinterpret_cast<const fgmp_packed_header*>(packed_acts);
    p.hw = reinterpret_cast<const fgmp_packed_header*>(packed_weights);
    p.status = status;
    p.q = qn;
    p.cls_a = 0; p.cls_w = 0; p.accumulate = 0;
    const int64_t tiles = ((M + P_BM - 1) / P_BM) * ((N + P_BN - 1) / P_BN);
    const int pairs = (int)(tiles < pairs_avail ? tiles : pairs_avail);
    FGMP_LAUNCH(FGMP_K_GEMM_BF16, s, gemm_bf16_pair_kernel<<<2 * pairs, GEMM_THREADS, PAIR_SMEM, s>>>(tmA, tmB, p));
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_linear(const void* packed_acts, const void* packed_weights,
                                   void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                                   void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!packed_acts || !packed_weights || !Y || !workspace) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || N < 1 || K < 64 || (K % 64) != 0 || ldy < N) return FGMP_ERR_SHAPE;
    if (((uintptr_t)packed_acts & 1023) || ((uintptr_t)packed_weights & 1023) || ((uintptr_t)workspace & 1023) ||
        ((uintptr_t)Y & 15)) return FGMP_ERR_SHAPE;
    if (ws_bytes < fgmp_ws_linear(M, N, K)) return FGMP_ERR_WORKSPACE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (fgmp_decode_supported(M, N, K))
        return fgmp_linear_decode(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, workspace, false, s);
    QuantNext off{};
    return launch_prefill(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, workspace, off, s);
}

size_t fgmp_ws_linear_classes(int64_t M, int64_t N, int64_t K)
{
    return (size_t)FGMP_WS_CONTROL_BYTES + fgmp_align1k((size_t)M * K * 2) + fgmp_align1k((size_t)N * K * 2);
}

// One accumulation per class of block pair: FP4 x FP4, FP4 x FP8, FP8 x FP8, FP8 x FP4, each a pass of the pair
// GEMM over planes that hold the blocks of one format (over their own tensor scale) and zeros elsewhere; the
// epilogue multiplies by the two scales of the pass and adds to Y.
extern "C" fgmp_status fgmp_linear_classes(const void* packed_acts, const void* packed_weights,
                                           void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                                           void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!packed_acts || !packed_weights || !Y || !workspace || y_is_bf16) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || N < 1 || K < 64 || (K % 64) != 0 || ldy < N) return FGMP_ERR_SHAPE;
    if (((uintptr_t)packed_acts & 1023) || ((uintptr_t)packed_weights & 1023) || ((uintptr_t)workspace & 1023) ||
        ((uintptr_t)Y & 15)) return FGMP_ERR_SHAPE;
    if (ws_bytes < fgmp_ws_linear_classes(M, N, K)) return FGMP_ERR_WORKSPACE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint8_t* ws = (uint8_t*)workspace;
    int* status = reinterpret_cast<int*>(ws);
    uint8_t* planeA = ws + FGMP_WS_CONTROL_BYTES;
    uint8_t* planeW = planeA + fgmp_align1k((size_t)M * K * 2);
    int pairs_avail = 0;
    if ((st = resident_pairs(&pairs_avail)) != FGMP_OK) return st;
    CUtensorMap tmA, tmB;
    if (!make_tmap_bf16(&tmA, planeA, M, K, 128) || !make_tmap_bf16(&tmB, planeW, N, K, 128)) return FGMP_ERR_CUDA;
    if (cudaMemsetAsync(status, 0, 256, s) != cudaSuccess) return FGMP_ERR_CUDA;
    const int sms = fgmp_sm_count();
    const int64_t nb = M * (K / 16);
    const int ga = (int)((nb + 255) / 256 < (int64_t)sms * 8 ? (nb + 255) / 256 : (int64_t)sms * 8);
    const PackedLayout LW = fgmp_layout(N, K, 1, 0);
    GemmParams p;
    p.Y = Y; p.ldy = ldy; p.y_is_bf16 = 0; p.M = M; p.N = N; p.K = K;
    p.ha = reinterpret_cast<const fgmp_packed_header*>(packed_acts);
    p.hw = reinterpret_cast<const fgmp_packed_header*>(packed_weights);
    p.status = status;
    p.q = QuantNext{};
    const int64_t tiles = ((M + P_BM - 1) / P_BM) * ((N + P_BN - 1) / P_BN);
    const int pairs = (int)(tiles < pairs_avail ? tiles : pairs_avail);
    // (activation class, weight class) in an order that re-expands one operand per pass
    const int order[4][2] = {{1, 1}, {1, 2}, {2, 2}, {2, 1}};
    int have_a = 0, have_w = 0;
    for (int i = 0; i < 4; ++i) {
        const int ca = order[i][0], cw = order[i][1];
        if (ca != have_a) {
            FGMP_LAUNCH(FGMP_K_EXPAND_A, s, expand_kernel<<<ga, 256, 0, s>>>((const uint8_t*)packed_acts, M, K, reinterpret_cast<uint4*>(planeA), status, ca));
            have_a = ca;
        }
        if (cw != have_w) {
            FGMP_LAUNCH(FGMP_K_EXPAND_W, s, expand_w_kernel<<<(unsigned)LW.units, 128, 0, s>>>((const uint8_t*)packed_weights, N, K, reinterpret_cast<uint4*>(planeW), status, cw));
            have_w = cw;
        }
        p.cls_a = ca; p.cls_w = cw; p.accumulate = i > 0;
        FGMP_LAUNCH(FGMP_K_GEMM_BF16, s, gemm_bf16_pair_kernel<<<2 * pairs, GEMM_THREADS, PAIR_SMEM, s>>>(tmA, tmB, p));
    }
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_linear_quantize(const void* packed_acts, const void* packed_weights,
                                            int64_t M, int64_t N, int64_t K,
                                            const float* fisher_chan_next, fgmp_scales sc_next, fgmp_score_mode sm,
                                            float tau_next, void* packed_out, size_t packed_bytes,
                                            void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!packed_acts || !packed_weights || !fisher_chan_next || !packed_out || !workspace) return FGMP_ERR_INVALID_ARG;
    if ((int)sm < 0 || (int)sm > 1 || tau_next != tau_next) return FGMP_ERR_INVALID_ARG;
    if (!(sc_next.scale_fp4 > 0.f) || !isfinite(sc_next.scale_fp4)) return FGMP_ERR_INVALID_ARG;
    if (!fgmp_scales_valid(sc_next)) return FGMP_ERR_INVALID_ARG;
    // the output is a packed activation tensor [M, N]: N is the next layer's K
    if (M < 1 || N < 64 || (N % 64) != 0 || K < 64 || (K % 64) != 0) return FGMP_ERR_SHAPE;
    if (((uintptr_t)packed_acts & 1023) || ((uintptr_t)packed_weights & 1023) || ((uintptr_t)workspace & 1023) ||
        ((uintptr_t)packed_out & 1023) || ((uintptr_t)fisher_chan_next & 15)) return FGMP_ERR_SHAPE;
    if (ws_bytes < fgmp_ws_linear_quantize(M, N, K)) return FGMP_ERR_WORKSPACE;
    if (fgmp_decode_supported(M, N, K)) {
        // decode-sized batch: the weight-streaming kernel holds an output row per thread, not a token row, so the
        // two steps stay two launches; the bf16 outputs (at most 16 x N) pass through the end of the workspace
        uint8_t* ybf = (uint8_t*)workspace + fgmp_ws_linear(M, N, K);
        fgmp_status st2 = fgmp_linear(packed_acts, packed_weights, ybf, 1, N, M, N, K, workspace, fgmp_ws_linear(M, N, K), cuda_stream);
        if (st2 != FGMP_OK) return st2;
        return fgmp_quantize_activations(ybf, N, fisher_chan_next, M, N, sc_next, sm, tau_next, packed_out, packed_bytes,
                                         nullptr, 0, cuda_stream);
    }
    const PackedLayout L = fgmp_layout(M, N, 0, 0);
    if (packed_bytes < L.total) return FGMP_ERR_WORKSPACE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    uint8_t* blob = (uint8_t*)packed_out;
    QuantNext q{};
    q.fisher = fisher_chan_next;
    // the same scalars, computed the same way, as fgmp_quantize_activations uses
    q.s4 = sc_next.scale_fp4;
    q.k6 = 1.0f / (6.0f * sc_next.scale_fp4);
    q.s8 = fgmp_fp8_scale(sc_next); q.free8 = fgmp_fp8_free(sc_next) ? 1 : 0;
    q.inv8 = 1.0f / q.s8;
    q.tau = tau_next; q.mode = (int)sm; q.ratio = sc_next.fp8_log2_ratio;
    q.codes4 = blob + L.off_codes4; q.sf = blob + L.off_sf;
    q.mask = reinterpret_cast<uint32_t*>(blob + L.off_mask); q.codes8 = blob + L.off_codes8;
    q.header = reinterpret_cast<fgmp_packed_header*>(blob);
    q.MW = L.MW;
    return launch_prefill(packed_acts, packed_weights, nullptr, 0, N, M, N, K, workspace, q, (cudaStream_t)cuda_stream);
}

extern "C" fgmp_status fgmp_workspace_init(void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!workspace || ((uintptr_t)workspace & 1023)) return FGMP_ERR_INVALID_ARG;
    const size_t n = ws_bytes < (size_t)FGMP_WS_CONTROL_BYTES ? ws_bytes : (size_t)FGMP_WS_CONTROL_BYTES;
    if (n && cudaMemsetAsync(workspace, 0, n, (cudaStream_t)cuda_stream) != cudaSuccess) return FGMP_ERR_CUDA;
    return FGMP_OK;
}

extern "C" fgmp_status fgmp_check(const void* workspace, void* cuda_stream)
{
    if (!workspace) return FGMP_ERR_INVALID_ARG;
    int host[2] = {0, 0};
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return FGMP_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FGMP_ERR_CUDA;
    return host[0] == 0 ? FGMP_OK : (fgmp_status)host[0];
}

extern "C" size_t fgmp_workspace_bytes(int op, int64_t M, int64_t N, int64_t K)
{
    if (op == FGMP_OP_GLOBAL_TAU) return M >= 1 ? fgmp_ws_global_tau(M) : 0;
    if (K < 64 || (K % 64) != 0) return 0;
    switch (op) {
        case FGMP_OP_QUANTIZE_WEIGHTS: return N >= 1 ? fgmp_ws_quantize_weights(N, K) : 0;
        case FGMP_OP_QUANTIZE_ACTIVATIONS: return 0;
        case FGMP_OP_LINEAR: return (M >= 1 && N >= 1) ? fgmp_ws_linear(M, N, K) : 0;
        case FGMP_OP_CALIBRATE_TAU: return M >= 1 ? fgmp_ws_calibrate(M, K) : 0;
        case FGMP_OP_LINEAR_QUANTIZE: return (M >= 1 && N >= 1) ? fgmp_ws_linear_quantize(M, N, K) : 0;
        case FGMP_OP_LINEAR_FUSED: return (M >= 1 && N >= 1) ? fgmp_ws_linear_fused(M, N, K) : 0;
        case FGMP_OP_LINEAR_CLASSES: return (M >= 1 && N >= 1) ? fgmp_ws_linear_classes(M, N, K) : 0;
    }
    return 0;
}
