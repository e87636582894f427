// fgmp_linear for decode-sized batches (M <= 16 tokens): a weight-streaming kernel that
// reads the packed weights exactly once (Section 4.1 of the paper: the four block-pair
// products, FP32 accumulation).  All arithmetic runs on the tensor cores; the CUDA cores only
// move and convert the few blocks that need it.
//
// Decomposition (exact).  Call a block column "hot" when at least one token has an FP8 block
// there.  With W4z the NVFP4 weight codes (zero in FP8 blocks), A4z' the NVFP4 activation codes
// with every hot column zeroed, At the true activation values (fp16, either format) and T the
// fp16 tile that holds the FP8 weight blocks everywhere plus, in hot columns, the dequantized
// NVFP4 weight blocks (so T = the true weights there):
//     Y = A4z'.W4z^T    tcgen05.mma kind::mxf4nvf4, UE4M3 block scales in TMEM
//       + At.T^T        tcgen05.mma kind::f16 into the same FP32 accumulator
// In a cold column A4z'.W4z covers NVFP4 x NVFP4 and At.T covers every pair with an FP8 weight
// block; in a hot column At.T is the complete product.  T is mostly zero: per quarter of a unit
// (4 block columns) it is a 128 x 64 fp16 tile that scatter threads fill from the unit's record
// and clear again after use.
//
// Work is split stream-K style over (128-row tile, 256-element K chunk) units so that all SMs
// stream the same number of bytes; a unit is two bulk copies (its weight record, the activation
// record of its chunk).  Tiles shared by several CTAs are reduced in a fixed order by the CTA
// that arrives last; the accumulation order inside TMEM is the issue order: results are
// reproducible bit for bit.
//
// Warp roles (704 threads): warp 0 = producer, warp 1 = MMA issuer and TMEM owner,
// warps 2-5 = epilogue (one TMEM lane quadrant each), warps 6-21 = scatter (eight groups of two).
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <cuda_fp16.h>

namespace {

constexpr int DEC_THREADS = 704;
constexpr int SCAT_THREADS = 512, GRP_WARPS = 2, GRP_THREADS = 64;   // eight groups: (quarter of T, unit parity)
constexpr int TOK = 16;                         // MMA N (token rows, zero padded)
constexpr uint32_t FP8_CAP_BLOCKS = 320;        // FP8 blocks of a unit that fit a stage; more are read from global
constexpr uint32_t WREC_CAP = (REC_ROWID + FP8_CAP_BLOCKS + FP8_CAP_BLOCKS * 16 + 127) & ~127u;   // 23936
constexpr uint32_t STG_A = (WREC_CAP + 1023) & ~1023u;                                           // 24576
constexpr uint32_t DEC_STAGE_BYTES = STG_A + AREC_BYTES;                                         // 37888
constexpr int DEC_STAGES = 4;
constexpr uint32_t TQ_BYTES = 128 * 128;        // one quarter of T: 128 rows x 64 fp16, 128B-swizzled
constexpr int NACC = 4;                         // independent accumulators per tile: back-to-back MMAs into one
                                                // accumulator wait for each other, so the MMAs of a unit rotate over four
constexpr uint32_t ACC_COLS = NACC * TOK;       // columns of one accumulator buffer
constexpr uint32_t SF_COL0 = 2 * ACC_COLS;      // scale columns start behind the two accumulator buffers
constexpr uint32_t DEC_TMEM_COLS = 256;         // 2 x 64 accumulator columns + 4 stages x 32 scale columns
constexpr size_t DEC_SMEM = (size_t)DEC_STAGES * DEC_STAGE_BYTES + 4 * TQ_BYTES + 1024 /*alignment*/ + 512 /*barriers*/ + 8192 /*lists*/;
static_assert(DEC_STAGE_BYTES % 1024 == 0 && (STG_A + AREC_TRUE) % 1024 == 0, "swizzled tiles need 1 KiB alignment");

// kind::mxf4nvf4, E2M1 x E2M1, UE4M3 scales, K-major operands, M = 128, N = 16, dense K = 64
constexpr uint32_t IDESC_NVF4 = (1u << 7) | (1u << 10) | ((uint32_t)(TOK >> 3) << 17) | (0u << 23) | ((uint32_t)(128 >> 4) << 24);
// kind::f16, D = f32, A = B = fp16, K-major operands, M = 128, N = 16, K = 16
constexpr uint32_t IDESC_F16 = (1u << 4) | ((uint32_t)(TOK >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

// shared-memory matrix descriptors as (low word | start address >> 4, constant high word)
constexpr uint32_t SW128_LO = 1u << 16, SW128_HI = (1024u >> 4) | (1u << 14) | (2u << 29);   // 128B swizzle, 8-row groups 1 KiB apart
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}

struct DecParams {
    const uint8_t* wblob; const uint8_t* ablob;
    PackedLayout LW, LA;
    float* Y; void* Ybf; int64_t ldy; int y_is_bf16;
    int64_t M, N, K;
    int64_t total;            // tiles * chunks
    int64_t chunks;
    int* status; uint32_t* counters; float* partials; int maxseg;
};

struct StageMeta { uint32_t step, staged; };     // record start (128-byte steps), bytes of it in the stage

__device__ __forceinline__ int64_t cta_of_unit(int64_t i, int64_t G, int64_t total) { return ((i + 1) * G - 1) / total; }

__device__ __forceinline__ uint32_t byte_sum(uint32_t x) { return __dp4a(x, 0x01010101u, 0u); }

// 16 E4M3 codes -> 16 fp16 (two 16-byte halves), scaled by a power of two
__device__ __forceinline__ void e4m3x16_to_h16(const uint4& c, __half2 scale, uint4& lo, uint4& hi)
{
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t h0, h1;
        const uint16_t l = (uint16_t)w[i], h = (uint16_t)(w[i] >> 16);
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h0) : "h"(l));
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h1) : "h"(h));
        const __half2 x0 = __hmul2(*reinterpret_cast<__half2*>(&h0), scale), x1 = __hmul2(*reinterpret_cast<__half2*>(&h1), scale);
        o[2 * i] = *reinterpret_cast<const uint32_t*>(&x0); o[2 * i + 1] = *reinterpret_cast<const uint32_t*>(&x1);
    }
    lo = make_uint4(o[0], o[1], o[2], o[3]); hi = make_uint4(o[4], o[5], o[6], o[7]);
}

// 16 E2M1 codes (8 bytes) times an E4M3 microscale -> 16 fp16, exact
__device__ __forceinline__ void nvfp4x16_to_h16(const uint2& c, uint32_t scale_code, uint4& lo, uint4& hi)
{
    uint32_t sc2;
    const uint16_t s16 = (uint16_t)(scale_code | (scale_code << 8));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2) : "h"(s16));
    const __half2 sc = *reinterpret_cast<__half2*>(&sc2);
    const uint32_t w[2] = {c.x, c.y};
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t q;
        const uint32_t byte = (w[i >> 2] >> ((i & 3) * 8)) & 0xffu;
        asm("{\n\t.reg .b8 t;\n\tcvt.u8.u32 t, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, t;\n\t}" : "=r"(q) : "r"(byte));
        const __half2 x = __hmul2(*reinterpret_cast<__half2*>(&q), sc);
        o[i] = *reinterpret_cast<const uint32_t*>(&x);
    }
    lo = make_uint4(o[0], o[1], o[2], o[3]); hi = make_uint4(o[4], o[5], o[6], o[7]);
}

__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(DecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* tq = smem + (size_t)DEC_STAGES * DEC_STAGE_BYTES;                 // four quarter tiles of T
    uint64_t* bars = reinterpret_cast<uint64_t*>(tq + 4 * TQ_BYTES);
    // bars (S = stages): [0,S) full, [S,2S) empty, [2S,3S) a4 ready, then T quarter full [4], T quarter
    // done [2 unit parities][4] (a parity wait can only tell two consecutive phases apart, so each of
    // the two groups that share a quarter has a barrier of its own), scatter group sync [8],
    // acc_full[2], acc_empty[2]
    StageMeta* smeta = reinterpret_cast<StageMeta*>(bars + 3 * DEC_STAGES + 28);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smeta + DEC_STAGES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint32_t* qcnt = tmem_slot + 2;                                            // [4 quarters]
    uint16_t* qlist = reinterpret_cast<uint16_t*>(tq + 4 * TQ_BYTES + 512);     // [4 quarters][1024]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * DEC_STAGES, a4r0 = empty0 + 8 * DEC_STAGES;
    const uint32_t tfull0 = a4r0 + 8 * DEC_STAGES, tdone0 = tfull0 + 32, gbar0 = tdone0 + 64;
    const uint32_t accf0 = gbar0 + 64, acce0 = accf0 + 16;

    // this CTA's span of (tile, chunk) units
    const int64_t G = gridDim.x, C = p.chunks;
    const int64_t u_begin = ((int64_t)blockIdx.x * p.total) / G, u_end = ((int64_t)(blockIdx.x + 1) * p.total) / G;
    const uint32_t* uptr = reinterpret_cast<const uint32_t*>(p.wblob + p.LW.off_uptr);
    const uint8_t* recs = p.wblob + p.LW.off_rec;

    // the producer's first record offsets are on their way while the CTA sets itself up
    int64_t pf_base = u_begin;
    uint32_t pf = 0;
    if (warp == 0 && pf_base + lane <= p.total) pf = __ldg(uptr + pf_base + lane);

    if (threadIdx.x == 0) {
        for (int s = 0; s < DEC_STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1 + 8); mbar_init(a4r0 + 8 * s, 8);   // 8 scatter warps serve a unit
        }
        for (int b = 0; b < 4; ++b) {
            mbar_init(tfull0 + 8 * b, GRP_WARPS); mbar_init(tdone0 + 8 * b, 1); mbar_init(tdone0 + 32 + 8 * b, 1);
            mbar_init(gbar0 + 8 * b, GRP_WARPS); mbar_init(gbar0 + 32 + 8 * b, GRP_WARPS);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 128); }
        *abort_flag = 0;
        for (int i = 0; i < 4; ++i) qcnt[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), DEC_TMEM_COLS);
    if (warp >= 6) {                                   // T starts all zero
        uint4* z = reinterpret_cast<uint4*>(tq);
        for (int i = (warp - 6) * 32 + lane; i < (int)(4 * TQ_BYTES / 16); i += SCAT_THREADS) z[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ producer (whole warp; lane 0 issues)
        int stage = 0; uint32_t phase = 0;
        const uint8_t* arec = p.ablob + p.LA.off_arec;
        for (int64_t u = u_begin; u < u_end; ++u) {
            if (u + 1 - pf_base > 31) {                // next 32 record offsets
                pf_base = u;
                pf = (pf_base + lane <= p.total) ? __ldg(uptr + pf_base + lane) : 0u;
            }
            const uint32_t step0 = __shfl_sync(0xffffffffu, pf, (int)(u - pf_base));
            const uint32_t step1 = __shfl_sync(0xffffffffu, pf, (int)(u + 1 - pf_base));
            int ok = 1;
            if (lane == 0) {
                ok = mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1) ? 1 : 0;
                if (ok) {
                    const uint32_t bytes = (step1 - step0) * 128u;
                    const uint32_t staged = bytes < WREC_CAP ? bytes : WREC_CAP;
                    smeta[stage].step = step0; smeta[stage].staged = staged;
                    const uint32_t fb = full0 + 8 * stage;
                    const uint32_t sb = smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES);
                    mbar_expect_tx(fb, staged + AREC_BYTES);
                    bulk_load(sb, recs + (size_t)step0 * 128, staged, fb);
                    bulk_load(sb + STG_A, arec + (size_t)(u % C) * AREC_BYTES, AREC_BYTES, fb);
                }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) break;
            if (++stage == DEC_STAGES) { stage = 0; phase ^= 1; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop (its values stay warp-uniform, which keeps the descriptor
        // arithmetic cheap); lane 0 alone issues the tcgen05 instructions, so that every commit
        // tracks every MMA before it.
        const uint32_t smem0 = smem_u32(smem), tq0 = smem_u32(tq);
        int stage = 0; uint32_t phase = 0; bool ok = true;
        int seg = 0; uint32_t useq = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_end = min(u_end, (tile + 1) * C);
            const int acc = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            if (!(ok = mbar_wait(acce0 + 8 * acc, acc_phase ^ 1, abort_flag, p.status, 2))) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)acc * ACC_COLS;
            uint32_t accum = 0;
            for (; u < seg_end && ok; ++u, ++useq) {
                if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 3))) break;
                tc_fence_after();
                const uint32_t sb = smem0 + (uint32_t)stage * DEC_STAGE_BYTES;
                const uint32_t sf_t = tmem_base + SF_COL0 + (uint32_t)stage * 32;   // [0,16) weights, [16,32) tokens
                // the scatter warps have put the microscales into TMEM and zeroed the hot columns of the
                // activation codes
                if (!(ok = mbar_wait(a4r0 + 8 * stage, phase, abort_flag, p.status, 8))) break;
                tc_fence_after();
                const uint32_t w4_lo = ((sb + REC_W4) >> 4) | SW128_LO, a4_lo = ((sb + STG_A + AREC_A4) >> 4) | SW128_LO;
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        umma_nvf4(d_tmem + j * TOK, desc64(w4_lo + 2 * j, SW128_HI), desc64(a4_lo + 2 * j, SW128_HI), IDESC_NVF4,
                                  sf_t + 4 * j, sf_t + 16 + 4 * j, accum);
                }
                accum = 1;
                const uint32_t at_lo = ((sb + STG_A + AREC_TRUE) >> 4) | SW128_LO;
#pragma unroll
                for (int qq = 0; qq < 4; ++qq) {
                    if (!(ok = mbar_wait(tfull0 + 8 * qq, useq & 1u, abort_flag, p.status, 9))) break;
                    tc_fence_after();
                    const uint32_t t_lo = ((tq0 + qq * TQ_BYTES) >> 4) | SW128_LO;
                    if (lane == 0) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_f16(d_tmem + k * TOK, desc64(t_lo + 2 * k, SW128_HI), desc64(at_lo + qq * 128 + 2 * k, SW128_HI), IDESC_F16, 1u);
                        umma_commit(tdone0 + 32 * (useq & 1u) + 8 * qq);
                    }
                }
                if (!ok) break;
                if (lane == 0) umma_commit(empty0 + 8 * stage);
                __syncwarp();
                if (++stage == DEC_STAGES) { stage = 0; phase ^= 1; }
            }
            if (ok && lane == 0) umma_commit(accf0 + 8 * acc);
            __syncwarp();
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------ epilogue: TMEM lane quadrant warp % 4
        const int q = warp & 3;
        const fgmp_packed_header* ha = reinterpret_cast<const fgmp_packed_header*>(p.ablob);
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const float alpha = __fmul_rn(ha->scale_fp4, hw->scale_fp4);
        bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_begin = u, seg_end = min(u_end, (tile + 1) * C);
            u = seg_end;
            const int accb = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            if (!(ok = mbar_wait(accf0 + 8 * accb, acc_phase, abort_flag, p.status, 4))) break;
            tc_fence_after();
            float v[16];
            {
                // the four partial accumulators of the tile, added in a fixed order
                uint32_t r0[16], r1[16], r2[16], r3[16];
                const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)accb * ACC_COLS;
                tmem_ld16(t0, r0); tmem_ld16(t0 + TOK, r1); tmem_ld16(t0 + 2 * TOK, r2); tmem_ld16(t0 + 3 * TOK, r3);
                tc_fence_before();
                mbar_arrive(acce0 + 8 * accb);
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    v[j] = ((__uint_as_float(r0[j]) + __uint_as_float(r1[j])) + __uint_as_float(r2[j])) + __uint_as_float(r3[j]);
            }
            const int row = 32 * q + lane;
            const int64_t n = tile * 128 + row;
            const bool whole = (seg_begin == tile * C) && (seg_end == (tile + 1) * C);
            bool write_out = whole;
            if (!whole) {
                // partial tile: publish, and let the warp that arrives last add everything up
                const int64_t c_first = cta_of_unit(tile * C, G, p.total);
                const int64_t c_last = cta_of_unit((tile + 1) * C - 1, G, p.total);
                const int nseg = (int)(c_last - c_first + 1);
                const int slot = (int)(blockIdx.x - c_first);
                float* dst = p.partials + (((size_t)tile * p.maxseg + slot) * 128 + row) * 16;
#pragma unroll
                for (int j = 0; j < 16; j += 4) __stcg(reinterpret_cast<float4*>(dst + j), make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]));
                __threadfence();
                __syncwarp();
                uint32_t old = 0;
                if (lane == 0) old = atomicAdd(p.counters + tile * 8 + q, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == (uint32_t)(nseg - 1)) {
                    __threadfence();
                    // all partials first (independent loads), then one sum in slot order
                    float4 x[4][4];
#pragma unroll
                    for (int sgi = 0; sgi < 4; ++sgi) {
                        const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16;
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            x[sgi][j] = sgi < nseg ? __ldcg(reinterpret_cast<const float4*>(src) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
#pragma unroll
                    for (int sgi = 0; sgi < 4; ++sgi) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            v[4 * j] += x[sgi][j].x; v[4 * j + 1] += x[sgi][j].y; v[4 * j + 2] += x[sgi][j].z; v[4 * j + 3] += x[sgi][j].w;
                        }
                    }
                    for (int sgi = 4; sgi < nseg; ++sgi) {       // more than four contributors: rare, serial
                        const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16;
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            const float4 y4 = __ldcg(reinterpret_cast<const float4*>(src + j));
                            v[j] += y4.x; v[j + 1] += y4.y; v[j + 2] += y4.z; v[j + 3] += y4.w;
                        }
                    }
                    write_out = true;
                }
            }
            if (write_out && n < p.N) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < p.M) {
                        if (p.y_is_bf16) reinterpret_cast<__nv_bfloat16*>(p.Ybf)[(int64_t)j * p.ldy + n] = __float2bfloat16_rn(v[j] * alpha);
                        else p.Y[(int64_t)j * p.ldy + n] = v[j] * alpha;
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ scatter: fill and clear T
        // Eight groups of two warps: group (q, h) owns quarter q of T for the units of parity h, so a
        // group has two unit times per unit and the two groups of a quarter take turns on its tile.
        // Per unit a group zeroes the hot columns of its quarter in the activation codes, (four of the
        // warps) loads the microscales into TMEM, converts its blocks, and then, once the previous
        // unit's MMAs on the quarter are done, clears what that unit left there and stores its own.
        const int sw = warp - 6;                       // 0..15
        const int half = sw >> 3, qq = (sw >> 1) & 3;  // unit parity served, quarter owned
        const int grp = sw >> 1;                       // 0..7
        const int gtid = (sw & 1) * 32 + lane;         // 0..63 inside the group
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const __half2 rw2 = __float2half2_rn(__int_as_float((127 + hw->fp8_log2_ratio) << 23));
        uint8_t* tile = tq + qq * TQ_BYTES;
        uint16_t* list = qlist + qq * 1024;            // T offsets written for the last unit in this quarter (0xffff = none)

        bool ok = true;
        uint32_t gphase = 0;
        for (int64_t useq = half; u_begin + useq < u_end && ok; useq += 2) {
            const int stage = (int)(useq & 3);
            const uint32_t phase = (uint32_t)(useq >> 2) & 1u;
            uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
            uint8_t* sa = sb + STG_A;
            if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 5))) break;
            const uint32_t staged = smeta[stage].staged;
            const uint8_t* rec_g = recs + (size_t)smeta[stage].step * 128;

            // hot columns: some token has an FP8 block there; their activation codes leave the NVFP4 product
            const uint32_t mword = lane < 16 ? *reinterpret_cast<const uint16_t*>(sa + AREC_MASK + lane * 2) : 0u;
            const uint32_t hot = __reduce_or_sync(0xffffffffu, mword);
            {
                const uint32_t col = 4u * qq + ((uint32_t)gtid >> 4), tok = (uint32_t)gtid & 15u;
                if ((hot >> col) & 1u) *reinterpret_cast<uint2*>(sa + AREC_A4 + fgmp_rec_w4_offset(tok, col)) = make_uint2(0, 0);
            }
            fence_proxy_async();
            if ((sw & 7) < 4) {
                // Microscales of the stage into TMEM, one warp per lane quadrant (warp % 4): lane i holds,
                // for MMA step j, the four scale bytes of rows i, 32+i, 64+i, 96+i in columns 4j..4j+3,
                // which is 16 bytes of scale tile j; the token scales follow in columns 16..31.
                uint32_t r[16];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 x = *reinterpret_cast<const uint4*>(sb + REC_SF + 512 * j + lane * 16);
                    r[4 * j] = x.x; r[4 * j + 1] = x.y; r[4 * j + 2] = x.z; r[4 * j + 3] = x.w;
                }
                const uint32_t sf_t = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + SF_COL0 + (uint32_t)stage * 32;
                tmem_st16(sf_t, r);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 x = *reinterpret_cast<const uint4*>(sa + AREC_SF + 512 * j + lane * 16);
                    r[4 * j] = x.x; r[4 * j + 1] = x.y; r[4 * j + 2] = x.z; r[4 * j + 3] = x.w;
                }
                tmem_st16(sf_t + 16, r);
                tmem_wait_st();
                tc_fence_before();
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(a4r0 + 8 * stage);

            const uint4 kc = *reinterpret_cast<const uint4*>(sb + REC_KBCNT);
            const uint32_t ks0 = byte_sum(kc.x), ks1 = byte_sum(kc.y), ks2 = byte_sum(kc.z), ks3 = byte_sum(kc.w);
            const uint32_t off8 = fgmp_rec_fp8_offset(ks0 + ks1 + ks2 + ks3);
            const uint32_t kword = qq == 0 ? kc.x : (qq == 1 ? kc.y : (qq == 2 ? kc.z : kc.w));
            const uint32_t n8 = qq == 0 ? ks0 : (qq == 1 ? ks1 : (qq == 2 ? ks2 : ks3));
            const uint32_t qstart = (qq > 0 ? ks0 : 0u) + (qq > 1 ? ks1 : 0u) + (qq > 2 ? ks2 : 0u);
            const uint32_t c0 = kword & 0xffu, c1 = (kword >> 8) & 0xffu, c2 = (kword >> 16) & 0xffu;
            const uint32_t hotq = (hot >> (4 * qq)) & 15u;
            const uint32_t nhot = __popc(hotq);

            // One FP8 block of the quarter (list entries qstart .. qstart + n8, ordered by (column, row)):
            // where it goes in T and its 16 values as fp16.
            auto fp8_item = [&](uint32_t it, uint32_t& pos, uint4& lo, uint4& hi) {
                const uint32_t e = qstart + it;
                const uint32_t o = off8 + e * 16;
                const uint4 raw = o + 16 <= staged ? *reinterpret_cast<const uint4*>(sb + o) : __ldg(reinterpret_cast<const uint4*>(rec_g + o));
                const uint32_t r = REC_ROWID + e < staged ? sb[REC_ROWID + e] : __ldg(rec_g + REC_ROWID + e);
                const uint32_t jq = (it >= c0) + (it >= c0 + c1) + (it >= c0 + c1 + c2);
                pos = fgmp_h16_tile_offset(r, jq, 0);
                e4m3x16_to_h16(raw, rw2, lo, hi);
            };
            // The NVFP4 block of a row in hot column jq of the quarter; pos = 0xffff when its microscale
            // is 0 (the block is FP8 or all zero) and nothing is to be written.
            auto hot_item = [&](uint32_t row, uint32_t jq, uint32_t& pos, uint4& lo, uint4& hi) {
                const uint32_t j = 4u * qq + jq;
                const uint32_t sc = sb[REC_SF + fgmp_rec_sf_offset(row, j)];
                pos = 0xffffu;
                if (sc != 0) {
                    pos = fgmp_h16_tile_offset(row, jq, 0);
                    nvfp4x16_to_h16(*reinterpret_cast<const uint2*>(sb + REC_W4 + fgmp_rec_w4_offset(row, j)), sc, lo, hi);
                }
            };
            auto put = [&](uint32_t slot, uint32_t pos, const uint4& lo, const uint4& hi) {
                list[slot] = (uint16_t)pos;
                if (pos != 0xffffu) {
                    *reinterpret_cast<uint4*>(tile + pos) = lo;
                    *reinterpret_cast<uint4*>(tile + (pos ^ 16u)) = hi;
                }
            };

            // converted ahead of the wait below: this thread's first FP8 block and its two rows of the first hot column
            uint32_t posA = 0xffffu, posB = 0xffffu, posC = 0xffffu;
            uint4 loA = make_uint4(0, 0, 0, 0), hiA = loA, loB = loA, hiB = loA, loC = loA, hiC = loA;
            if ((uint32_t)gtid < n8) fp8_item((uint32_t)gtid, posA, loA, hiA);
            const uint32_t jq_first = hotq ? (uint32_t)__ffs(hotq) - 1u : 0u;
            if (hotq) {
                hot_item((uint32_t)gtid, jq_first, posB, loB, hiB);
                hot_item((uint32_t)gtid + 64u, jq_first, posC, loC, hiC);
            }

            // the previous unit's MMAs on this quarter are done: clear what was written for it
            if (useq > 0) {
                if (!(ok = mbar_wait(tdone0 + 32 * (uint32_t)((useq - 1) & 1) + 8 * qq, (uint32_t)((useq - 1) >> 1) & 1u,
                                     abort_flag, p.status, 10))) break;
                const uint32_t n_old = qcnt[qq];
                for (uint32_t i = gtid; i < n_old; i += GRP_THREADS) {
                    const uint32_t o = list[i];
                    if (o != 0xffffu) {
                        *reinterpret_cast<uint4*>(tile + o) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4*>(tile + (o ^ 16u)) = make_uint4(0, 0, 0, 0);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(gbar0 + 8 * grp);          // the whole group has cleared its share
            if (!(ok = mbar_wait(gbar0 + 8 * grp, gphase, abort_flag, p.status, 11))) break;
            gphase ^= 1u;
            if (gtid == 0) qcnt[qq] = n8 + nhot * 128u;

            // list slots: [0, n8) the FP8 blocks, then 128 per hot column in column order
            if ((uint32_t)gtid < n8) put((uint32_t)gtid, posA, loA, hiA);
            for (uint32_t it = gtid + GRP_THREADS; it < n8; it += GRP_THREADS) {
                uint32_t pos; uint4 lo, hi;
                fp8_item(it, pos, lo, hi);
                put(it, pos, lo, hi);
            }
            if (hotq) {
                put(n8 + (uint32_t)gtid, posB, loB, hiB);
                put(n8 + (uint32_t)gtid + 64u, posC, loC, hiC);
                uint32_t rest = hotq & (hotq - 1u), slot = n8 + 128u + (uint32_t)gtid;
                while (rest) {
                    const uint32_t jq = (uint32_t)__ffs(rest) - 1u;
                    rest &= rest - 1u;
#pragma unroll
                    for (uint32_t rr = 0; rr < 2; ++rr) {
                        uint32_t pos; uint4 lo = make_uint4(0, 0, 0, 0), hi = lo;
                        hot_item((uint32_t)gtid + 64u * rr, jq, pos, lo, hi);
                        put(slot + 64u * rr, pos, lo, hi);
                    }
                    slot += 128u;
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) { mbar_arrive(tfull0 + 8 * qq); mbar_arrive(empty0 + 8 * stage); }
        }
    }

    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, DEC_TMEM_COLS);
    }
}

struct DecPlan { int64_t tiles, chunks, total; int grid; int maxseg; };

DecPlan decode_plan(int64_t N, int64_t K)
{
    DecPlan d;
    d.tiles = (N + 127) / 128; d.chunks = K / 256; d.total = d.tiles * d.chunks;
    const int sms = fgmp_sm_count();
    d.grid = (int)(d.total < sms ? d.total : sms);
    // a tile of `chunks` units meets at most this many CTA spans of >= floor(total/grid) units
    const int64_t span = d.total / d.grid;
    d.maxseg = (int)((d.chunks + span - 1) / span + 1);
    return d;
}

}  // namespace

bool fgmp_decode_supported(int64_t M, int64_t N, int64_t K)
{
    return M >= 1 && M <= 16 && N >= 1 && K >= 256 && (K % 256) == 0;
}

size_t fgmp_ws_decode(int64_t M, int64_t N, int64_t K)
{
    if (!fgmp_decode_supported(M, N, K)) return 0;
    const DecPlan d = decode_plan(N, K);
    return 1024 + fgmp_align1k((size_t)d.tiles * 32) + (size_t)d.tiles * d.maxseg * 128 * 16 * 4;
}

fgmp_status fgmp_linear_decode(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                               int64_t M, int64_t N, int64_t K, void* workspace, cudaStream_t s)
{
    const DecPlan d = decode_plan(N, K);
    uint8_t* ws = (uint8_t*)workspace;
    DecParams p;
    p.wblob = (const uint8_t*)packed_weights; p.ablob = (const uint8_t*)packed_acts;
    p.LW = fgmp_layout(N, K, 1, 0); p.LA = fgmp_layout(M, K, 0, 0);
    p.Y = (float*)Y; p.Ybf = Y; p.ldy = ldy; p.y_is_bf16 = y_is_bf16;
    p.M = M; p.N = N; p.K = K; p.total = d.total; p.chunks = d.chunks;
    p.status = reinterpret_cast<int*>(ws);
    p.counters = reinterpret_cast<uint32_t*>(ws + 1024);
    p.partials = reinterpret_cast<float*>(ws + 1024 + fgmp_align1k((size_t)d.tiles * 32));
    p.maxseg = d.maxseg;

    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess)
            return FGMP_ERR_CUDA;
        attr_set[dev] = true;
    }
    if (cudaMemsetAsync(ws, 0, 1024 + (size_t)d.tiles * 32, s) != cudaSuccess) return FGMP_ERR_CUDA;
    FGMP_LAUNCH(FGMP_K_DECODE, s, decode_kernel<<<d.grid, DEC_THREADS, DEC_SMEM, s>>>(p));
    return fgmp_launch_status();
}

// ------------------------------------------------------------------ allocation-free variant
// Scratch of fgmp_linear_static: one array per GPU that loads the library, held until exit.
static __device__ __align__(256) unsigned char g_static_scratch[FGMP_STATIC_SCRATCH_BYTES];

extern "C" fgmp_status fgmp_linear_static(const void* packed_acts, const void* packed_weights,
                                          void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                                          int32_t* status_out, void* cuda_stream)
{
    if (!packed_acts || !packed_weights || !Y) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || N < 1 || K < 64 || (K % 64) != 0 || ldy < N) return FGMP_ERR_SHAPE;
    if (((uintptr_t)packed_acts & 1023) || ((uintptr_t)packed_weights & 1023) || ((uintptr_t)Y & 15) ||
        ((uintptr_t)status_out & 3)) return FGMP_ERR_SHAPE;
    if (!fgmp_decode_supported(M, N, K)) return FGMP_ERR_SHAPE;
    if (fgmp_ws_decode(M, N, K) > (size_t)FGMP_STATIC_SCRATCH_BYTES) return FGMP_ERR_WORKSPACE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;

    // The array's name is only a host-side handle; the kernel needs its device address, which
    // differs per GPU.  Looked up once per device, with that device current.
    static void* scratch_of_device[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FGMP_ERR_CUDA;
    if (!scratch_of_device[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return FGMP_ERR_CUDA;
        scratch_of_device[dev] = ptr;
    }
    void* scratch = scratch_of_device[dev];
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // fgmp_linear_decode zeroes the status word and the tile counters at the start of the
    // scratch; the partial sums behind them are always written before they are read.
    st = fgmp_linear_decode(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, scratch, s);
    if (st != FGMP_OK) return st;
    if (status_out && cudaMemcpyAsync(status_out, scratch, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return FGMP_ERR_CUDA;
    return FGMP_OK;
}
