// fgmp_linear for decode-sized batches (M <= 16 tokens): a weight-streaming kernel that
// reads the packed weights exactly once (Section 4.1 of the paper: the four block-pair
// products, FP32 accumulation).
//
// Decomposition (exact).  With A4z / W4z the NVFP4 planes (zero in FP8 blocks), W8 the FP8
// blocks of the weights and At the true activation values (fp16 copy, either format):
//     Y = A4z.W4z^T            (1) tcgen05.mma kind::mxf4nvf4, UE4M3 block scales in TMEM,
//                                  weights are the 128-row MMA operand, the 16 tokens are N
//       + At.W8^T              (2) the FP8 weight blocks, which a record keeps grouped by block
//                                  column: sixteen blocks that meet the same 16 activation
//                                  elements form the M side of mma.sync m16n8k16; results are
//                                  added to their rows in a tile private to the warp
//       + At[FP8 blocks].W4z^T (3) only block columns in which some token is FP8: the NVFP4
//                                  weights of the stage are dequantized for mma.sync
// Work is split stream-K style over (128-row tile, 256-element K chunk) units so that all
// SMs stream the same number of bytes; a unit is two bulk copies (its weight record, the
// activation record of its chunk).  Tiles shared by several CTAs are reduced in a fixed order
// by the CTA that arrives last.  Every sum is taken in a fixed order: results are
// reproducible bit for bit.
//
// Warp roles (320 threads): warp 0 = producer, warp 1 = MMA issuer and TMEM owner,
// warps 2-9 = corrections (2) and (3), then epilogue.
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <cuda_fp16.h>

namespace {

constexpr int DEC_THREADS = 320;
constexpr int DEC_CORR_WARPS = 8;
constexpr int TOK = 16;                         // MMA N (token rows, zero padded)
constexpr uint32_t FP8_CAP_BLOCKS = 320;        // FP8 blocks of a unit that fit a stage; more are read from global
constexpr uint32_t WREC_CAP = (REC_ROWID + FP8_CAP_BLOCKS + FP8_CAP_BLOCKS * 16 + 127) & ~127u;   // 23936
constexpr uint32_t STG_A = (WREC_CAP + 1023) & ~1023u;                                           // 24576
constexpr uint32_t DEC_STAGE_BYTES = (STG_A + AREC_BYTES + 1023) & ~1023u;                       // 37888
constexpr int DEC_STAGES = 4;
constexpr uint32_t PRIV_FLOATS = 128 * TOK;     // one [row][token] tile per correction warp
constexpr uint32_t DEC_TMEM_COLS = 256;         // 2 x 16 accumulator columns + 4 stages x 32 scale columns
constexpr size_t DEC_SMEM = (size_t)DEC_STAGES * DEC_STAGE_BYTES + DEC_CORR_WARPS * PRIV_FLOATS * 4 + 1024 + 512;

// kind::mxf4nvf4, E2M1 x E2M1, UE4M3 scales, K-major operands, M = 128, N = 16, dense K = 64
constexpr uint32_t IDESC_NVF4 = (1u << 7) | (1u << 10) | ((uint32_t)(TOK >> 3) << 17) | (0u << 23) | ((uint32_t)(128 >> 4) << 24);

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

// two E4M3 pairs (4 bytes) -> two fp16 pairs, scaled by a power of two
__device__ __forceinline__ void e4m3x4_to_h2x2(uint32_t raw, __half2 scale, uint32_t& lo, uint32_t& hi)
{
    uint32_t h0, h1;
    const uint16_t l = (uint16_t)raw, h = (uint16_t)(raw >> 16);
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h0) : "h"(l));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h1) : "h"(h));
    const __half2 x0 = __hmul2(*reinterpret_cast<__half2*>(&h0), scale), x1 = __hmul2(*reinterpret_cast<__half2*>(&h1), scale);
    lo = *reinterpret_cast<const uint32_t*>(&x0); hi = *reinterpret_cast<const uint32_t*>(&x1);
}

__device__ __forceinline__ void add2(float* p, float a, float b)
{
    float2 v = *reinterpret_cast<float2*>(p);
    v.x += a; v.y += b;
    *reinterpret_cast<float2*>(p) = v;
}

__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(DecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float* priv = reinterpret_cast<float*>(smem + (size_t)DEC_STAGES * DEC_STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(priv + DEC_CORR_WARPS * PRIV_FLOATS);
    // bars: [0,S) full, [S,2S) empty, [2S,2S+2) acc_full, [2S+2,2S+4) acc_empty, [2S+4,2S+6) segment syncs
    StageMeta* smeta = reinterpret_cast<StageMeta*>(bars + 2 * DEC_STAGES + 6);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smeta + DEC_STAGES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + DEC_STAGES);
    const uint32_t accf0 = smem_u32(bars + 2 * DEC_STAGES), acce0 = smem_u32(bars + 2 * DEC_STAGES + 2);
    const uint32_t seg0 = smem_u32(bars + 2 * DEC_STAGES + 4);

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
        for (int s = 0; s < DEC_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1 + DEC_CORR_WARPS); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 32 * DEC_CORR_WARPS);
            mbar_init(seg0 + 8 * b, 32 * DEC_CORR_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), DEC_TMEM_COLS);
    if (warp >= 2) {                                   // the private tiles start at zero
        float4* z = reinterpret_cast<float4*>(priv + (warp - 2) * PRIV_FLOATS);
#pragma unroll
        for (int i = 0; i < (int)PRIV_FLOATS / 128; ++i) z[i * 32 + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
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
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool ok = true;
            int seg = 0;
            for (int64_t u = u_begin; u < u_end && ok; ++seg) {
                const int64_t tile = u / C;
                const int64_t seg_end = min(u_end, (tile + 1) * C);
                const int acc = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
                if (!(ok = mbar_wait(acce0 + 8 * acc, acc_phase ^ 1, abort_flag, p.status, 2))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TOK);
                bool first = true;
                for (; u < seg_end; ++u) {
                    if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 3))) break;
                    tc_fence_after();
                    const uint32_t sb = smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES);
                    const uint32_t sf_t = tmem_base + 32 + (uint32_t)stage * 32;   // [0,16) weights, [16,32) tokens
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        tmem_cp_sf(sf_t + 4 * j, smem_desc_sf(sb + REC_SF + 512 * j));
                        tmem_cp_sf(sf_t + 16 + 4 * j, smem_desc_sf(sb + STG_A + AREC_SF + 512 * j));
                    }
                    const uint64_t adesc = smem_desc_sw128(sb + REC_W4), bdesc = smem_desc_sw128(sb + STG_A + AREC_A4);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        umma_nvf4(d_tmem, adesc + 2 * j, bdesc + 2 * j, IDESC_NVF4, sf_t + 4 * j, sf_t + 16 + 4 * j,
                                  (first && j == 0) ? 0u : 1u);
                    }
                    first = false;
                    umma_commit(empty0 + 8 * stage);
                    if (++stage == DEC_STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit(accf0 + 8 * acc);
            }
        }
    } else {
        // ------------------------------------------------------------ corrections + epilogue
        // A warp may read TMEM lanes [32q, 32q+32), q = warp % 4; two warps share a quadrant and
        // each owns 16 of its rows for correction (3) and for the epilogue.
        const int cw = warp - 2;                       // 0..7
        const int q = warp & 3, h = cw >> 2;
        const int rowbase = 32 * q + 16 * h;           // first owned row inside the tile
        const int slice = 2 * q + h;                   // 0..7
        const int g = lane >> 2, t = lane & 3;
        const fgmp_packed_header* ha = reinterpret_cast<const fgmp_packed_header*>(p.ablob);
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const float alpha = __fmul_rn(ha->scale_fp4, hw->scale_fp4);
        const __half2 rw2 = __float2half2_rn(__int_as_float((127 + hw->fp8_log2_ratio) << 23));
        float* mypriv = priv + cw * PRIV_FLOATS;

        int stage = 0; uint32_t phase = 0; bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_begin = u, seg_end = min(u_end, (tile + 1) * C);
            float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};

            for (; u < seg_end; ++u) {
                if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 5))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint8_t* sa = sb + STG_A;
                const uint32_t staged = smeta[stage].staged;
                const uint8_t* rec_g = recs + (size_t)smeta[stage].step * 128;

                // (2) FP8 weight blocks of block columns cw and cw + 8
                const uint4 kc = *reinterpret_cast<const uint4*>(sb + REC_KBCNT);
                const uint32_t ks0 = byte_sum(kc.x), ks1 = byte_sum(kc.y), ks2 = byte_sum(kc.z);
                const uint32_t off8 = fgmp_rec_fp8_offset(ks0 + ks1 + ks2 + byte_sum(kc.w));
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int kb = cw + 8 * hh, wi = kb >> 2, sh8 = (kb & 3) * 8;
                    const uint32_t word = wi == 0 ? kc.x : (wi == 1 ? kc.y : (wi == 2 ? kc.z : kc.w));
                    const uint32_t start = (wi > 0 ? ks0 : 0u) + (wi > 1 ? ks1 : 0u) + (wi > 2 ? ks2 : 0u)
                                         + byte_sum(word & ((1u << sh8) - 1u));
                    const uint32_t end = start + ((word >> sh8) & 0xffu);
                    if (start == end) continue;
                    // B fragments: true activation values of tokens g and g + 8, elements 4t..4t+3 of the column
                    const uint2 bt0 = *reinterpret_cast<const uint2*>(sa + AREC_TRUE + kb * 512 + g * 32 + t * 8);
                    const uint2 bt1 = *reinterpret_cast<const uint2*>(sa + AREC_TRUE + kb * 512 + (g + 8) * 32 + t * 8);
                    for (uint32_t e = start; e < end; e += 16) {
                        // A fragments: FP8 blocks e + g and e + g + 8, the same four elements
                        const uint32_t iA = e + g, iB = iA + 8;
                        uint32_t rawA = 0, rawB = 0, rowA = 0, rowB = 0;
                        if (iA < end) {
                            const uint32_t o = off8 + iA * 16 + t * 4;
                            rawA = o + 4 <= staged ? *reinterpret_cast<const uint32_t*>(sb + o) : __ldg(reinterpret_cast<const uint32_t*>(rec_g + o));
                            rowA = REC_ROWID + iA < staged ? sb[REC_ROWID + iA] : __ldg(rec_g + REC_ROWID + iA);
                        }
                        if (iB < end) {
                            const uint32_t o = off8 + iB * 16 + t * 4;
                            rawB = o + 4 <= staged ? *reinterpret_cast<const uint32_t*>(sb + o) : __ldg(reinterpret_cast<const uint32_t*>(rec_g + o));
                            rowB = REC_ROWID + iB < staged ? sb[REC_ROWID + iB] : __ldg(rec_g + REC_ROWID + iB);
                        }
                        uint32_t a0, a1, a2, a3;
                        e4m3x4_to_h2x2(rawA, rw2, a0, a2);
                        e4m3x4_to_h2x2(rawB, rw2, a1, a3);
                        float c[4] = {0.f, 0.f, 0.f, 0.f}, d[4] = {0.f, 0.f, 0.f, 0.f};
                        mma_f16_16816(c, a0, a1, a2, a3, bt0.x, bt0.y);     // tokens 2t, 2t+1
                        mma_f16_16816(d, a0, a1, a2, a3, bt1.x, bt1.y);     // tokens 8+2t, 9+2t
                        // c[0..1] / d[0..1]: block iA, c[2..3] / d[2..3]: block iB.  Within one column every
                        // block has its own row, so no two lanes touch the same address here.
                        if (iA < end) {
                            add2(mypriv + rowA * TOK + 2 * t, c[0], c[1]);
                            add2(mypriv + rowA * TOK + 8 + 2 * t, d[0], d[1]);
                        }
                        if (iB < end) {
                            add2(mypriv + rowB * TOK + 2 * t, c[2], c[3]);
                            add2(mypriv + rowB * TOK + 8 + 2 * t, d[2], d[3]);
                        }
                        __syncwarp();                  // the next group may add to the same rows
                    }
                }

                // (3) FP8 activation blocks against the NVFP4 weights of the warp's 16 rows
                const uint32_t am0 = *reinterpret_cast<const uint16_t*>(sa + AREC_MASK + g * 2);
                const uint32_t am1 = *reinterpret_cast<const uint16_t*>(sa + AREC_MASK + (g + 8) * 2);
                uint32_t todo = am0 | am1;             // block columns in which any token is FP8
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) todo |= __shfl_xor_sync(0xffffffffu, todo, o);
                while (todo) {
                    const int kb = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const uint32_t bit = 1u << kb;
                    const uint2 at0 = *reinterpret_cast<const uint2*>(sa + AREC_TRUE + kb * 512 + g * 32 + t * 8);
                    const uint2 at1 = *reinterpret_cast<const uint2*>(sa + AREC_TRUE + kb * 512 + (g + 8) * 32 + t * 8);
                    const uint32_t a0 = (am0 & bit) ? at0.x : 0u, a2 = (am0 & bit) ? at0.y : 0u;
                    const uint32_t a1 = (am1 & bit) ? at1.x : 0u, a3 = (am1 & bit) ? at1.y : 0u;
#pragma unroll
                    for (int rg = 0; rg < 2; ++rg) {
                        const uint32_t r = rowbase + 8 * rg + g;       // row inside the tile
                        const uint32_t codes = *reinterpret_cast<const uint16_t*>(sb + REC_W4 + fgmp_rec_w4_offset(r, kb) + t * 2);
                        const uint32_t sfb = sb[REC_SF + fgmp_rec_sf_offset(r, kb)];
                        uint32_t q0, q1, sc2;
                        asm("{\n\t.reg .b8 lo, hi;\n\tmov.b16 {lo, hi}, %2;\n\tcvt.rn.f16x2.e2m1x2 %0, lo;\n\tcvt.rn.f16x2.e2m1x2 %1, hi;\n\t}"
                            : "=r"(q0), "=r"(q1) : "h"((uint16_t)codes));
                        const uint16_t s16 = (uint16_t)(sfb | (sfb << 8));
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2) : "h"(s16));
                        const __half2 x0 = __hmul2(*reinterpret_cast<__half2*>(&q0), *reinterpret_cast<__half2*>(&sc2));
                        const __half2 x1 = __hmul2(*reinterpret_cast<__half2*>(&q1), *reinterpret_cast<__half2*>(&sc2));
                        mma_f16_16816(acc[rg], a0, a1, a2, a3, *reinterpret_cast<const uint32_t*>(&x0), *reinterpret_cast<const uint32_t*>(&x1));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (++stage == DEC_STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;

            // fold the (3) sums into the warp's own tile: acc[rg] = (token g | g+8) x (row 2t | 2t+1)
#pragma unroll
            for (int rg = 0; rg < 2; ++rg) {
                const int r = rowbase + 8 * rg + 2 * t;
                mypriv[r * TOK + g] += acc[rg][0];
                mypriv[(r + 1) * TOK + g] += acc[rg][1];
                mypriv[r * TOK + g + 8] += acc[rg][2];
                mypriv[(r + 1) * TOK + g + 8] += acc[rg][3];
            }
            // all eight tiles are complete for this segment once every correction thread is here
            const uint32_t seg_phase = (uint32_t)(seg & 1);
            mbar_arrive(seg0);
            if (!(ok = mbar_wait(seg0, seg_phase, abort_flag, p.status, 6))) break;

            const int accb = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            if (!(ok = mbar_wait(accf0 + 8 * accb, acc_phase, abort_flag, p.status, 4))) break;
            tc_fence_after();
            uint32_t rr[16];
            tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(accb * TOK), rr);
            tc_fence_before();
            mbar_arrive(acce0 + 8 * accb);
            // lanes 16h .. 16h+15 hold this warp's rows
            const bool mine = (lane >> 4) == h;
            const int lr = lane & 15;
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(rr[j]);
            if (mine) {
#pragma unroll
                for (int w = 0; w < DEC_CORR_WARPS; ++w) {
                    const float4* src = reinterpret_cast<const float4*>(priv + w * PRIV_FLOATS + (rowbase + lr) * TOK);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 x = src[j];
                        v[4 * j] += x.x; v[4 * j + 1] += x.y; v[4 * j + 2] += x.z; v[4 * j + 3] += x.w;
                    }
                }
            }
            // every warp has read all tiles before any tile is cleared for the next segment
            mbar_arrive(seg0 + 8);
            if (!(ok = mbar_wait(seg0 + 8, seg_phase, abort_flag, p.status, 7))) break;
            {
                float4* z = reinterpret_cast<float4*>(mypriv);
#pragma unroll
                for (int i = 0; i < (int)PRIV_FLOATS / 128; ++i) z[i * 32 + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            __syncwarp();

            const int64_t n = tile * 128 + rowbase + lr;
            const bool whole = (seg_begin == tile * C) && (seg_end == (tile + 1) * C);
            bool write_out = whole;
            if (!whole) {
                // partial tile: publish, and let the warp that arrives last add everything up
                const int64_t c_first = cta_of_unit(tile * C, G, p.total);
                const int64_t c_last = cta_of_unit((tile + 1) * C - 1, G, p.total);
                const int nseg = (int)(c_last - c_first + 1);
                const int slot = (int)(blockIdx.x - c_first);
                if (mine) {
                    float* dst = p.partials + (((size_t)tile * p.maxseg + slot) * 128 + rowbase + lr) * 16;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) __stcg(reinterpret_cast<float4*>(dst + j), make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]));
                }
                __threadfence();
                __syncwarp();
                uint32_t old = 0;
                if (lane == 0) old = atomicAdd(p.counters + tile * 8 + slice, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                if (old == (uint32_t)(nseg - 1)) {
                    __threadfence();
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
                    if (mine) {
                        for (int sgi = 0; sgi < nseg; ++sgi) {
                            const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + rowbase + lr) * 16;
#pragma unroll
                            for (int j = 0; j < 16; j += 4) {
                                float4 x = __ldcg(reinterpret_cast<const float4*>(src + j));
                                v[j] += x.x; v[j + 1] += x.y; v[j + 2] += x.z; v[j + 3] += x.w;
                            }
                        }
                    }
                    write_out = true;
                }
            }
            if (write_out && mine && n < p.N) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    if (j < p.M) {
                        if (p.y_is_bf16) reinterpret_cast<__nv_bfloat16*>(p.Ybf)[(int64_t)j * p.ldy + n] = __float2bfloat16_rn(v[j] * alpha);
                        else p.Y[(int64_t)j * p.ldy + n] = v[j] * alpha;
                    }
                }
            }
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
