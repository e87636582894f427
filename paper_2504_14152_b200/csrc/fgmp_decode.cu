// fgmp_linear for decode-sized batches (M <= 16 tokens): a weight-streaming kernel that
// reads the packed weights exactly once (Section 4.1 of the paper: the four block-pair
// products, FP32 accumulation).
//
// At this size the layer is bound by the weight stream, not by arithmetic, and every block pair
// has an exact fp16 form: an E2M1 code times its E4M3 microscale has 6 significant bits, an E4M3
// code times the power of two between the tensor scales has 4.  So both operands go through
// mma.sync m16n8k16 (fp16 in, fp32 accumulation) as their true values over the tensor scales, and
// the mixing of formats costs nothing extra per pair:
//   (1) NVFP4 weight blocks: 16 weight rows are the M side, the tokens the N side.  Lane (g, t)
//       owns, of rows g and g + 8, the 64 elements 64t .. 64t+63 of the unit; MMA step s takes
//       elements 64t + 4s .. 64t + 4s + 3 of every lane (the order of the contraction index is
//       free as long as both operands agree), so a lane's codes are two 16-byte loads per row and
//       all four codes of a step share one microscale.  Codes become fp16 with
//       cvt.rn.f16x2.e2m1x2, times the microscale (exact).  FP8 blocks are zero in this plane.
//   (2) FP8 weight blocks, which a record keeps grouped by block column: sixteen blocks that meet
//       the same 16 activation elements form the M side; the sums are added to their rows in a
//       [row][token] fp32 tile private to the warp.
// The activation quantizer leaves the fp16 values of each 256-element chunk in the order (1)
// reads them, 16 bytes per lane.
//
// Work is split stream-K style over (128-row tile, 256-element K chunk) units so that all SMs
// stream the same number of bytes; a unit is two bulk copies (its weight record, the activation
// record of its chunk).  Tiles shared by several CTAs are reduced in a fixed order by the CTA
// that arrives last.  Every sum is taken in a fixed order: results are reproducible bit for bit.
//
// Warp roles (672 threads): warp 0 = producer, warps 1-4 = epilogue (32 rows each), warps 5-12 =
// (1): warp (jr, h) does rows 32jr .. 32jr+31, MMA steps 8h .. 8h+7, warps 13-20 = (2), two block
// columns each.  Either kind alone keeps up with the weight stream; on warps of their own they run
// beside each other.
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <cuda_fp16.h>
#include <type_traits>

namespace {

constexpr int MAIN_WARPS = 8, FP8_WARPS = 8, MATH_WARPS = MAIN_WARPS + FP8_WARPS;
constexpr int DEC_THREADS = 32 * (1 + 4 + MATH_WARPS);
constexpr int TOK = 16;                         // token rows of a tile (zero padded)
constexpr uint32_t FP8_CAP_BLOCKS = 320;        // FP8 blocks of a unit that fit a stage; more are read from global
constexpr uint32_t WREC_CAP = (REC_ROWID + FP8_CAP_BLOCKS + FP8_CAP_BLOCKS * 16 + 127) & ~127u;   // 23936
constexpr uint32_t STG_A = (WREC_CAP + 1023) & ~1023u;                                           // 24576
constexpr uint32_t DEC_STAGE_BYTES = STG_A + AREC_BYTES;                                         // 32768
constexpr int DEC_STAGES = 4;                   // at most; a launch uses DecParams::stages of them
constexpr int NTILES = FP8_WARPS + 2;           // [row][token] fp32 tiles: one per (2) warp, one per half of the MMA steps of (1)
constexpr uint32_t TILE_FLOATS = 128 * TOK;
constexpr size_t dec_smem(int stages) { return (size_t)stages * DEC_STAGE_BYTES + NTILES * TILE_FLOATS * 4 + 1024 /*alignment*/ + 512 /*barriers*/; }
constexpr size_t DEC_SMEM = dec_smem(DEC_STAGES);
static_assert(DEC_SMEM <= 232448, "shared memory of one CTA");

struct DecParams {
    const uint8_t* wblob; const uint8_t* ablob;
    PackedLayout LW, LA;
    float* Y; void* Ybf; int64_t ldy; int y_is_bf16;
    int64_t M, N, K;
    int64_t total;            // tiles * chunks
    int64_t chunks;
    int* status; uint32_t* counters; float* partials; int maxseg;
    int stages;               // depth of the unit ring, 2 .. DEC_STAGES
};

struct StageMeta { uint32_t step, staged; };     // record start (128-byte steps), bytes of it in the stage

__device__ __forceinline__ int64_t cta_of_unit(int64_t i, int64_t G, int64_t total) { return ((i + 1) * G - 1) / total; }

// A tile holds [128 rows][16 tokens] fp32, a row = 64 bytes = four 16-byte pieces of four tokens;
// piece index is XOR-ed with (row >> 1) & 3 so that 32 lanes reading one piece of 32 consecutive
// rows (the epilogue) do not collide on banks.

// eight E2M1 codes (one word) times a microscale (both halves of sc2) -> four fp16 pairs, exact
__device__ __forceinline__ void dq8(uint32_t c32, uint32_t sc2, uint32_t (&x)[4])
{
    uint32_t q0, q1, q2, q3;
    asm("{\n\t.reg .b8 b0, b1, b2, b3;\n\tmov.b32 {b0, b1, b2, b3}, %4;\n\t"
        "cvt.rn.f16x2.e2m1x2 %0, b0;\n\tcvt.rn.f16x2.e2m1x2 %1, b1;\n\t"
        "cvt.rn.f16x2.e2m1x2 %2, b2;\n\tcvt.rn.f16x2.e2m1x2 %3, b3;\n\t}"
        : "=r"(q0), "=r"(q1), "=r"(q2), "=r"(q3) : "r"(c32));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[0]) : "r"(q0), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[1]) : "r"(q1), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[2]) : "r"(q2), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[3]) : "r"(q3), "r"(sc2));
}

// NH = token octets in use: 1 for M <= 8, else 2
template <int NH>
__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(DecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    // 1 KiB aligned; an offset from the array keeps the pointer known to be shared memory (plain ld.shared / st.shared)
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int S = p.stages;
    float* tiles = reinterpret_cast<float*>(smem + (size_t)S * DEC_STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NTILES * TILE_FLOATS);
    // bars (S = stages): [0,S) full, [S,2S) empty, then sums of a segment in the tiles [2], tiles free [1]
    StageMeta* smeta = reinterpret_cast<StageMeta*>(bars + 2 * DEC_STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smeta + DEC_STAGES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * DEC_STAGES;
    const uint32_t cdone0 = empty0 + 8 * DEC_STAGES, tfree = cdone0 + 16;

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
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, MATH_WARPS); }
        for (int b = 0; b < 2; ++b) mbar_init(cdone0 + 8 * b, MATH_WARPS);
        mbar_init(tfree, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp >= 5) {                                   // the tiles of (2) start at zero
        float4* z = reinterpret_cast<float4*>(tiles);
        for (int i = (warp - 5) * 32 + lane; i < (int)(FP8_WARPS * TILE_FLOATS / 4); i += MATH_WARPS * 32) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // One unit's two copies into a stage (lane 0 of the producer warp): the weight record, then the
    // activation record of the unit's chunk
    const uint8_t* arec = p.ablob + p.LA.off_arec;
    auto issue_w = [&](int stage, uint32_t step0, uint32_t step1) {
        const uint32_t bytes = (step1 - step0) * 128u;
        const uint32_t staged = bytes < WREC_CAP ? bytes : WREC_CAP;
        smeta[stage].step = step0; smeta[stage].staged = staged;
        const uint32_t fb = full0 + 8 * stage;
        mbar_expect_tx(fb, staged + AREC_BYTES);
        bulk_load(smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES), recs + (size_t)step0 * 128, staged, fb);
    };
    auto issue_a = [&](int64_t u, int stage) {
        bulk_load(smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES) + STG_A, arec + (size_t)(u % C) * AREC_BYTES, AREC_BYTES, full0 + 8 * stage);
    };
    // The first stages need no consumer to have freed them, and the packed weights are not written by
    // whatever runs before this kernel: their copies start before the CTA has finished setting itself
    // up (thread 0, which initialised the barriers, issues them) and before the wait below.
    int pre = 0;
    if (warp == 0) {
        pre = (int)min((int64_t)S, u_end - u_begin);
        for (int s = 0; s < pre; ++s) {
            const uint32_t step0 = __shfl_sync(0xffffffffu, pf, s), step1 = __shfl_sync(0xffffffffu, pf, s + 1);
            if (lane == 0) issue_w(s, step0, step1);
        }
    }
    __syncthreads();
    // Launched as a programmatic dependent of the preceding kernel in the stream (normally the
    // activation quantizer), this kernel may have started before that one finished: everything above
    // touches neither its output nor the workspace.  From here on both are read.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        // ------------------------------------------------------------ producer (whole warp; lane 0 issues)
        if (lane == 0)
            for (int s = 0; s < pre; ++s) issue_a(u_begin + s, s);
        int stage = pre % S; uint32_t phase = (uint32_t)(pre / S) & 1u;
        for (int64_t u = u_begin + pre; u < u_end; ++u) {
            if (u + 1 - pf_base > 31) {                // next 32 record offsets
                pf_base = u;
                pf = (pf_base + lane <= p.total) ? __ldg(uptr + pf_base + lane) : 0u;
            }
            const uint32_t step0 = __shfl_sync(0xffffffffu, pf, (int)(u - pf_base));
            const uint32_t step1 = __shfl_sync(0xffffffffu, pf, (int)(u + 1 - pf_base));
            int ok = 1;
            if (lane == 0) {
                ok = mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1) ? 1 : 0;
                if (ok) { issue_w(stage, step0, step1); issue_a(u, stage); }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) break;
            if (++stage == S) { stage = 0; phase ^= 1; }
        }
    } else if (warp < 5) {
        // ------------------------------------------------------------ epilogue: rows 32q .. 32q + 31 of the tile
        const int q = warp - 1;
        const fgmp_packed_header* ha = reinterpret_cast<const fgmp_packed_header*>(p.ablob);
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const float alpha = __fmul_rn(ha->scale_fp4, hw->scale_fp4);
        const int row = 32 * q + lane;
        bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_begin = u, seg_end = min(u_end, (tile + 1) * C);
            u = seg_end;
            const int accb = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            // a tile shared with other CTAs: how many of them have handed in their sums already (the answer is
            // needed only after this CTA's own sums are complete, so the load costs nothing)
            const bool whole = (seg_begin == tile * C) && (seg_end == (tile + 1) * C);
            int nseg = 1, slot = 0;
            uint32_t seen = 0;
            if (!whole) {
                const int64_t c_first = cta_of_unit(tile * C, G, p.total);
                const int64_t c_last = cta_of_unit((tile + 1) * C - 1, G, p.total);
                nseg = (int)(c_last - c_first + 1);
                slot = (int)(blockIdx.x - c_first);
                if (lane == 0) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.counters + tile * 8 + q) : "memory");
            }
            // the segment's sums: this row of every tile, in tile order; the rows of (2) are cleared for the
            // next segment on the way
            if (!(ok = mbar_wait(cdone0 + 8 * accb, acc_phase, abort_flag, p.status, 6))) break;
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0.f;
#pragma unroll
            for (int w = 0; w < NTILES; ++w) {
                float4* src = reinterpret_cast<float4*>(tiles + w * TILE_FLOATS + row * TOK);
                float4 x[2 * NH];
#pragma unroll
                for (int j = 0; j < 2 * NH; ++j) x[j] = src[(j ^ (row >> 1)) & 3];  // tokens 4j .. 4j+3
#pragma unroll
                for (int j = 0; j < 2 * NH; ++j) {
                    v[4 * j] += x[j].x; v[4 * j + 1] += x[j].y; v[4 * j + 2] += x[j].z; v[4 * j + 3] += x[j].w;
                    if (w < FP8_WARPS) src[(j ^ (row >> 1)) & 3] = make_float4(0.f, 0.f, 0.f, 0.f);   // the tiles of (1) are overwritten
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(tfree);

            const int64_t n = tile * 128 + row;
            bool write_out = whole;
            if (!whole) {
                // partial tile: publish, and let the warp that arrives last add everything up.  When all the
                // others were seen to have arrived, this warp is the last without asking and skips the counter.
                float* dst = p.partials + (((size_t)tile * p.maxseg + slot) * 128 + row) * 16;
#pragma unroll
                for (int j = 0; j < 8 * NH; j += 4) __stcg(reinterpret_cast<float4*>(dst + j), make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]));
                // The counter wraps to zero with the last arrival (or is put back by the warp that skipped
                // it), so the workspace is ready for the next call without being cleared.
                uint32_t old = __shfl_sync(0xffffffffu, seen, 0);
                if (old != (uint32_t)(nseg - 1)) {
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) old = atomicInc(p.counters + tile * 8 + q, (uint32_t)(nseg - 1));
                    old = __shfl_sync(0xffffffffu, old, 0);
                } else if (lane == 0) {
                    p.counters[tile * 8 + q] = 0u;
                }
                if (old == (uint32_t)(nseg - 1)) {
                    __threadfence();
                    // all partials first (independent loads), then one sum in slot order
                    float4 x[4][2 * NH];
#pragma unroll
                    for (int sgi = 0; sgi < 4; ++sgi) {
                        const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16;
#pragma unroll
                        for (int j = 0; j < 2 * NH; ++j)
                            x[sgi][j] = sgi < nseg ? __ldcg(reinterpret_cast<const float4*>(src) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
#pragma unroll
                    for (int sgi = 0; sgi < 4; ++sgi) {
#pragma unroll
                        for (int j = 0; j < 2 * NH; ++j) {
                            v[4 * j] += x[sgi][j].x; v[4 * j + 1] += x[sgi][j].y; v[4 * j + 2] += x[sgi][j].z; v[4 * j + 3] += x[sgi][j].w;
                        }
                    }
                    for (int sgi = 4; sgi < nseg; ++sgi) {       // more than four contributors: rare, serial
                        const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16;
#pragma unroll
                        for (int j = 0; j < 8 * NH; j += 4) {
                            const float4 y4 = __ldcg(reinterpret_cast<const float4*>(src + j));
                            v[j] += y4.x; v[j + 1] += y4.y; v[j + 2] += y4.z; v[j + 3] += y4.w;
                        }
                    }
                    write_out = true;
                }
            }
            if (write_out && n < p.N) {
#pragma unroll
                for (int j = 0; j < 8 * NH; ++j) {
                    if (j < p.M) {
                        if (p.y_is_bf16) reinterpret_cast<__nv_bfloat16*>(p.Ybf)[(int64_t)j * p.ldy + n] = __float2bfloat16_rn(v[j] * alpha);
                        else p.Y[(int64_t)j * p.ldy + n] = v[j] * alpha;
                    }
                }
            }
        }
    } else if (warp < 5 + MAIN_WARPS) {
        // ------------------------------------------------------------ (1): NVFP4 weight blocks
        const int w = warp - 5;
        const int jr = w & 3, h = w >> 2;
        const uint32_t g = lane >> 2, t = lane & 3;
        float* htile = tiles + (FP8_WARPS + h) * TILE_FLOATS;          // sums of a segment: rows 32jr .. 32jr+31 of the tile of this h
        // this lane's codes and microscales of rows 32jr + 16mt + 8rh + g
        uint32_t w4_off[2][2], sf_off[2][2];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const uint32_t r = (uint32_t)(32 * jr + 16 * mt + 8 * rh) + g;
                w4_off[mt][rh] = REC_W4 + r * 128 + (((2 * t + (uint32_t)h) ^ g) << 4);
                sf_off[mt][rh] = REC_SF + r * 16 + 4 * t + 2 * (uint32_t)h;
            }
        const uint32_t a_off = STG_A + (uint32_t)(8 * h) * 512 + ((g << 2) | (t ^ (g & 3u))) * 16;
        const uint32_t tcol = (2 * t) & 3u, tpiece = t >> 1;

        int stage = 0; uint32_t phase = 0; bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_end = min(u_end, (tile + 1) * C);
            float acc[2][NH][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) acc[mt][nh][0] = acc[mt][nh][1] = acc[mt][nh][2] = acc[mt][nh][3] = 0.f;
            for (; u < seg_end; ++u) {
                if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 5))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                uint4 cw[2][2];
                uint32_t sc2[2][2][2];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                    for (int rh = 0; rh < 2; ++rh) {
                        cw[mt][rh] = *reinterpret_cast<const uint4*>(sb + w4_off[mt][rh]);
                        const uint32_t s16 = *reinterpret_cast<const uint16_t*>(sb + sf_off[mt][rh]);
                        const uint32_t s0 = __byte_perm(s16, 0u, 0x4400), s1 = __byte_perm(s16, 0u, 0x4411);
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2[mt][rh][0]) : "h"((uint16_t)s0));
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2[mt][rh][1]) : "h"((uint16_t)s1));
                    }
#pragma unroll
                for (int sp = 0; sp < 4; ++sp) {
                    const uint4 alo = *reinterpret_cast<const uint4*>(sb + a_off + (uint32_t)sp * 1024);
                    uint4 ahi = make_uint4(0, 0, 0, 0);
                    if (NH == 2) ahi = *reinterpret_cast<const uint4*>(sb + a_off + (uint32_t)sp * 1024 + 512);
                    uint32_t xg[2][4], xg8[2][4];       // rows g / g + 8 of both M tiles: steps 2sp (0, 1) and 2sp + 1 (2, 3)
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        const uint32_t wg = sp == 0 ? cw[mt][0].x : sp == 1 ? cw[mt][0].y : sp == 2 ? cw[mt][0].z : cw[mt][0].w;
                        const uint32_t wg8 = sp == 0 ? cw[mt][1].x : sp == 1 ? cw[mt][1].y : sp == 2 ? cw[mt][1].z : cw[mt][1].w;
                        dq8(wg, sc2[mt][0][sp >> 1], xg[mt]);
                        dq8(wg8, sc2[mt][1][sp >> 1], xg8[mt]);
                    }
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
#pragma unroll
                        for (int mt = 0; mt < 2; ++mt) {
                            mma_f16_16816(acc[mt][0], xg[mt][2 * half], xg8[mt][2 * half], xg[mt][2 * half + 1], xg8[mt][2 * half + 1],
                                          half ? alo.z : alo.x, half ? alo.w : alo.y);
                            if (NH == 2)
                                mma_f16_16816(acc[mt][NH - 1], xg[mt][2 * half], xg8[mt][2 * half], xg[mt][2 * half + 1], xg8[mt][2 * half + 1],
                                              half ? ahi.z : ahi.x, half ? ahi.w : ahi.y);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (++stage == S) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            // the epilogue has taken the previous segment's sums; now this segment's go in:
            // acc[mt][nh] = rows 32jr + 16mt + {g, g + 8} x tokens 8nh + {2t, 2t+1}
            if (seg > 0 && !(ok = mbar_wait(tfree, (uint32_t)(seg - 1) & 1u, abort_flag, p.status, 7))) break;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int rh = 0; rh < 2; ++rh) {
                    const uint32_t r = (uint32_t)(32 * jr + 16 * mt + 8 * rh) + g;
                    float2* pt = reinterpret_cast<float2*>(htile + r * 16u + (((tpiece ^ (r >> 1)) & 3u) << 2) + tcol);
                    pt[0] = make_float2(acc[mt][0][2 * rh], acc[mt][0][2 * rh + 1]);
                    if (NH == 2)
                        *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pt) ^ 32) = make_float2(acc[mt][NH - 1][2 * rh], acc[mt][NH - 1][2 * rh + 1]);
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(cdone0 + 8 * (seg & 1));
        }
    } else {
        // ------------------------------------------------------------ (2): FP8 weight blocks of block columns cw, cw + 8
        const int cw = warp - 5 - MAIN_WARPS;
        const uint32_t g = lane >> 2, t = lane & 3;
        float* mytile = tiles + cw * TILE_FLOATS;
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const float r8 = __int_as_float((127 + hw->fp8_log2_ratio) << 23);     // FP8 tensor scale / NVFP4 tensor scale of the weights
        // where this lane's activation fragments of the two columns sit (token g; token g + 8 is 512 bytes on)
        uint32_t boff[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const uint32_t j = (uint32_t)cw + 8u * hh;
            boff[hh] = STG_A + fgmp_arec_offset(g, j, t >> 1) + (t & 1u) * 8;
        }
        const uint32_t tcol = (2 * t) & 3u, tpiece = t >> 1;

        int stage = 0; uint32_t phase = 0; bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_end = min(u_end, (tile + 1) * C);
            // the epilogue has taken (and cleared) the previous segment's sums
            if (seg > 0 && !(ok = mbar_wait(tfree, (uint32_t)(seg - 1) & 1u, abort_flag, p.status, 7))) break;
            for (; u < seg_end; ++u) {
                if (!(ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 5))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint32_t staged = smeta[stage].staged;
                const uint8_t* rec_g = recs + (size_t)smeta[stage].step * 128;
                const uint16_t* kbs = reinterpret_cast<const uint16_t*>(sb + REC_KBSTART);
                const uint32_t ntot = kbs[16];
                const uint32_t off8 = fgmp_rec_fp8_offset(ntot);
                const uint32_t start[2] = {kbs[cw], kbs[cw + 8]}, end[2] = {kbs[cw + 1], kbs[cw + 9]};
                // B fragments: activation values of tokens g and g + 8, elements 4t..4t+3 of each column
                const uint2 b00 = *reinterpret_cast<const uint2*>(sb + boff[0]), b10 = *reinterpret_cast<const uint2*>(sb + boff[1]);
                uint2 b01 = make_uint2(0, 0), b11 = b01;
                if (NH == 2) { b01 = *reinterpret_cast<const uint2*>(sb + boff[0] + 512); b11 = *reinterpret_cast<const uint2*>(sb + boff[1] + 512); }

                // ALL = every FP8 block of the unit is in the stage (the usual case); otherwise the tail of the
                // list is read from global memory
                auto body = [&](auto all_c) {
                    constexpr bool ALL = decltype(all_c)::value;
                    // One group of up to 16 blocks of one column: blocks e + g and e + g + 8 are the M side.
                    // c/d[0..1]: block iA, tokens 2t, 2t+1 / 8+2t, 9+2t; [2..3]: block iB.
                    auto group_mma = [&](uint32_t e, uint32_t end_, const uint2& bt0, const uint2& bt1, float (&c)[4], float (&d)[4],
                                         uint32_t& rowA, uint32_t& rowB) {
                        const uint32_t iA = e + g, iB = iA + 8;
                        uint32_t rawA = 0, rawB = 0;
                        rowA = 0xffffffffu; rowB = 0xffffffffu;
                        if (iA < end_) {
                            const uint32_t o = off8 + iA * 16 + t * 4;
                            rawA = (ALL || o + 4 <= staged) ? *reinterpret_cast<const uint32_t*>(sb + o) : __ldg(reinterpret_cast<const uint32_t*>(rec_g + o));
                            rowA = (ALL || REC_ROWID + iA < staged) ? sb[REC_ROWID + iA] : __ldg(rec_g + REC_ROWID + iA);
                        }
                        if (iB < end_) {
                            const uint32_t o = off8 + iB * 16 + t * 4;
                            rawB = (ALL || o + 4 <= staged) ? *reinterpret_cast<const uint32_t*>(sb + o) : __ldg(reinterpret_cast<const uint32_t*>(rec_g + o));
                            rowB = (ALL || REC_ROWID + iB < staged) ? sb[REC_ROWID + iB] : __ldg(rec_g + REC_ROWID + iB);
                        }
                        uint32_t a0, a1, a2, a3;
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a0) : "h"((uint16_t)rawA));
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a2) : "h"((uint16_t)(rawA >> 16)));
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a1) : "h"((uint16_t)rawB));
                        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a3) : "h"((uint16_t)(rawB >> 16)));
                        c[0] = c[1] = c[2] = c[3] = 0.f; d[0] = d[1] = d[2] = d[3] = 0.f;
                        mma_f16_16816(c, a0, a1, a2, a3, bt0.x, bt0.y);
                        if (NH == 2) mma_f16_16816(d, a0, a1, a2, a3, bt1.x, bt1.y);
                    };
                    // tile[row][tokens] += 2^ratio x sums.  Within one column every block has its own row, so the
                    // read-modify-writes of a group touch distinct addresses: all loads first, then all stores.
                    auto group_add = [&](const float (&c)[4], const float (&d)[4], uint32_t rowA, uint32_t rowB) {
                        float2 *pA = nullptr, *pB = nullptr;    // tokens 2t, 2t+1; tokens 8+2t, 9+2t are 8 floats on (piece ^ 2)
                        float2 vA0 = make_float2(0.f, 0.f), vA1 = vA0, vB0 = vA0, vB1 = vA0;
                        if (rowA != 0xffffffffu) {
                            pA = reinterpret_cast<float2*>(mytile + rowA * 16u + (((tpiece ^ (rowA >> 1)) & 3u) << 2) + tcol);
                            vA0 = pA[0];
                            if (NH == 2) vA1 = *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pA) ^ 32);
                        }
                        if (rowB != 0xffffffffu) {
                            pB = reinterpret_cast<float2*>(mytile + rowB * 16u + (((tpiece ^ (rowB >> 1)) & 3u) << 2) + tcol);
                            vB0 = pB[0];
                            if (NH == 2) vB1 = *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pB) ^ 32);
                        }
                        if (rowA != 0xffffffffu) {
                            pA[0] = make_float2(fmaf(c[0], r8, vA0.x), fmaf(c[1], r8, vA0.y));
                            if (NH == 2) *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pA) ^ 32) = make_float2(fmaf(d[0], r8, vA1.x), fmaf(d[1], r8, vA1.y));
                        }
                        if (rowB != 0xffffffffu) {
                            pB[0] = make_float2(fmaf(c[2], r8, vB0.x), fmaf(c[3], r8, vB0.y));
                            if (NH == 2) *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pB) ^ 32) = make_float2(fmaf(d[2], r8, vB1.x), fmaf(d[3], r8, vB1.y));
                        }
                        __syncwarp();                  // a later group may add to the same rows
                    };
                    // the first group of both columns side by side (their MMAs are independent), then their sums in order
                    {
                        float c0[4], d0[4], c1[4], d1[4];
                        uint32_t rA0, rB0, rA1, rB1;
                        group_mma(start[0], end[0], b00, b01, c0, d0, rA0, rB0);
                        group_mma(start[1], end[1], b10, b11, c1, d1, rA1, rB1);
                        group_add(c0, d0, rA0, rB0);
                        group_add(c1, d1, rA1, rB1);
                    }
                    // columns with more than 16 FP8 blocks
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        for (uint32_t e = start[hh] + 16; e < end[hh]; e += 16) {
                            float c[4], d[4];
                            uint32_t rA, rB;
                            group_mma(e, end[hh], hh ? b10 : b00, hh ? b11 : b01, c, d, rA, rB);
                            group_add(c, d, rA, rB);
                        }
                    }
                };
                if (off8 + ntot * 16 <= staged) body(std::true_type{}); else body(std::false_type{});
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (++stage == S) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(cdone0 + 8 * (seg & 1));
        }
    }

    __syncthreads();
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
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

// Workspace of the decode path: status word at 0, stream-K tile counters at 1024 (32 bytes per
// tile), both inside the control area that must be zero before a call; partial sums behind it.
bool fgmp_decode_supported(int64_t M, int64_t N, int64_t K)
{
    return M >= 1 && M <= 16 && N >= 1 && K >= 256 && (K % 256) == 0 &&
           1024 + ((N + 127) / 128) * 32 <= (int64_t)FGMP_WS_CONTROL_BYTES;
}

size_t fgmp_ws_decode(int64_t M, int64_t N, int64_t K)
{
    if (!fgmp_decode_supported(M, N, K)) return 0;
    const DecPlan d = decode_plan(N, K);
    return (size_t)FGMP_WS_CONTROL_BYTES + (size_t)d.tiles * d.maxseg * 128 * 16 * 4;
}

// clear_first: zero the control area on the stream before the kernel (for scratch whose state the
// caller cannot vouch for); otherwise the kernel is launched as a programmatic dependent of the
// kernel before it in the stream, so that its set-up and first weight copies overlap that kernel's end.
fgmp_status fgmp_linear_decode(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                               int64_t M, int64_t N, int64_t K, void* workspace, bool clear_first, cudaStream_t s)
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
    p.partials = reinterpret_cast<float*>(ws + FGMP_WS_CONTROL_BYTES);
    p.maxseg = d.maxseg;
    // Ring depth: long spans of few tokens are bound by the weight stream and want every stage; the others
    // are bound by arithmetic or by set-up and run as fast or faster with a smaller footprint (measured on
    // Llama-2 shapes).
    p.stages = (d.total / d.grid >= 24 && M <= 8) ? DEC_STAGES : DEC_STAGES - 1;

    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(decode_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess)
            return FGMP_ERR_CUDA;
        attr_set[dev] = true;
    }
    if (clear_first && cudaMemsetAsync(ws, 0, 1024 + (size_t)d.tiles * 32, s) != cudaSuccess) return FGMP_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)d.grid); cfg.blockDim = dim3(DEC_THREADS); cfg.dynamicSmemBytes = dec_smem(p.stages); cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = clear_first ? 0 : 1;
    if (M <= 8) { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<1>, p)); }
    else        { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<2>, p)); }
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
    // the status word and the tile counters at the start of the scratch are zeroed first; the
    // partial sums behind them are always written before they are read
    st = fgmp_linear_decode(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, scratch, true, s);
    if (st != FGMP_OK) return st;
    if (status_out && cudaMemcpyAsync(status_out, scratch, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return FGMP_ERR_CUDA;
    return FGMP_OK;
}
