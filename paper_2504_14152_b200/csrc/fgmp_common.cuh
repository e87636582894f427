// Shared device/host helpers of libfgmp: packed-blob layout arithmetic, number-format
// conversions and the pinned single-precision quantization sequence.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "fgmp.h"

#define FGMP_MAGIC 0x504d4746u
#define FGMP_BS 16

// ---------------------------------------------------------------- blob layout
// A "unit" is one 128-row tile x one chunk of 16 blocks (256 K elements).
//
// Weights (kind 1): header | mask | uptr | records.  Everything a GEMM needs of one unit is one
// contiguous record, so that a unit streams from HBM with a single bulk copy:
//   REC_W4    16384 B : E2M1 codes, row r of the tile = 128 bytes whose 16-byte pieces are
//                       XOR-swizzled with (r & 7) -- the 128B-swizzled K-major tile tcgen05 reads;
//                       zero in FP8 blocks and in rows beyond the tensor
//   REC_SF     2048 B : E4M3 microscales, [128 rows][16 block columns] (the decode GEMM reads two
//                       neighbouring bytes per lane, rows 16 bytes apart: no bank conflicts)
//   REC_KBCNT    16 B : FP8 blocks of the unit per block column
//   REC_KBSTART  48 B : uint16 x 17 (padded): FP8 blocks of the unit before block column j; entry 16 = all
//   REC_ROWID         : row of every FP8 block of the unit, padded to 16 bytes
//   then              : the FP8 blocks, 16 E4M3 codes each, ordered by (block column, row) so that
//                       blocks meeting the same 16 activation elements are neighbours
// Records are 128-byte aligned; uptr[u] (uint32, units + 1 entries) = start of record u in
// 128-byte steps from the first record.
//
// Activations (kind 0): header | codes4 | sf | mask | arec | codes8.  codes4 is row-major, sf
// uses the same 512-byte tiles over all rows, codes8 is a dense plane of which only FP8 blocks are
// written.  arec exists when rows <= 16: one record of AREC_BYTES per chunk holding the fp16 value
// over the tensor scale (E2M1 x microscale, or E4M3 x 2^ratio; exact) of 16 token rows (rows >= M
// are zero), in the order the decode GEMM's mma.sync fragments take them: 16 pieces of 512 bytes,
// piece 2*sp + nh = MMA steps 2sp, 2sp+1 of token octet nh; in a piece lane (g, t) has 16 bytes =
// elements 64t + 8sp .. 64t + 8sp + 7 of token 8nh + g, at 16-byte slot 4g + (t ^ (g & 3)) (the
// XOR spreads the eight tokens of one block column over more banks).
constexpr uint32_t REC_W4 = 0, REC_SF = 16384, REC_KBCNT = 18432, REC_KBSTART = 18448, REC_ROWID = 18496;
constexpr uint32_t AREC_BYTES = 8192;

// byte offset, inside an activation record, of the first (half = 0) or second (half = 1) 8 elements
// of block column j (0..15) of token row m
__host__ __device__ inline uint32_t fgmp_arec_offset(uint32_t m, uint32_t j, uint32_t half)
{
    return ((((((j & 3u) << 1) | half) << 1) | (m >> 3)) << 9) + ((((m & 7u) << 2) | ((j >> 2) ^ (m & 3u))) << 4);
}

struct PackedLayout {
    int64_t rows, K, KB, MW;          // KB = K/16 blocks per row, MW = mask words per row
    int64_t tiles, chunks, units;     // 128-row tiles, 16-block K chunks, tiles * chunks
    size_t off_codes4, off_sf, off_mask, off_arec, off_codes8;   // activations (mask: both)
    size_t off_uptr, off_rec;                                    // weights
    size_t total;
};

__host__ __device__ inline size_t fgmp_align1k(size_t x) { return (x + 1023) & ~(size_t)1023; }

// bytes of the record of a unit with cnt FP8 blocks
__host__ __device__ inline uint32_t fgmp_rec_fp8_offset(uint32_t cnt) { return REC_ROWID + ((cnt + 15u) & ~15u); }
__host__ __device__ inline uint32_t fgmp_rec_bytes(uint32_t cnt) { return (fgmp_rec_fp8_offset(cnt) + cnt * 16u + 127u) & ~127u; }

// kind 0 = activations, 1 = weights (max_fp8 = room for that many FP8 blocks in the records)
__host__ __device__ inline PackedLayout fgmp_layout(int64_t rows, int64_t K, int kind, int64_t max_fp8)
{
    PackedLayout L;
    L.rows = rows; L.K = K; L.KB = K / 16; L.MW = (L.KB + 31) / 32;
    L.tiles = (rows + 127) / 128; L.chunks = (L.KB + 15) / 16; L.units = L.tiles * L.chunks;
    size_t o = 1024;                                   // header section
    L.off_codes4 = L.off_sf = L.off_arec = L.off_codes8 = L.off_uptr = L.off_rec = 0;
    if (kind == 0) {
        L.off_codes4 = o;  o = fgmp_align1k(o + (size_t)rows * (size_t)(K / 2));
        L.off_sf = o;      o = fgmp_align1k(o + (size_t)L.tiles * (size_t)(K / 64) * 512);
        L.off_mask = o;    o = fgmp_align1k(o + (size_t)rows * (size_t)L.MW * 4);
        L.off_arec = o;    if (rows <= 16) o = fgmp_align1k(o + (size_t)L.chunks * AREC_BYTES);
        L.off_codes8 = o;  o = fgmp_align1k(o + (size_t)rows * (size_t)K);
    } else {
        L.off_mask = o;    o = fgmp_align1k(o + (size_t)rows * (size_t)L.MW * 4);
        L.off_uptr = o;    o = fgmp_align1k(o + ((size_t)L.units + 1) * 4);
        L.off_rec = o;
        // a record is at most REC_ROWID + 15 + 127 bytes plus 17 per FP8 block
        o = fgmp_align1k(o + (size_t)L.units * (REC_ROWID + 144) + (size_t)max_fp8 * 17);
    }
    L.total = o;
    return L;
}

// byte offset of the microscale of (row r, block kb) inside the sf section of packed activations
__host__ __device__ inline size_t fgmp_sf_offset(int64_t r, int64_t kb, int64_t K)
{
    return ((size_t)(r >> 7) * (size_t)(K >> 6) + (size_t)(kb >> 2)) * 512
         + (size_t)(r & 31) * 16 + (size_t)((r & 127) >> 5) * 4 + (size_t)(kb & 3);
}

// inside a record (r = row in the tile, j = block column in the chunk): the 8 code bytes and
// the microscale byte
__host__ __device__ inline uint32_t fgmp_rec_w4_offset(uint32_t r, uint32_t j)
{
    return r * 128u + (((j >> 1) ^ (r & 7u)) << 4) + (j & 1u) * 8u;
}
__host__ __device__ inline uint32_t fgmp_rec_sf_offset(uint32_t r, uint32_t j)
{
    return r * 16u + j;
}

#ifdef __CUDACC__
// Where the FP8 blocks of one unit sit in its record.  Called by all 128 threads of a CTA, thread
// i = row i of the tile, m16 = that row's 16 mask bits of the chunk (0 beyond the last row).
// On return s_pos[row * 16 + j] = index of block (row, j) among the unit's FP8 blocks (0xffff if
// the block is not FP8), s_cnt[j] = FP8 blocks in column j, and the return value is their total.
// s_warp is scratch of 64 words.  Ends with a __syncthreads().
__device__ __forceinline__ uint32_t fgmp_unit_positions(uint32_t m16, uint32_t* s_warp, uint16_t* s_pos, uint32_t* s_cnt)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t rank[16];
#pragma unroll
    for (int kb = 0; kb < 16; ++kb) {
        const uint32_t bal = __ballot_sync(0xffffffffu, (m16 >> kb) & 1u);
        rank[kb] = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) s_warp[w * 16 + kb] = __popc(bal);
    }
    __syncthreads();
    uint32_t run = 0;
#pragma unroll
    for (int kb = 0; kb < 16; ++kb) {
        const uint32_t c0 = s_warp[kb], c1 = s_warp[16 + kb], c2 = s_warp[32 + kb], c3 = s_warp[48 + kb];
        const uint32_t below = (w > 0 ? c0 : 0u) + (w > 1 ? c1 : 0u) + (w > 2 ? c2 : 0u);
        s_pos[threadIdx.x * 16 + kb] = ((m16 >> kb) & 1u) ? (uint16_t)(run + below + rank[kb]) : (uint16_t)0xffff;
        if (threadIdx.x == 0) s_cnt[kb] = c0 + c1 + c2 + c3;
        run += c0 + c1 + c2 + c3;
    }
    __syncthreads();
    return run;
}

// the 16 mask bits of (row r, chunk c) of a packed tensor; 0 beyond the last row
__device__ __forceinline__ uint32_t fgmp_chunk_mask(const uint32_t* mask, const PackedLayout& L, int64_t r, int64_t c)
{
    if (r >= L.rows) return 0u;
    return (mask[r * L.MW + (c >> 1)] >> ((c & 1) * 16)) & 0xffffu;
}

struct UnitScratch { uint32_t warp[64]; uint32_t cnt[16]; uint16_t pos[128 * 16]; };

// record of unit u of a packed weight tensor
__device__ __forceinline__ const uint8_t* fgmp_record(const uint8_t* blob, const PackedLayout& L, int64_t u)
{
    return blob + L.off_rec + (size_t)reinterpret_cast<const uint32_t*>(blob + L.off_uptr)[u] * 128;
}

// Visits every block of one unit of a packed weight tensor, 128 threads per unit, consecutive
// threads on consecutive blocks of one row: f(row, kb, row in tile, column in chunk, rec, e8) with
// rec = the unit's record and e8 = address of the block's 16 E4M3 codes, or nullptr if NVFP4.
template <class F>
__device__ __forceinline__ void fgmp_for_each_block(const uint8_t* blob, const PackedLayout& L, int64_t unit,
                                                    UnitScratch& sc, F f)
{
    const int64_t tile = unit / L.chunks, c = unit % L.chunks;
    const uint32_t* mask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const uint32_t m16 = fgmp_chunk_mask(mask, L, tile * 128 + threadIdx.x, c);
    const uint32_t cnt = fgmp_unit_positions(m16, sc.warp, sc.pos, sc.cnt);
    const uint8_t* rec = fgmp_record(blob, L, unit);
    const uint8_t* fp8 = rec + fgmp_rec_fp8_offset(cnt);
    const int j = threadIdx.x & 15;
#pragma unroll 1
    for (int i = 0; i < 16; ++i) {
        const int row = (threadIdx.x >> 4) + 8 * i;
        const int64_t r = tile * 128 + row, kb = c * 16 + j;
        if (r >= L.rows || kb >= L.KB) continue;
        const uint32_t pos = sc.pos[row * 16 + j];
        f(r, kb, row, j, rec, pos != 0xffffu ? fp8 + (size_t)pos * 16 : (const uint8_t*)nullptr);
    }
    __syncthreads();
}
#endif

// ---------------------------------------------------------------- conversions
#ifdef __CUDACC__

// two floats -> two E2M1 codes in one byte: `lo` in bits 0..3, `hi` in bits 4..7.
// Round to nearest even, saturating to +-6 (cvt.rn.satfinite.e2m1x2.f32).
__device__ __forceinline__ uint32_t f32x2_to_e2m1x2(float lo, float hi)
{
    uint32_t r;
    asm("{\n\t.reg .b8 t;\n\tcvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\tcvt.u32.u8 %0, t;\n\t}"
        : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// two floats -> two E4M3 codes: `lo` in bits 0..7, `hi` in bits 8..15 (satfinite, RNE).
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// byte of two E2M1 codes -> two floats (exact)
__device__ __forceinline__ float2 e2m1x2_to_f32x2(uint32_t byte)
{
    uint32_t h2;
    asm("{\n\t.reg .b8 t;\n\tcvt.u8.u32 t, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, t;\n\t}" : "=r"(h2) : "r"(byte));
    __half2 h = *reinterpret_cast<__half2*>(&h2);
    return __half22float2(h);
}

// two E4M3 codes (low 16 bits) -> two floats (exact)
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t two)
{
    uint32_t h2;
    uint16_t s = (uint16_t)two;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(s));
    __half2 h = *reinterpret_cast<__half2*>(&h2);
    return __half22float2(h);
}

__device__ __forceinline__ float e4m3_to_f32(uint32_t code) { return e4m3x2_to_f32x2(code & 0xff).x; }

__device__ __forceinline__ float bf16lo_to_f32(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

// ---------------------------------------------------------------- block math
// One block of 16 values in registers.  Every step below is a single IEEE fp32 operation
// (no contraction): this sequence is what makes codes and scores reproducible bit for bit.

struct BlockQ {
    uint32_t c4[2];     // 16 E2M1 codes, element i in nibble i
    float score;
};

// dynamic-max microscale code: E4M3(amax * k6), k6 = 1 / (6 * s4)
__device__ __forceinline__ uint32_t block_dynamic_scale(const float (&v)[16], float k6)
{
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
    return f32x2_to_e4m3x2(__fmul_rn(amax, k6), 0.f) & 0x7f;
}

// NVFP4 rounding under microscale code `sc`; dq receives the dequantized values
__device__ __forceinline__ void block_nvfp4(const float (&v)[16], uint32_t sc, float s4,
                                            uint32_t (&c4)[2], float (&dq)[16])
{
    float d = __fmul_rn(e4m3_to_f32(sc), s4);
    float inv = (d == 0.f) ? 0.f : __fdiv_rn(1.0f, d);
    c4[0] = 0; c4[1] = 0;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        float y0 = __fmul_rn(v[i], inv), y1 = __fmul_rn(v[i + 1], inv);
        // inv == 0 (zero scale): keep only the signs, as -0.0 * 0 = -0.0 does
        uint32_t b = f32x2_to_e2m1x2(y0, y1);
        float2 q = e2m1x2_to_f32x2(b);
        dq[i] = __fmul_rn(q.x, d);
        dq[i + 1] = __fmul_rn(q.y, d);
        c4[i >> 3] |= b << ((i & 7) * 4);
    }
}

// FP8 rounding of the block: 16 E4M3 codes in 4 words, dq8 = dequantized values
__device__ __forceinline__ void block_fp8(const float (&v)[16], float inv8, float s8,
                                          uint32_t (&c8)[4], float (&dq)[16])
{
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
        uint32_t two = f32x2_to_e4m3x2(__fmul_rn(v[i], inv8), __fmul_rn(v[i + 1], inv8));
        float2 q = e4m3x2_to_f32x2(two);
        dq[i] = __fmul_rn(q.x, s8);
        dq[i + 1] = __fmul_rn(q.y, s8);
        if ((i & 3) == 0) c8[i >> 2] = two; else c8[i >> 2] |= two << 16;
    }
}

// sum_i (f_i * e_i) * e_i, in element order
__device__ __forceinline__ float weighted_sq_sum(const float (&a)[16], const float (&b)[16],
                                                 const float (&f)[16])
{
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float e = __fsub_rn(a[i], b[i]);
        s = __fadd_rn(s, __fmul_rn(__fmul_rn(f[i], e), e));
    }
    return s;
}

// 16 bf16 (two 128-bit words) -> 16 floats
__device__ __forceinline__ void unpack_bf16x16(const uint4& a, const uint4& b, float (&v)[16])
{
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) { v[2 * i] = bf16lo_to_f32(w[i]); v[2 * i + 1] = bf16hi_to_f32(w[i]); }
}

#endif  // __CUDACC__
