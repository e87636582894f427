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
// Weights (kind 1): header | mask | uptr | records | overflow.  A unit's record has a fixed size and
// sits at a fixed place, so that it streams from HBM with one bulk copy whose address needs no
// look-up; what does not fit the fixed part (the second half of every FP8 block) follows in the
// overflow section, found through uptr.  Inside a record the blocks are in the order in which the
// decode GEMM's warps take them: warp w = 4*(r/32) + j%4 owns rows 32*(r/32) .. +31 and the block
// columns j with j%4 == w%4; its lane 4*(r%8) + j/4 holds, as slot k = (r/8)%4, block (r, j).
//   REC_W4    16384 B : one 8-byte slot per block at w*1024 + (k/2)*512 + lane*16 + (k%2)*8: the 16 E2M1
//                       codes of an NVFP4 block, or E4M3 codes 0..7 of an FP8 block
//   REC_SF     2048 B : one byte per block at (w/4)*512 + lane*16 + (w%4)*4 + k (the sixteen blocks of one
//                       lane of the four warps of a row group side by side): the E4M3 microscale (bit 7 clear) of an
//                       NVFP4 block; for an FP8 block 0x80 | E4M3(2^fp8_log2_ratio), i.e. bit 7 is the
//                       block's precision flag and the low bits the factor between the tensor scales
//   REC_WSTART  128 B : uint16 x 17: FP8 blocks of the unit that precede warp w's in (w, lane, k)
//                       order; entry 16 = all of them
// Overflow of a unit: E4M3 codes 8..15 of its FP8 blocks, 8 bytes each, in (w, lane, k) order, padded
// to 16 bytes; uptr[u] (uint32, units + 1 entries) = its start in 16-byte steps from off_ovf.
//
// Activations (kind 0): header | codes4 | sf | mask | arec | codes8.  codes4 is row-major, sf
// uses 512-byte tiles over all rows, codes8 is a dense plane of which only FP8 blocks are
// written.  arec exists when rows <= 16: one record of AREC_BYTES per chunk holding the fp16 value
// over the tensor scale (E2M1 x microscale, or E4M3 x 2^ratio; exact) of 16 token rows (rows >= M
// are zero), in the order the decode GEMM's mma.sync fragments take them: token octet o = m/8 in
// its own half of 4096 bytes; there 8 pieces of 512 bytes, piece 2*(j%4) + half holding elements
// 8*half .. 8*half+7 of block column j of token m for lane 4*(m%8) + j/4, 16 bytes per lane.
constexpr uint32_t REC_W4 = 0, REC_SF = 16384, REC_WSTART = 18432, REC_BYTES = 18560;
constexpr uint32_t AREC_BYTES = 8192;

// byte offset, inside an activation record, of the first (half = 0) or second (half = 1) 8 elements
// of block column j (0..15) of token row m
__host__ __device__ inline uint32_t fgmp_arec_offset(uint32_t m, uint32_t j, uint32_t half)
{
    return ((m >> 3) << 12) + (((((j & 3u) << 1) | half)) << 9) + ((((m & 7u) << 2) | (j >> 2)) << 4);
}

struct PackedLayout {
    int64_t rows, K, KB, MW;          // KB = K/16 blocks per row, MW = mask words per row
    int64_t tiles, chunks, units;     // 128-row tiles, 16-block K chunks, tiles * chunks
    size_t off_codes4, off_sf, off_mask, off_arec, off_codes8;   // activations (mask: both)
    size_t off_uptr, off_rec, off_ovf;                           // weights
    size_t total;
};

__host__ __device__ inline size_t fgmp_align1k(size_t x) { return (x + 1023) & ~(size_t)1023; }

// overflow of a unit with cnt FP8 blocks, in 16-byte steps
__host__ __device__ inline uint32_t fgmp_ovf_steps(uint32_t cnt) { return (cnt + 1u) >> 1; }

// kind 0 = activations, 1 = weights (max_fp8 = room for that many FP8 blocks in the overflow section)
__host__ __device__ inline PackedLayout fgmp_layout(int64_t rows, int64_t K, int kind, int64_t max_fp8)
{
    PackedLayout L;
    L.rows = rows; L.K = K; L.KB = K / 16; L.MW = (L.KB + 31) / 32;
    L.tiles = (rows + 127) / 128; L.chunks = (L.KB + 15) / 16; L.units = L.tiles * L.chunks;
    size_t o = 1024;                                   // header section
    L.off_codes4 = L.off_sf = L.off_arec = L.off_codes8 = L.off_uptr = L.off_rec = L.off_ovf = 0;
    if (kind == 0) {
        L.off_codes4 = o;  o = fgmp_align1k(o + (size_t)rows * (size_t)(K / 2));
        L.off_sf = o;      o = fgmp_align1k(o + (size_t)L.tiles * (size_t)(K / 64) * 512);
        L.off_mask = o;    o = fgmp_align1k(o + (size_t)rows * (size_t)L.MW * 4);
        L.off_arec = o;    if (rows <= 16) o = fgmp_align1k(o + (size_t)L.chunks * AREC_BYTES);
        L.off_codes8 = o;  o = fgmp_align1k(o + (size_t)rows * (size_t)K);
    } else {
        L.off_mask = o;    o = fgmp_align1k(o + (size_t)rows * (size_t)L.MW * 4);
        L.off_uptr = o;    o = fgmp_align1k(o + ((size_t)L.units + 1) * 4);
        L.off_rec = o;     o = fgmp_align1k(o + (size_t)L.units * REC_BYTES);
        // 8 bytes per FP8 block, and up to 8 bytes of padding per unit
        L.off_ovf = o;     o = fgmp_align1k(o + (size_t)max_fp8 * 8 + (size_t)L.units * 8);
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

// inside a record (r = row in the tile, j = block column in the chunk): who holds the block ...
__host__ __device__ inline uint32_t fgmp_rec_warp(uint32_t r, uint32_t j) { return ((r >> 5) << 2) | (j & 3u); }
__host__ __device__ inline uint32_t fgmp_rec_lane(uint32_t r, uint32_t j) { return ((r & 7u) << 2) | (j >> 2); }
__host__ __device__ inline uint32_t fgmp_rec_slot(uint32_t r, uint32_t j) { (void)j; return (r >> 3) & 3u; }
// ... where its 8-byte slot and its scale byte sit, and its rank in the order of the overflow entries
__host__ __device__ inline uint32_t fgmp_rec_w4_offset(uint32_t r, uint32_t j)
{
    const uint32_t k = fgmp_rec_slot(r, j);
    return fgmp_rec_warp(r, j) * 1024u + (k >> 1) * 512u + fgmp_rec_lane(r, j) * 16u + (k & 1u) * 8u;
}
__host__ __device__ inline uint32_t fgmp_rec_sf_offset(uint32_t r, uint32_t j)
{
    const uint32_t w = fgmp_rec_warp(r, j);
    return (w >> 2) * 512u + fgmp_rec_lane(r, j) * 16u + (w & 3u) * 4u + fgmp_rec_slot(r, j);
}
__host__ __device__ inline uint32_t fgmp_rec_order(uint32_t r, uint32_t j)
{
    return ((fgmp_rec_warp(r, j) * 32u + fgmp_rec_lane(r, j)) << 2) | fgmp_rec_slot(r, j);
}
// the inverse: row and block column of slot k of lane `lane` of warp w
__host__ __device__ inline uint32_t fgmp_rec_row(uint32_t w, uint32_t lane, uint32_t k) { return ((w >> 2) << 5) + (k << 3) + (lane >> 2); }
__host__ __device__ inline uint32_t fgmp_rec_col(uint32_t w, uint32_t lane) { return ((lane & 3u) << 2) | (w & 3u); }

// E4M3 code of 2^ratio, -7 <= ratio <= 7 (2^-7 is subnormal)
__host__ __device__ inline uint32_t fgmp_pow2_e4m3(int ratio) { return ratio >= -6 ? (uint32_t)(ratio + 7) << 3 : 0x04u; }

#ifdef __CUDACC__
// the 16 mask bits of (row r, chunk c) of a packed tensor; 0 beyond the last row
__device__ __forceinline__ uint32_t fgmp_chunk_mask(const uint32_t* mask, const PackedLayout& L, int64_t r, int64_t c)
{
    if (r >= L.rows) return 0u;
    return (mask[r * L.MW + (c >> 1)] >> ((c & 1) * 16)) & 0xffffu;
}

// Kernels that walk a unit in record order run 512 threads per unit: thread = (warp w, lane), four
// slots each.  Exclusive prefix over the lanes of a warp of the number of flagged slots (flags = the
// bits 0x80808080 of the lane's four scale bytes, or any word with one bit per flagged slot).
__device__ __forceinline__ uint32_t fgmp_warp_excl_count(uint32_t flags, uint32_t& warp_total)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t cnt = __popc(flags);
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= (uint32_t)o) incl += y;
    }
    warp_total = __shfl_sync(0xffffffffu, incl, 31);
    return incl - cnt;
}

// What thread (w, lane) of a 512-thread CTA needs to read its four blocks of one unit of a packed
// weight tensor: the record, the unit's overflow entries, the lane's four scale bytes and the index
// of the overflow entry of its first FP8 block (its further FP8 blocks follow, in slot order).
struct UnitLaneView { const uint8_t* rec; const uint8_t* ovf; uint32_t sc4, idx; };
__device__ __forceinline__ UnitLaneView fgmp_unit_lane(const uint8_t* blob, const PackedLayout& L, int64_t unit)
{
    UnitLaneView v;
    const uint32_t w = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    v.rec = blob + L.off_rec + (size_t)unit * REC_BYTES;
    v.ovf = blob + L.off_ovf + (size_t)reinterpret_cast<const uint32_t*>(blob + L.off_uptr)[unit] * 16;
    v.sc4 = *reinterpret_cast<const uint32_t*>(v.rec + REC_SF + (w >> 2) * 512u + lane * 16u + (w & 3u) * 4u);
    uint32_t total;
    const uint32_t excl = fgmp_warp_excl_count(v.sc4 & 0x80808080u, total);
    v.idx = reinterpret_cast<const uint16_t*>(v.rec + REC_WSTART)[w] + excl;
    return v;
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
