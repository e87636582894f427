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
// Weights (kind 1): header | mask | uptr | records | lists.  A unit's record has a fixed size and
// sits at a fixed place, so that it streams from HBM with one bulk copy whose address needs no
// look-up; the list of its FP8 blocks follows in the lists section, found through uptr.
//   REC_W4    16384 B : one 8-byte slot per block, row r of the tile = 128 bytes whose 16-byte pieces are
//                       XOR-swizzled with (r & 7) -- the 128B-swizzled K-major tile tcgen05 reads: the 16
//                       E2M1 codes of an NVFP4 block, or E4M3 codes 0..7 of an FP8 block (which the tensor
//                       core ignores because the block's scale byte is zero); zero in rows beyond the tensor
//   REC_SF     2048 B : E4M3 microscales, 0x00 for FP8 blocks, in the order the scales go to tensor
//                       memory: four 512-byte tiles (one per MMA step of 64 elements), in a tile 16 bytes
//                       per r % 32, there 4 bytes per r / 32, there one byte per block of the step
//   REC_KBSTART 128 B : uint16 x 17 (padded): FP8 blocks of the unit before block column j; entry 16 = all
// List of a unit with cnt FP8 blocks, ordered by (block column, row) so that blocks meeting the same 16
// activation elements are neighbours: one uint32 per block (padded to 16 bytes) -- low half: where the
// block's slot sits in REC_W4, high half: 16 * row + 4 * ((row / 2) % 4), the place of its row in a swizzled
// [row][16 tokens] fp32 tile -- then E4M3 codes 8..15 of every block (8 bytes each, padded to 16).  uptr[u] (uint32, units + 1 entries) = start of
// unit u's list in 16-byte steps from off_ovf.
//
// Activations (kind 0): header | codes4 | sf | mask | arec | codes8.  codes4 is row-major, sf
// uses 512-byte tiles over all rows, codes8 is a dense plane of which only FP8 blocks are
// written.  arec exists when rows <= 16: one record of AREC_BYTES per chunk for the decode GEMM, 16
// token rows (rows >= M are zero):
//   AREC_A4   2048 B : the E2M1 codes as a 16-row x 128-byte tile, swizzled like REC_W4 (zero in FP8 blocks)
//   AREC_SF    256 B : E4M3 microscales, [token][block column], 0x00 for FP8 blocks
//   AREC_HOT    16 B : two uint32, one per token octet (readers use their OR): bit j set if block column j of some token is
//                      FP8 ("hot" column); then padding
//   AREC_AT   8192 B : the value over the tensor scale of every element in fp16 (E2M1 x microscale, or E4M3 x
//                      2^ratio; exact): token octet m / 8 in its own 4096 bytes, there 256 bytes per block
//                      column, there 32 bytes per token -- what a warp reads for one column is contiguous
constexpr uint32_t REC_W4 = 0, REC_SF = 16384, REC_KBSTART = 18432, REC_BYTES = 18560;
constexpr uint32_t AREC_A4 = 0, AREC_SF = 2048, AREC_HOT = 2304, AREC_AT = 2560, AREC_BYTES = 10752;

// byte offset, inside an activation record, of the fp16 values of block column j (0..15) of token row m
__host__ __device__ inline uint32_t fgmp_arec_at_offset(uint32_t m, uint32_t j)
{
    return AREC_AT + ((m >> 3) << 12) + (j << 8) + ((m & 7u) << 5);
}

struct PackedLayout {
    int64_t rows, K, KB, MW;          // KB = K/16 blocks per row, MW = mask words per row
    int64_t tiles, chunks, units;     // 128-row tiles, 16-block K chunks, tiles * chunks
    size_t off_codes4, off_sf, off_mask, off_arec, off_codes8;   // activations (mask: both)
    size_t off_uptr, off_rec, off_ovf;                           // weights
    size_t total;
};

__host__ __device__ inline size_t fgmp_align1k(size_t x) { return (x + 1023) & ~(size_t)1023; }

// list of a unit with cnt FP8 blocks: where the second halves start, and its size in 16-byte steps
__host__ __device__ inline uint32_t fgmp_list_halves_offset(uint32_t cnt) { return (cnt * 4u + 15u) & ~15u; }
__host__ __device__ inline uint32_t fgmp_list_entry(uint32_t row, uint32_t j);
__host__ __device__ inline uint32_t fgmp_list_steps(uint32_t cnt) { return (fgmp_list_halves_offset(cnt) + ((cnt * 8u + 15u) & ~15u)) >> 4; }

// kind 0 = activations, 1 = weights (max_fp8 = room for that many FP8 blocks in the lists section)
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
        // 12 bytes per FP8 block, and up to 24 bytes of padding per unit
        L.off_ovf = o;     o = fgmp_align1k(o + (size_t)max_fp8 * 12 + (size_t)L.units * 32);
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

// inside a record or the A4 tile of an activation record (r = row in the tile, j = block column in the
// chunk): the 8-byte slot and the scale byte
__host__ __device__ inline uint32_t fgmp_rec_w4_offset(uint32_t r, uint32_t j)
{
    return r * 128u + (((j >> 1) ^ (r & 7u)) << 4) + (j & 1u) * 8u;
}
__host__ __device__ inline uint32_t fgmp_rec_sf_offset(uint32_t r, uint32_t j)
{
    return (j >> 2) * 512u + (r & 31u) * 16u + (r >> 5) * 4u + (j & 3u);
}

// what a unit's list says about its FP8 block (row r of the tile, block column j)
__host__ __device__ inline uint32_t fgmp_list_entry(uint32_t r, uint32_t j)
{
    return fgmp_rec_w4_offset(r, j) | ((r * 16u + (((r >> 1) & 3u) << 2)) << 16);
}

#ifdef __CUDACC__
// Where the FP8 blocks of one unit sit in its list.  Called by all 128 threads of a CTA, thread
// i = row i of the tile, m16 = that row's 16 mask bits of the chunk (0 beyond the last row).
// On return s_pos[row * 16 + j] = index of block (row, j) among the unit's FP8 blocks in (column, row)
// order (0xffff if the block is not FP8), s_cnt[j] = FP8 blocks in column j, and the return value is
// their total.  s_warp is scratch of 64 words.  Ends with a __syncthreads().
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

// Visits every block of one unit of a packed weight tensor, 128 threads per unit, consecutive
// threads on consecutive blocks of one row: f(row, kb, row in tile, column in chunk, rec, hi) with
// rec = the unit's record and hi = address of E4M3 codes 8..15 of an FP8 block (codes 0..7 are in its
// slot), or nullptr if the block is NVFP4.
template <class F>
__device__ __forceinline__ void fgmp_for_each_block(const uint8_t* blob, const PackedLayout& L, int64_t unit,
                                                    UnitScratch& sc, F f)
{
    const int64_t tile = unit / L.chunks, c = unit % L.chunks;
    const uint32_t* mask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const uint32_t m16 = fgmp_chunk_mask(mask, L, tile * 128 + threadIdx.x, c);
    const uint32_t cnt = fgmp_unit_positions(m16, sc.warp, sc.pos, sc.cnt);
    const uint8_t* rec = blob + L.off_rec + (size_t)unit * REC_BYTES;
    const uint8_t* halves = blob + L.off_ovf + (size_t)reinterpret_cast<const uint32_t*>(blob + L.off_uptr)[unit] * 16 + fgmp_list_halves_offset(cnt);
    const int j = threadIdx.x & 15;
#pragma unroll 1
    for (int i = 0; i < 16; ++i) {
        const int row = (threadIdx.x >> 4) + 8 * i;
        const int64_t r = tile * 128 + row, kb = c * 16 + j;
        if (r >= L.rows || kb >= L.KB) continue;
        const uint32_t pos = sc.pos[row * 16 + j];
        f(r, kb, row, j, rec, pos != 0xffffu ? halves + (size_t)pos * 8 : (const uint8_t*)nullptr);
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
