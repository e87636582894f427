// The activation quantizer of one block spread over four lanes (Section 4.2: dynamic-max NVFP4
// scale, NVFP4 rounding, sensitivity-weighted error, FP8 iff the score exceeds the threshold).
// Every arithmetic step is the single-precision operation of the one-thread-per-block form in
// fgmp_common.cuh, in the same order, so codes, scales and scores agree with it bit for bit; the
// ordered sum of the sixteen error terms is handed from lane to lane.
#pragma once
#include "fgmp_common.cuh"
#include <cuda_fp16.h>

struct ActQuantScalars {
    float s4, k6, s8, inv8, tau, r8;     // NVFP4 tensor scale, 1/(6 s4), FP8 tensor scale and its inverse, threshold, 2^ratio
    int ratio;
};

struct BlockQuarter {
    uint32_t c4;        // this lane's four E2M1 codes (16 bits), zero if the block is FP8
    uint32_t c8;        // this lane's four E4M3 codes, valid if the block is FP8
    uint32_t sc;        // microscale code, zero if the block is FP8
    uint2 h;            // this lane's four values over the tensor scale, fp16 (exact)
    float score;
    bool is8;
};

// Lanes 4b .. 4b+3 of the warp hold block b: lane li = lane % 4 has elements 4 li .. 4 li + 3 (x: four
// bf16, f: their sensitivity weights).  All 32 lanes must call.
template <int MODE>
__device__ __forceinline__ BlockQuarter quantize_block_quarter(uint2 x, float4 f4, const ActQuantScalars& q)
{
    const uint32_t lane = threadIdx.x & 31u, li = lane & 3u, base = lane & ~3u;
    const float v[4] = {bf16lo_to_f32(x.x), bf16hi_to_f32(x.x), bf16lo_to_f32(x.y), bf16hi_to_f32(x.y)};
    const float f[4] = {f4.x, f4.y, f4.z, f4.w};
    float amax = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    BlockQuarter r;
    r.sc = f32x2_to_e4m3x2(__fmul_rn(amax, q.k6), 0.f) & 0x7f;
    const float ds = e4m3_to_f32(r.sc);
    const float d = __fmul_rn(ds, q.s4);
    const float inv = (d == 0.f) ? 0.f : __fdiv_rn(1.0f, d);
    const uint32_t b0 = f32x2_to_e2m1x2(__fmul_rn(v[0], inv), __fmul_rn(v[1], inv));
    const uint32_t b1 = f32x2_to_e2m1x2(__fmul_rn(v[2], inv), __fmul_rn(v[3], inv));
    r.c4 = b0 | (b1 << 8);
    const float2 q0 = e2m1x2_to_f32x2(b0), q1 = e2m1x2_to_f32x2(b1);
    const float qv[4] = {q0.x, q0.y, q1.x, q1.y};
    float dq4[4], dq8[4], e[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) dq4[i] = __fmul_rn(qv[i], d);
    float2 p0 = make_float2(0.f, 0.f), p1 = p0;          // E4M3 values of the FP8 form
    auto fp8_codes = [&]() {
        const uint32_t t0 = f32x2_to_e4m3x2(__fmul_rn(v[0], q.inv8), __fmul_rn(v[1], q.inv8));
        const uint32_t t1 = f32x2_to_e4m3x2(__fmul_rn(v[2], q.inv8), __fmul_rn(v[3], q.inv8));
        r.c8 = t0 | (t1 << 16);
        p0 = e4m3x2_to_f32x2(t0); p1 = e4m3x2_to_f32x2(t1);
    };
    r.c8 = 0;
    if (MODE == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = __fsub_rn(v[i], dq4[i]);
    } else {
        fp8_codes();
        dq8[0] = __fmul_rn(p0.x, q.s8); dq8[1] = __fmul_rn(p0.y, q.s8); dq8[2] = __fmul_rn(p1.x, q.s8); dq8[3] = __fmul_rn(p1.y, q.s8);
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = __fsub_rn(dq4[i], dq8[i]);
    }
    float t[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) t[i] = __fmul_rn(__fmul_rn(f[i], e[i]), e[i]);
    // sum over the sixteen elements in element order: lane 0 adds its four terms, hands the sum on, ...
    float s = 0.f;
#pragma unroll
    for (uint32_t L = 0; L < 4; ++L) {
        float u = s;
#pragma unroll
        for (int i = 0; i < 4; ++i) u = __fadd_rn(u, t[i]);
        if (li == L) s = u;
        s = __shfl_sync(0xffffffffu, s, (int)(base + L));
    }
    r.score = s;
    r.is8 = s > q.tau;
    if (r.is8) {
        if (MODE == 0) fp8_codes();
        const __half2 h0 = __floats2half2_rn(p0.x * q.r8, p0.y * q.r8), h1 = __floats2half2_rn(p1.x * q.r8, p1.y * q.r8);
        r.h = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
        r.c4 = 0; r.sc = 0;
    } else {
        const __half2 h0 = __floats2half2_rn(q0.x * ds, q0.y * ds), h1 = __floats2half2_rn(q1.x * ds, q1.y * ds);
        r.h = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
    }
    return r;
}
