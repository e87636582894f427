// Online activation quantizer (Section 4.2 of the paper), block scores, and the
// packed -> canonical unpacker.
//
// Thread mapping: one thread owns one 16-element block column (kb) and walks down the rows
// of its CTA, so the 16 per-channel Fisher weights stay in registers.  A warp covers 32
// consecutive blocks of one row = one mask word, produced with a ballot.
#include "fgmp_common.cuh"
#include "fgmp_host.h"
#include <cuda_bf16.h>

namespace {

constexpr int QA_THREADS = 256;

struct ActParams {
    const uint4* X; int64_t ldx8;        // row stride in 16-byte units
    const float* fisher;
    int64_t M, K, KB, MW;
    float s4, k6, s8, inv8, tau;
    uint8_t* codes4; uint8_t* sf; uint32_t* mask; uint8_t* codes8;   // codes8: dense plane
    float* scores;                       // optional (score-only kernel)
    uint8_t* arec;                       // optional per-chunk records for the decode GEMM (M <= 16)
    fgmp_packed_header* header;
    float r8;                            // 2^ratio
    int ratio;
    int free8;                           // the FP8 tensor scale was given on its own
    int rows_per_cta;
};

template <int MODE, bool SCORE_ONLY>
__global__ void __launch_bounds__(QA_THREADS) quant_act_kernel(ActParams p)
{
    // A kernel launched behind this one as a programmatic dependent (the decode-sized GEMM) may
    // start setting itself up now; it waits for this grid to complete before it reads the result.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t kb = (int64_t)blockIdx.x * QA_THREADS + threadIdx.x;
    const bool active = kb < p.KB;
    const int64_t m0 = (int64_t)blockIdx.y * p.rows_per_cta;
    const int64_t m1 = min(m0 + (int64_t)p.rows_per_cta, p.M);
    if (!SCORE_ONLY) {
        if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
            fgmp_packed_header* h = p.header;
            h->magic = FGMP_MAGIC; h->version = 7; h->rows = p.M; h->K = p.K; h->scale_fp4 = p.s4;
            h->fp8_log2_ratio = p.ratio; h->n_fp8 = (p.tau == INFINITY) ? 0 : -1; h->tau_eff = 0.f; h->kind = 0; h->capacity = 0;
            h->error = 0; h->scale_fp8 = p.s8; h->fp8_scale_free = p.free8;
        }
        // token rows M..15 of the decode records are zero (the grid covers 16 rows in that mode)
        if (p.arec && m0 >= p.M) {
            if (active) {
                uint8_t* rec = p.arec + (size_t)(kb >> 4) * AREC_BYTES;
                const uint32_t j = (uint32_t)kb & 15u, m = (uint32_t)m0;
                *reinterpret_cast<uint2*>(rec + AREC_A4 + fgmp_rec_w4_offset(m, j)) = make_uint2(0u, 0u);
                rec[AREC_SF + m * 16 + j] = 0;
                uint4* at = reinterpret_cast<uint4*>(rec + fgmp_arec_at_offset(m, j));
                at[0] = make_uint4(0, 0, 0, 0); at[1] = make_uint4(0, 0, 0, 0);
            }
            return;
        }
    }

    float f[16];
    if (active) {
        const float4* fp = reinterpret_cast<const float4*>(p.fisher + kb * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 t = __ldg(fp + i);
            f[4 * i] = t.x; f[4 * i + 1] = t.y; f[4 * i + 2] = t.z; f[4 * i + 3] = t.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) f[i] = 0.f;
    }

    for (int64_t m = m0; m < m1; ++m) {
        bool is8 = false;
        if (active) {
            const uint4* xp = p.X + m * p.ldx8 + kb * 2;
            uint4 xa = __ldcs(xp), xb = __ldcs(xp + 1);
            float v[16], dq4[16];
            unpack_bf16x16(xa, xb, v);
            uint32_t sc = block_dynamic_scale(v, p.k6);
            uint32_t c4[2];
            block_nvfp4(v, sc, p.s4, c4, dq4);
            float score;
            uint32_t c8[4];
            if (MODE == 0) {
                score = weighted_sq_sum(v, dq4, f);
            } else {
                float dq8[16];
                block_fp8(v, p.inv8, p.s8, c8, dq8);
                score = weighted_sq_sum(dq4, dq8, f);
            }
            if (SCORE_ONLY) {
                p.scores[m * p.KB + kb] = score;
            } else {
                is8 = score > p.tau;
                if (is8) {
                    if (MODE == 0) {
                        float dq8[16];
                        block_fp8(v, p.inv8, p.s8, c8, dq8);
                    }
                    *reinterpret_cast<uint4*>(p.codes8 + m * p.K + kb * 16) = make_uint4(c8[0], c8[1], c8[2], c8[3]);
                    c4[0] = 0; c4[1] = 0; sc = 0;
                }
                if (p.arec) {
                    // value / tensor scale, exact in fp16: E2M1 x microscale or E4M3 x 2^ratio
                    uint32_t o[8];
                    if (is8) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float2 a = e4m3x2_to_f32x2(c8[i] & 0xffff), b = e4m3x2_to_f32x2(c8[i] >> 16);
                            __half2 h0 = __floats2half2_rn(a.x * p.r8, a.y * p.r8), h1 = __floats2half2_rn(b.x * p.r8, b.y * p.r8);
                            o[2 * i] = *reinterpret_cast<uint32_t*>(&h0); o[2 * i + 1] = *reinterpret_cast<uint32_t*>(&h1);
                        }
                    } else {
                        const float d = e4m3_to_f32(sc);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float2 q = e2m1x2_to_f32x2((c4[i >> 2] >> ((i & 3) * 8)) & 0xff);
                            __half2 h = __floats2half2_rn(q.x * d, q.y * d);
                            o[i] = *reinterpret_cast<uint32_t*>(&h);
                        }
                    }
                    uint8_t* rec = p.arec + (size_t)(kb >> 4) * AREC_BYTES;
                    const uint32_t j = (uint32_t)kb & 15u;
                    uint4* at = reinterpret_cast<uint4*>(rec + fgmp_arec_at_offset((uint32_t)m, j));
                    at[0] = make_uint4(o[0], o[1], o[2], o[3]);
                    at[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    // what the tensor core reads: codes and microscale (both zero for an FP8 block), and the
                    // chunk's set of block columns that hold an FP8 block of some token
                    *reinterpret_cast<uint2*>(rec + AREC_A4 + fgmp_rec_w4_offset((uint32_t)m, j)) = make_uint2(c4[0], c4[1]);
                    rec[AREC_SF + (uint32_t)m * 16 + j] = (uint8_t)sc;
                    if (is8) atomicOr(reinterpret_cast<unsigned int*>(rec + AREC_HOT), 1u << j);
                }
                *reinterpret_cast<uint2*>(p.codes4 + (m * p.K) / 2 + kb * 8) = make_uint2(c4[0], c4[1]);
                p.sf[fgmp_sf_offset(m, kb, p.K)] = (uint8_t)sc;
            }
        }
        if (!SCORE_ONLY) {
            uint32_t word = __ballot_sync(0xffffffffu, is8);
            int64_t w = kb >> 5;
            if ((threadIdx.x & 31) == 0 && w < p.MW) {
                p.mask[m * p.MW + w] = word;
            }
        }
    }
}

// packed activations -> canonical arrays; one thread per block
__global__ void unpack_kernel(const uint8_t* blob, int64_t rows, int64_t K,
                              uint8_t* codes4, uint8_t* codes8, uint8_t* scales, uint32_t* mask)
{
    const PackedLayout L = fgmp_layout(rows, K, 0, 0);
    const uint32_t* pmask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const int64_t nblk = rows * L.KB;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblk; b += (int64_t)gridDim.x * blockDim.x) {
        int64_t r = b / L.KB, kb = b % L.KB;
        uint32_t word = pmask[r * L.MW + (kb >> 5)];
        bool is8 = (word >> (kb & 31)) & 1;
        if (mask && (kb & 31) == 0) mask[r * L.MW + (kb >> 5)] = word;
        if (scales) scales[b] = blob[L.off_sf + fgmp_sf_offset(r, kb, K)];
        if (codes4) {
            uint2 c = *reinterpret_cast<const uint2*>(blob + L.off_codes4 + (r * K) / 2 + kb * 8);
            *reinterpret_cast<uint2*>(codes4 + (r * K) / 2 + kb * 8) = c;
        }
        if (codes8) {
            uint4 c = make_uint4(0, 0, 0, 0);
            if (is8) c = *reinterpret_cast<const uint4*>(blob + L.off_codes8 + (size_t)(r * K + kb * 16));
            *reinterpret_cast<uint4*>(codes8 + r * K + kb * 16) = c;
        }
    }
}

// packed weights -> canonical arrays; one CTA of 128 threads per unit record
__global__ void __launch_bounds__(128) unpack_w_kernel(const uint8_t* blob, int64_t rows, int64_t K,
                                                       uint8_t* codes4, uint8_t* codes8, uint8_t* scales, uint32_t* mask)
{
    __shared__ UnitScratch sc;
    const PackedLayout L = fgmp_layout(rows, K, 1, 0);
    if (mask) {
        const uint32_t* pmask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
        for (int64_t i = (int64_t)blockIdx.x * 128 + threadIdx.x; i < rows * L.MW; i += (int64_t)gridDim.x * 128) mask[i] = pmask[i];
    }
    fgmp_for_each_block(blob, L, blockIdx.x, sc, [&](int64_t r, int64_t kb, int row, int j, const uint8_t* rec, const uint8_t* hi) {
        const uint2 slot = *reinterpret_cast<const uint2*>(rec + REC_W4 + fgmp_rec_w4_offset(row, j));
        if (scales) scales[r * L.KB + kb] = rec[REC_SF + fgmp_rec_sf_offset(row, j)];
        if (codes4) *reinterpret_cast<uint2*>(codes4 + (r * K) / 2 + kb * 8) = hi ? make_uint2(0u, 0u) : slot;
        if (codes8) {
            uint4 c = make_uint4(0, 0, 0, 0);
            if (hi) { const uint2 h = *reinterpret_cast<const uint2*>(hi); c = make_uint4(slot.x, slot.y, h.x, h.y); }
            *reinterpret_cast<uint4*>(codes8 + r * K + kb * 16) = c;
        }
    });
}

// mean of squares per column of a bf16 matrix; thread per column, rows in order (one fp32 multiply
// and one fp32 add per element, then one division): reproducible bit for bit
__global__ void channel_mean_sq_kernel(const __nv_bfloat16* X, int64_t ld, int64_t rows, int64_t K, float* out)
{
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= K) return;
    float s = 0.f;
    for (int64_t r = 0; r < rows; ++r) {
        const float v = __bfloat162float(X[r * ld + c]);
        s = __fadd_rn(s, __fmul_rn(v, v));
    }
    out[c] = __fdiv_rn(s, (float)rows);
}

fgmp_status check_act_args(const void* X, int64_t ldx, const float* fisher, int64_t M, int64_t K, fgmp_scales sc, int sm)
{
    if (!X || !fisher) return FGMP_ERR_INVALID_ARG;
    if (sm != 0 && sm != 1) return FGMP_ERR_INVALID_ARG;
    if (!(sc.scale_fp4 > 0.f) || !isfinite(sc.scale_fp4)) return FGMP_ERR_INVALID_ARG;
    if (!fgmp_scales_valid(sc)) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || K < 64 || (K % 64) != 0 || ldx < K || (ldx % 8) != 0) return FGMP_ERR_SHAPE;
    if (((uintptr_t)X & 15) || ((uintptr_t)fisher & 15)) return FGMP_ERR_SHAPE;
    return FGMP_OK;
}

ActParams make_act_params(const void* X, int64_t ldx, const float* fisher, int64_t M, int64_t K, fgmp_scales sc, float tau)
{
    ActParams p{};
    p.X = reinterpret_cast<const uint4*>(X); p.ldx8 = ldx / 8; p.fisher = fisher;
    p.M = M; p.K = K; p.KB = K / 16; p.MW = (p.KB + 31) / 32;
    p.s4 = sc.scale_fp4;
    p.k6 = 1.0f / (6.0f * sc.scale_fp4);
    p.s8 = fgmp_fp8_scale(sc);
    p.inv8 = 1.0f / p.s8;
    p.free8 = fgmp_fp8_free(sc) ? 1 : 0;
    p.tau = tau;
    p.ratio = sc.fp8_log2_ratio;
    p.r8 = ldexpf(1.0f, sc.fp8_log2_ratio);
    // enough CTAs to fill the machine when M is small, few row-loop iterations otherwise
    p.rows_per_cta = (M >= 2048) ? 8 : (M >= 256 ? 4 : 1);
    return p;
}

}  // namespace

extern "C" fgmp_status fgmp_quantize_activations(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                                 int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm, float tau,
                                                 void* packed_out, size_t packed_bytes,
                                                 void* workspace, size_t ws_bytes, void* cuda_stream)
{
    (void)workspace; (void)ws_bytes;
    fgmp_status st = check_act_args(X_bf16, ldx, fisher_chan, M, K, sc, (int)sm);
    if (st != FGMP_OK) return st;
    if (!packed_out || ((uintptr_t)packed_out & 1023)) return packed_out ? FGMP_ERR_SHAPE : FGMP_ERR_INVALID_ARG;
    if (tau != tau) return FGMP_ERR_INVALID_ARG;
    const PackedLayout L = fgmp_layout(M, K, 0, 0);
    if (packed_bytes < L.total) return FGMP_ERR_WORKSPACE;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint8_t* blob = (uint8_t*)packed_out;

    ActParams p = make_act_params(X_bf16, ldx, fisher_chan, M, K, sc, tau);
    p.codes4 = blob + L.off_codes4; p.sf = blob + L.off_sf;
    p.mask = reinterpret_cast<uint32_t*>(blob + L.off_mask); p.codes8 = blob + L.off_codes8;
    p.header = reinterpret_cast<fgmp_packed_header*>(blob);
    int64_t grid_rows = M;
    if (M <= 16 && !p.free8) {         // decode-sized batch: also emit the records of the decode GEMM, 16 token rows (tied scales only)
        p.arec = blob + L.off_arec;
        p.rows_per_cta = 1;
        grid_rows = 16;
        // the sets of hot block columns are OR-ed together by the kernel's threads
        if (cudaMemset2DAsync(blob + L.off_arec + AREC_HOT, AREC_BYTES, 0, 16, (size_t)L.chunks, s) != cudaSuccess) return FGMP_ERR_CUDA;
    }
    dim3 grid((unsigned)((p.KB + QA_THREADS - 1) / QA_THREADS), (unsigned)((grid_rows + p.rows_per_cta - 1) / p.rows_per_cta));
    if (sm == FGMP_SCORE_LP_ERROR) FGMP_LAUNCH(FGMP_K_ACT_QUANT, s, quant_act_kernel<0, false><<<grid, QA_THREADS, 0, s>>>(p));
    else                           FGMP_LAUNCH(FGMP_K_ACT_QUANT, s, quant_act_kernel<1, false><<<grid, QA_THREADS, 0, s>>>(p));
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_activation_scores(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                              int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                                              float* scores, void* cuda_stream)
{
    fgmp_status st = check_act_args(X_bf16, ldx, fisher_chan, M, K, sc, (int)sm);
    if (st != FGMP_OK) return st;
    if (!scores) return FGMP_ERR_INVALID_ARG;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    ActParams p = make_act_params(X_bf16, ldx, fisher_chan, M, K, sc, 0.f);
    p.scores = scores;
    dim3 grid((unsigned)((p.KB + QA_THREADS - 1) / QA_THREADS), (unsigned)((M + p.rows_per_cta - 1) / p.rows_per_cta));
    if (sm == FGMP_SCORE_LP_ERROR) FGMP_LAUNCH(FGMP_K_ACT_SCORES, s, quant_act_kernel<0, true><<<grid, QA_THREADS, 0, s>>>(p));
    else                           FGMP_LAUNCH(FGMP_K_ACT_SCORES, s, quant_act_kernel<1, true><<<grid, QA_THREADS, 0, s>>>(p));
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_unpack(const void* packed, int64_t rows, int64_t K, uint8_t* codes4, uint8_t* codes8,
                                   uint8_t* scales, uint32_t* mask, void* cuda_stream)
{
    if (!packed) return FGMP_ERR_INVALID_ARG;
    if (rows < 1 || K < 64 || (K % 64) != 0 || ((uintptr_t)packed & 1023)) return FGMP_ERR_SHAPE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the blob says what it is: activations keep planes, weights keep unit records
    fgmp_packed_header h;
    if (cudaMemcpyAsync(&h, packed, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) return FGMP_ERR_CUDA;
    if (h.magic != FGMP_MAGIC || h.rows != rows || h.K != K || h.error != 0) return FGMP_ERR_INVALID_ARG;
    if (h.kind == 1) {
        const PackedLayout L = fgmp_layout(rows, K, 1, 0);
        FGMP_LAUNCH(FGMP_K_UNPACK, s, unpack_w_kernel<<<(unsigned)L.units, 128, 0, s>>>((const uint8_t*)packed, rows, K, codes4, codes8, scales, mask));
    } else {
        int64_t nblk = rows * (K / 16);
        int grid = (int)((nblk + 255) / 256 < 148 * 16 ? (nblk + 255) / 256 : 148 * 16);
        FGMP_LAUNCH(FGMP_K_UNPACK, s, unpack_kernel<<<grid, 256, 0, s>>>((const uint8_t*)packed, rows, K, codes4, codes8, scales, mask));
    }
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_channel_mean_sq(const void* X_bf16, int64_t ldx, int64_t rows, int64_t K,
                                            float* mean_sq, void* cuda_stream)
{
    if (!X_bf16 || !mean_sq) return FGMP_ERR_INVALID_ARG;
    if (rows < 1 || rows > ((int64_t)1 << 24) || K < 1 || ldx < K) return FGMP_ERR_SHAPE;
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    FGMP_LAUNCH(FGMP_K_ACT_AUX, s, channel_mean_sq_kernel<<<(unsigned)((K + 127) / 128), 128, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(X_bf16), ldx, rows, K, mean_sq));
    return fgmp_launch_status();
}
