// Offline weight packer: tensor scale, sensitivity-weighted clip search (Eq. 11), block
// scores (Eq. 6 / Eq. 8), exact top-R selection (Eq. 9) and emission of the packed blob.
// Also the activation-threshold calibration (Eq. 9 applied to a calibration batch), which
// reuses the selection kernels.
#include "fgmp_common.cuh"
#include "fgmp_host.h"

namespace {

// Device-resident state of one packing call (lives at the start of the workspace).
struct SelectState {
    uint32_t hist[256];
    uint32_t amax_bits;      // max |w| as fp32 bits
    float s4;                // NVFP4 tensor scale in use
    uint32_t prefix;         // radix-select prefix (high bits of the k-th largest score)
    uint32_t pad0;
    unsigned long long krem; // how many blocks are still to be taken inside the prefix group
    float tau;               // threshold: FP8 iff score > tau, or == tau within the first need_eq
    uint32_t use_eq;
    unsigned long long need_eq;
    unsigned long long n_fp8;
    float next_below;        // calibration: largest score strictly below tau
    uint32_t pad1;
};

constexpr size_t STATE_BYTES = 2048;

__global__ void state_init_kernel(SelectState* st, float s4_given, unsigned long long k)
{
    int t = threadIdx.x;
    if (t < 256) st->hist[t] = 0;
    if (t == 0) {
        st->amax_bits = 0; st->s4 = s4_given; st->prefix = 0; st->krem = k; st->tau = 0.f;
        st->use_eq = 0; st->need_eq = 0; st->n_fp8 = 0; st->next_below = 0.f;
    }
}

__global__ void w_amax_kernel(const uint4* W, int64_t ldw8, int64_t N, int64_t K8, SelectState* st)
{
    uint32_t m = 0;
    const int64_t total = N * K8;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / K8, c = i % K8;
        uint4 x = __ldg(W + n * ldw8 + c);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            m = max(m, (w[j] << 16) & 0x7fffffffu);
            m = max(m, w[j] & 0x7fff0000u);
        }
    }
    for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(&st->amax_bits, m);
}

__global__ void w_scale_kernel(SelectState* st)
{
    if (threadIdx.x == 0) st->s4 = __fdiv_rn(__uint_as_float(st->amax_bits), 2688.0f);
}

__device__ __forceinline__ void load_block(const uint4* W, int64_t ldw8, const float* F, int64_t ldf,
                                           int64_t n, int64_t kb, float (&v)[16], float (&f)[16])
{
    const uint4* wp = W + n * ldw8 + kb * 2;
    unpack_bf16x16(__ldg(wp), __ldg(wp + 1), v);
    if (F) {
        const float4* fp = reinterpret_cast<const float4*>(F + n * ldf + kb * 16);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 t = __ldg(fp + i);
            f[4 * i] = t.x; f[4 * i + 1] = t.y; f[4 * i + 2] = t.z; f[4 * i + 3] = t.w;
        }
    }
}

// per block: microscale (dynamic max or Eq. 11 brute force) and the score under it
template <int MODE, bool CLIP>
__global__ void __launch_bounds__(256) w_score_kernel(const uint4* W, int64_t ldw8, const float* F, int64_t ldf,
                                                      int64_t N, int64_t KB, int ratio, float s8_given, const SelectState* st,
                                                      uint8_t* sc_out, float* scores)
{
    __shared__ float s_d[128], s_inv[128];
    const float s4 = st->s4;
    if (CLIP) {
        if (threadIdx.x < 127) {
            float d = __fmul_rn(e4m3_to_f32(threadIdx.x), s4);
            s_d[threadIdx.x] = d;
            s_inv[threadIdx.x] = (d == 0.f) ? 0.f : __fdiv_rn(1.0f, d);
        }
        __syncthreads();
    }
    const float k6 = __fdiv_rn(1.0f, __fmul_rn(6.0f, s4));
    const float s8 = s8_given > 0.f ? s8_given : __fmul_rn(s4, __int_as_float((127 + ratio) << 23));
    const float inv8 = __fdiv_rn(1.0f, s8);
    const int64_t B = N * KB;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < B; b += (int64_t)gridDim.x * blockDim.x) {
        float v[16], f[16];
        load_block(W, ldw8, F, ldf, b / KB, b % KB, v, f);
        uint32_t sc = block_dynamic_scale(v, k6);
        if (CLIP) {
            // incumbent = dynamic max; ascending scan, strict improvement only
            float best;
            {
                float d = s_d[sc], inv = s_inv[sc];
                best = 0.f;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float2 q = e2m1x2_to_f32x2(f32x2_to_e2m1x2(__fmul_rn(v[i], inv), __fmul_rn(v[i + 1], inv)));
                    float e0 = __fsub_rn(__fmul_rn(q.x, d), v[i]);
                    best = __fadd_rn(best, __fmul_rn(__fmul_rn(f[i], e0), e0));
                    float e1 = __fsub_rn(__fmul_rn(q.y, d), v[i + 1]);
                    best = __fadd_rn(best, __fmul_rn(__fmul_rn(f[i + 1], e1), e1));
                }
            }
            for (uint32_t c = 1; c <= 0x7e; ++c) {
                float d = s_d[c], inv = s_inv[c];
                float j = 0.f;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    float2 q = e2m1x2_to_f32x2(f32x2_to_e2m1x2(__fmul_rn(v[i], inv), __fmul_rn(v[i + 1], inv)));
                    float e0 = __fsub_rn(__fmul_rn(q.x, d), v[i]);
                    j = __fadd_rn(j, __fmul_rn(__fmul_rn(f[i], e0), e0));
                    float e1 = __fsub_rn(__fmul_rn(q.y, d), v[i + 1]);
                    j = __fadd_rn(j, __fmul_rn(__fmul_rn(f[i + 1], e1), e1));
                }
                if (j < best) { best = j; sc = c; }
            }
        }
        uint32_t c4[2];
        float dq4[16];
        block_nvfp4(v, sc, s4, c4, dq4);
        float score;
        if (MODE == 0) {
            score = weighted_sq_sum(v, dq4, f);
        } else {
            uint32_t c8[4];
            float dq8[16];
            block_fp8(v, inv8, s8, c8, dq8);
            score = weighted_sq_sum(dq4, dq8, f);
        }
        sc_out[b] = (uint8_t)sc;
        scores[b] = score;
    }
}

// ------------------------------------------------------------ radix select (k-th largest)
// Scores are >= 0, so their fp32 bit patterns order like unsigned integers.
__global__ void select_hist_kernel(const float* scores, int64_t B, int pass, SelectState* st)
{
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int shift = 24 - 8 * pass;
    const uint32_t prefix = st->prefix;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < B; b += (int64_t)gridDim.x * blockDim.x) {
        uint32_t u = __float_as_uint(scores[b]);
        if (pass == 0 || (u >> (shift + 8)) == prefix) atomicAdd(&h[(u >> shift) & 255], 1u);
    }
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], h[threadIdx.x]);
}

__global__ void select_pick_kernel(SelectState* st, int pass)
{
    if (threadIdx.x == 0) {
        unsigned long long krem = st->krem, cum = 0;
        int bin = 255;
        for (; bin > 0; --bin) {
            if (cum + st->hist[bin] >= krem) break;
            cum += st->hist[bin];
        }
        st->prefix = (st->prefix << 8) | (uint32_t)bin;
        st->krem = krem - cum;
        if (pass == 3) {
            st->tau = __uint_as_float(st->prefix);
            st->need_eq = st->krem;          // of the blocks equal to tau, take this many
            st->use_eq = 1;
        }
    }
    __syncthreads();
    if (threadIdx.x < 256) st->hist[threadIdx.x] = 0;
}

// largest score strictly below tau (calibration: the (k+1)-th largest when there are no ties)
__global__ void next_below_kernel(const float* scores, int64_t B, SelectState* st)
{
    const float tau = st->tau;
    uint32_t m = 0;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < B; b += (int64_t)gridDim.x * blockDim.x) {
        float s = scores[b];
        if (s < tau) m = max(m, __float_as_uint(s));
    }
    for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) atomicMax(reinterpret_cast<uint32_t*>(&st->next_below), m);
}

__global__ void calib_finish_kernel(const SelectState* st, float* tau_out, int all_or_none)
{
    if (threadIdx.x == 0) {
        if (all_or_none == 1) *tau_out = __int_as_float(0x7f800000);   // k = 0: nothing exceeds +inf
        else if (all_or_none == 2) *tau_out = -1.0f;                   // k = all
        else {
            // midway between the k-th largest score and the next one below it; if fp32 cannot
            // separate them, the lower neighbour itself (score > tau still selects the top k)
            float t = __fmul_rn(0.5f, __fadd_rn(st->tau, st->next_below));
            *tau_out = (t < st->tau && t >= st->next_below) ? t : st->next_below;
        }
    }
}

// ------------------------------------------------------------ mask, prefix sums, emission
// per mask word: how many of its blocks have score == tau
__global__ void w_eqcount_kernel(const float* scores, int64_t N, int64_t KB, int64_t MW, const SelectState* st, uint32_t* cnt)
{
    const float tau = st->tau;
    const int lane = threadIdx.x & 31;
    const int64_t nw = N * MW;
    for (int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < nw; w += ((int64_t)gridDim.x * blockDim.x) >> 5) {
        int64_t n = w / MW, kb = (w % MW) * 32 + lane;
        bool eq = kb < KB && scores[n * KB + kb] == tau;
        uint32_t bal = __ballot_sync(0xffffffffu, eq);
        if (lane == 0) cnt[w] = __popc(bal);
    }
}

__global__ void w_mask_kernel(const float* scores, int64_t N, int64_t KB, int64_t MW, const SelectState* st,
                              const uint32_t* eqprefix, uint32_t* mask, uint32_t* wcnt)
{
    const float tau = st->tau;
    const bool use_eq = st->use_eq != 0;
    const unsigned long long need_eq = st->need_eq;
    const int lane = threadIdx.x & 31;
    const int64_t nw = N * MW;
    for (int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < nw; w += ((int64_t)gridDim.x * blockDim.x) >> 5) {
        int64_t n = w / MW, kb = (w % MW) * 32 + lane;
        float s = kb < KB ? scores[n * KB + kb] : -1.f;
        bool gt = kb < KB && s > tau;
        bool eq = use_eq && kb < KB && s == tau;
        uint32_t eqbal = __ballot_sync(0xffffffffu, eq);
        bool take = gt;
        if (eq) {
            unsigned long long rank = (unsigned long long)eqprefix[w] + __popc(eqbal & ((1u << lane) - 1u));
            take = rank < need_eq;
        }
        uint32_t word = __ballot_sync(0xffffffffu, take);
        if (lane == 0) { mask[w] = word; wcnt[w] = __popc(word); }
    }
}

// exclusive prefix sum of n uint32 by one CTA of 1024 threads; total -> *total_out (may be NULL)
__global__ void __launch_bounds__(1024) scan_kernel(const uint32_t* in, uint32_t* out, int64_t n, unsigned long long* total_out,
                                                    int append_total)
{
    __shared__ uint32_t warp_sums[32];
    __shared__ unsigned long long carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int64_t base = 0; base < n; base += 1024) {
        int64_t i = base + threadIdx.x;
        uint32_t x = i < n ? in[i] : 0;
        uint32_t incl = x;
        for (int o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        if (lane == 31) warp_sums[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            uint32_t s = warp_sums[lane], si = s;
            for (int o = 1; o < 32; o <<= 1) { uint32_t y = __shfl_up_sync(0xffffffffu, si, o); if (lane >= o) si += y; }
            warp_sums[lane] = si - s;       // exclusive warp offsets
        }
        __syncthreads();
        unsigned long long carry = carry_s;
        if (i < n) out[i] = (uint32_t)(carry + warp_sums[wid] + incl - x);
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_sums[31] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0 && total_out) *total_out = carry_s;
    if (threadIdx.x == 0 && append_total) out[n] = (uint32_t)carry_s;
}

// per unit (128-row tile x 16-block K chunk): size of its list of FP8 blocks in 16-byte steps, and the
// running total of FP8 blocks.  One CTA of 128 threads per unit, a thread per row.
__global__ void __launch_bounds__(128) w_unit_count_kernel(const uint32_t* mask, PackedLayout L, uint32_t* list_steps,
                                                           SelectState* st)
{
    __shared__ uint32_t s_cnt[4];
    const int64_t unit = blockIdx.x;
    const uint32_t m16 = fgmp_chunk_mask(mask, L, (unit / L.chunks) * 128 + threadIdx.x, unit % L.chunks);
    uint32_t c = __popc(m16);
    for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0) s_cnt[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t cnt = s_cnt[0] + s_cnt[1] + s_cnt[2] + s_cnt[3];
        list_steps[unit] = fgmp_list_steps(cnt);
        atomicAdd(&st->n_fp8, (unsigned long long)cnt);
    }
}

// Writes the record of one unit (codes and microscales of its NVFP4 blocks, the first halves of its FP8
// blocks, the per-column running counts) and the list of its FP8 blocks (rows, second halves).  One CTA
// of 128 threads per unit.
__global__ void __launch_bounds__(128) w_emit_kernel(const uint4* W, int64_t ldw8, int ratio, float s8_given, const SelectState* st,
                                                     const uint8_t* sc_in, uint8_t* blob, PackedLayout L, int64_t room_steps)
{
    __shared__ UnitScratch sc;
    const int64_t unit = blockIdx.x, tile = unit / L.chunks, c = unit % L.chunks;
    const uint32_t* uptr = reinterpret_cast<const uint32_t*>(blob + L.off_uptr);
    const bool fits = (int64_t)uptr[unit + 1] <= room_steps;   // else the blob is too small: header.error says so
    const float s4 = st->s4;
    const float s8 = s8_given > 0.f ? s8_given : __fmul_rn(s4, __int_as_float((127 + ratio) << 23));
    const float inv8 = __fdiv_rn(1.0f, s8);
    const uint32_t* mask = reinterpret_cast<const uint32_t*>(blob + L.off_mask);
    const uint32_t m16 = fgmp_chunk_mask(mask, L, tile * 128 + threadIdx.x, c);
    const uint32_t cnt = fgmp_unit_positions(m16, sc.warp, sc.pos, sc.cnt);
    uint8_t* rec = blob + L.off_rec + (size_t)unit * REC_BYTES;
    uint8_t* list = blob + L.off_ovf + (size_t)uptr[unit] * 16;
    uint32_t* entries = reinterpret_cast<uint32_t*>(list);
    uint8_t* halves = list + fgmp_list_halves_offset(cnt);
    if (threadIdx.x < 64) {                                    // running sums of the per-column counts, then padding
        uint32_t before = 0;
        for (int i = 0; i < 16 && i < (int)threadIdx.x; ++i) before += sc.cnt[i];
        reinterpret_cast<uint16_t*>(rec + REC_KBSTART)[threadIdx.x] = threadIdx.x <= 16 ? (uint16_t)before : (uint16_t)0;
    }
    if (fits) {                                                // padding behind the entries and behind the last half
        for (uint32_t i = cnt + threadIdx.x; i < fgmp_list_halves_offset(cnt) / 4; i += 128) entries[i] = 0;
        if (threadIdx.x == 0 && (cnt & 1u)) *reinterpret_cast<uint2*>(halves + (size_t)cnt * 8) = make_uint2(0u, 0u);
    }
    const int j = threadIdx.x & 15;
#pragma unroll 1
    for (int i = 0; i < 16; ++i) {
        const int row = (threadIdx.x >> 4) + 8 * i;
        const int64_t n = tile * 128 + row, kb = c * 16 + j;
        uint2 slot = make_uint2(0u, 0u);
        uint32_t scale = 0;
        if (n < L.rows && kb < L.KB) {
            float v[16], f[16];
            load_block(W, ldw8, nullptr, 0, n, kb, v, f);
            const uint32_t pos = sc.pos[row * 16 + j];
            if (pos != 0xffffu) {
                uint32_t c8[4];
                float dq8[16];
                block_fp8(v, inv8, s8, c8, dq8);
                slot = make_uint2(c8[0], c8[1]);
                if (fits) {
                    *reinterpret_cast<uint2*>(halves + (size_t)pos * 8) = make_uint2(c8[2], c8[3]);
                    entries[pos] = fgmp_list_entry((uint32_t)row, (uint32_t)j);
                }
            } else {
                float dq4[16];
                uint32_t c4[2];
                scale = sc_in[n * L.KB + kb];
                block_nvfp4(v, scale, s4, c4, dq4);
                slot = make_uint2(c4[0], c4[1]);
            }
        }
        *reinterpret_cast<uint2*>(rec + REC_W4 + fgmp_rec_w4_offset(row, j)) = slot;
        rec[REC_SF + fgmp_rec_sf_offset(row, j)] = (uint8_t)scale;
    }
}

// With too little room the starts of the overflow entries are pulled back inside the blob, so that a
// reader that follows them stays within the allocation (the entries themselves were not written).
__global__ void w_clamp_uptr_kernel(const fgmp_packed_header* h, uint32_t* uptr, int64_t n, int64_t room_steps)
{
    if (h->error == 0) return;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        if ((int64_t)uptr[i] > room_steps) uptr[i] = (uint32_t)room_steps;
}

__global__ void w_header_kernel(fgmp_packed_header* h, const SelectState* st, const uint32_t* uptr, int64_t units,
                                int64_t N, int64_t K, int ratio, float s8_given, int64_t room_steps, int fraction_mode, float tau_given,
                                float* tau_eff_out)
{
    if (threadIdx.x == 0) {
        h->magic = FGMP_MAGIC; h->version = 7; h->rows = N; h->K = K; h->scale_fp4 = st->s4;
        h->fp8_log2_ratio = ratio; h->n_fp8 = (int64_t)st->n_fp8; h->kind = 1; h->capacity = room_steps;
        float teff = fraction_mode ? st->tau : tau_given;
        h->tau_eff = teff;
        h->error = ((int64_t)uptr[units] > room_steps) ? (int32_t)FGMP_ERR_CAPACITY : 0;
        h->scale_fp8 = s8_given > 0.f ? s8_given : __fmul_rn(st->s4, __int_as_float((127 + ratio) << 23));
        h->fp8_scale_free = s8_given > 0.f ? 1 : 0;
        if (tau_eff_out) *tau_eff_out = teff;
    }
}

__global__ void set_tau_kernel(SelectState* st, float tau)
{
    if (threadIdx.x == 0) { st->tau = tau; st->use_eq = 0; st->need_eq = 0; }
}

int grid_for(int64_t work_items, int threads, int max_ctas_per_sm)
{
    int64_t g = (work_items + threads - 1) / threads;
    int64_t cap = (int64_t)fgmp_sm_count() * max_ctas_per_sm;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// runs the 4-pass radix select for the k-th largest of scores[0..B)
void run_select(const float* scores, int64_t B, SelectState* st, cudaStream_t s)
{
    int g = grid_for(B, 256, 8);
    for (int pass = 0; pass < 4; ++pass) {
        FGMP_LAUNCH(FGMP_K_SELECT, s, select_hist_kernel<<<g, 256, 0, s>>>(scores, B, pass, st));
        FGMP_LAUNCH(FGMP_K_SELECT, s, select_pick_kernel<<<1, 256, 0, s>>>(st, pass));
    }
}

// words in each of the two scratch arrays: one per mask word, or one per (tile, chunk) + 1
int64_t tmp_words(int64_t N, int64_t K)
{
    int64_t KB = K / 16, MW = (KB + 31) / 32;
    int64_t nct = ((N + 127) / 128) * ((KB + 15) / 16) + 1;
    return N * MW > nct ? N * MW : nct;
}

size_t ws_weights_bytes(int64_t N, int64_t K)
{
    int64_t KB = K / 16, B = N * KB;
    return STATE_BYTES + fgmp_align1k((size_t)B * 4) + fgmp_align1k((size_t)B) + 2 * fgmp_align1k((size_t)tmp_words(N, K) * 4);
}

}  // namespace

size_t fgmp_ws_quantize_weights(int64_t N, int64_t K) { return ws_weights_bytes(N, K); }
size_t fgmp_ws_calibrate(int64_t M, int64_t K) { return STATE_BYTES + fgmp_align1k((size_t)M * (K / 16) * 4); }

extern "C" fgmp_status fgmp_quantize_weights(const void* W_bf16, int64_t ldw, const float* fisher_elem, int64_t ldf,
                                             int64_t N, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                                             fgmp_clip_mode cm, double fp8_fraction, float tau,
                                             void* packed_out, size_t packed_bytes, float* tau_eff_out,
                                             void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!W_bf16 || !fisher_elem || !packed_out || !workspace) return FGMP_ERR_INVALID_ARG;
    if ((int)sm < 0 || (int)sm > 1 || (int)cm < 0 || (int)cm > 1) return FGMP_ERR_INVALID_ARG;
    if (!(sc.scale_fp4 >= 0.f) || !isfinite(sc.scale_fp4)) return FGMP_ERR_INVALID_ARG;
    if (!fgmp_scales_valid(sc)) return FGMP_ERR_INVALID_ARG;
    if (fp8_fraction != fp8_fraction || fp8_fraction > 1.0) return FGMP_ERR_INVALID_ARG;
    if (fp8_fraction < 0 && tau != tau) return FGMP_ERR_INVALID_ARG;
    if (N < 1 || K < 64 || (K % 64) != 0 || ldw < K || (ldw % 8) != 0 || ldf < K || (ldf % 4) != 0) return FGMP_ERR_SHAPE;
    if (((uintptr_t)W_bf16 & 15) || ((uintptr_t)fisher_elem & 15) || ((uintptr_t)packed_out & 1023) ||
        ((uintptr_t)workspace & 255)) return FGMP_ERR_SHAPE;
    const int64_t KB = K / 16, MW = (KB + 31) / 32, B = N * KB, NW = N * MW;
    if (B >= ((int64_t)1 << 32)) return FGMP_ERR_SHAPE;
    const bool fraction_mode = fp8_fraction >= 0.0;
    int64_t k = 0;
    if (fraction_mode) {
        k = (int64_t)floor(fp8_fraction * (double)B + 0.5);
        if (k > B) k = B;
    }
    // room for the lists of FP8 blocks, in 16-byte steps
    const PackedLayout L = fgmp_layout(N, K, 1, 0);
    if (packed_bytes < L.total) return FGMP_ERR_WORKSPACE;
    const int64_t room_steps = (int64_t)((packed_bytes - L.off_ovf) / 16);
    if (fraction_mode && packed_bytes < fgmp_layout(N, K, 1, k).total) return FGMP_ERR_WORKSPACE;
    if (ws_bytes < ws_weights_bytes(N, K)) return FGMP_ERR_WORKSPACE;
    fgmp_status stt;
    if ((stt = fgmp_require_sm100()) != FGMP_OK) return stt;

    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint8_t* ws = (uint8_t*)workspace;
    SelectState* st = reinterpret_cast<SelectState*>(ws);
    float* scores = reinterpret_cast<float*>(ws + STATE_BYTES);
    uint8_t* sc_tmp = ws + STATE_BYTES + fgmp_align1k((size_t)B * 4);
    uint32_t* tmp_a = reinterpret_cast<uint32_t*>(sc_tmp + fgmp_align1k((size_t)B));
    uint32_t* tmp_b = reinterpret_cast<uint32_t*>((uint8_t*)tmp_a + fgmp_align1k((size_t)tmp_words(N, K) * 4));
    uint8_t* blob = (uint8_t*)packed_out;
    const uint4* W = reinterpret_cast<const uint4*>(W_bf16);
    const int ratio = sc.fp8_log2_ratio;
    const float s8_given = sc.scale_fp8;

    FGMP_LAUNCH(FGMP_K_W_AUX, s, state_init_kernel<<<1, 256, 0, s>>>(st, sc.scale_fp4, (unsigned long long)k));
    if (sc.scale_fp4 == 0.f) {
        FGMP_LAUNCH(FGMP_K_W_AMAX, s, w_amax_kernel<<<grid_for(N * (K / 8), 256, 8), 256, 0, s>>>(W, ldw / 8, N, K / 8, st));
        FGMP_LAUNCH(FGMP_K_W_AUX, s, w_scale_kernel<<<1, 32, 0, s>>>(st));
    }
    {
        int g = grid_for(B, 256, 4);
        if (sm == FGMP_SCORE_LP_ERROR) {
            if (cm == FGMP_CLIP_SW_BRUTE) FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<0, true><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
            else                          FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<0, false><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
        } else {
            if (cm == FGMP_CLIP_SW_BRUTE) FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<1, true><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
            else                          FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<1, false><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
        }
    }
    uint32_t* mask = reinterpret_cast<uint32_t*>(blob + L.off_mask);
    uint32_t* uptr = reinterpret_cast<uint32_t*>(blob + L.off_uptr);
    const int64_t NCT = L.units;
    const int gw = grid_for(NW * 32, 256, 8);
    if (fraction_mode && k > 0) {
        run_select(scores, B, st, s);
        FGMP_LAUNCH(FGMP_K_W_MASK, s, w_eqcount_kernel<<<gw, 256, 0, s>>>(scores, N, KB, MW, st, tmp_a));
        FGMP_LAUNCH(FGMP_K_SCAN, s, scan_kernel<<<1, 1024, 0, s>>>(tmp_a, tmp_b, NW, nullptr, 0));
    } else {
        // k == 0: nothing is FP8 (tau_eff = +inf); threshold mode: the given tau
        FGMP_LAUNCH(FGMP_K_W_AUX, s, set_tau_kernel<<<1, 32, 0, s>>>(st, fraction_mode ? INFINITY : tau));
    }
    FGMP_LAUNCH(FGMP_K_W_MASK, s, w_mask_kernel<<<gw, 256, 0, s>>>(scores, N, KB, MW, st, tmp_b, mask, tmp_a));
    FGMP_LAUNCH(FGMP_K_W_MASK, s, w_unit_count_kernel<<<(unsigned)NCT, 128, 0, s>>>(mask, L, tmp_a, st));
    FGMP_LAUNCH(FGMP_K_SCAN, s, scan_kernel<<<1, 1024, 0, s>>>(tmp_a, uptr, NCT, nullptr, 1));
    FGMP_LAUNCH(FGMP_K_W_EMIT, s, w_emit_kernel<<<(unsigned)NCT, 128, 0, s>>>(W, ldw / 8, ratio, s8_given, st, sc_tmp, blob, L, room_steps));
    FGMP_LAUNCH(FGMP_K_W_AUX, s, w_header_kernel<<<1, 32, 0, s>>>(reinterpret_cast<fgmp_packed_header*>(blob), st, uptr, NCT, N, K, ratio, s8_given,
                                     room_steps, fraction_mode ? 1 : 0, tau, tau_eff_out));
    FGMP_LAUNCH(FGMP_K_W_AUX, s, w_clamp_uptr_kernel<<<grid_for(NCT + 1, 256, 1), 256, 0, s>>>(reinterpret_cast<const fgmp_packed_header*>(blob), uptr, NCT + 1, room_steps));
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_calibrate_tau(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                          int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                                          double fp8_fraction, float* tau_out,
                                          void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!tau_out || !workspace) return FGMP_ERR_INVALID_ARG;
    if (!(fp8_fraction >= 0.0) || fp8_fraction > 1.0) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || K < 64 || (K % 64) != 0) return FGMP_ERR_SHAPE;
    if ((uintptr_t)workspace & 255) return FGMP_ERR_SHAPE;
    const int64_t B = M * (K / 16);
    if (ws_bytes < fgmp_ws_calibrate(M, K)) return FGMP_ERR_WORKSPACE;
    uint8_t* ws = (uint8_t*)workspace;
    SelectState* st = reinterpret_cast<SelectState*>(ws);
    float* scores = reinterpret_cast<float*>(ws + STATE_BYTES);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    fgmp_status stt = fgmp_activation_scores(X_bf16, ldx, fisher_chan, M, K, sc, sm, scores, cuda_stream);
    if (stt != FGMP_OK) return stt;
    int64_t k = (int64_t)floor(fp8_fraction * (double)B + 0.5);
    if (k > B) k = B;
    FGMP_LAUNCH(FGMP_K_W_AUX, s, state_init_kernel<<<1, 256, 0, s>>>(st, sc.scale_fp4, (unsigned long long)k));
    if (k == 0 || k == B) {
        FGMP_LAUNCH(FGMP_K_W_AUX, s, calib_finish_kernel<<<1, 32, 0, s>>>(st, tau_out, k == 0 ? 1 : 2));
    } else {
        run_select(scores, B, st, s);
        FGMP_LAUNCH(FGMP_K_SELECT, s, next_below_kernel<<<grid_for(B, 256, 8), 256, 0, s>>>(scores, B, st));
        FGMP_LAUNCH(FGMP_K_W_AUX, s, calib_finish_kernel<<<1, 32, 0, s>>>(st, tau_out, 0));
    }
    return fgmp_launch_status();
}

extern "C" fgmp_status fgmp_weight_scores(const void* W_bf16, int64_t ldw, const float* fisher_elem, int64_t ldf,
                                          int64_t N, int64_t K, fgmp_scales sc, fgmp_score_mode sm, fgmp_clip_mode cm,
                                          float* scores, void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!W_bf16 || !fisher_elem || !scores || !workspace) return FGMP_ERR_INVALID_ARG;
    if ((int)sm < 0 || (int)sm > 1 || (int)cm < 0 || (int)cm > 1) return FGMP_ERR_INVALID_ARG;
    if (!(sc.scale_fp4 >= 0.f) || !isfinite(sc.scale_fp4)) return FGMP_ERR_INVALID_ARG;
    if (!fgmp_scales_valid(sc)) return FGMP_ERR_INVALID_ARG;
    if (N < 1 || K < 64 || (K % 64) != 0 || ldw < K || (ldw % 8) != 0 || ldf < K || (ldf % 4) != 0) return FGMP_ERR_SHAPE;
    if (((uintptr_t)W_bf16 & 15) || ((uintptr_t)fisher_elem & 15) || ((uintptr_t)scores & 15) || ((uintptr_t)workspace & 255))
        return FGMP_ERR_SHAPE;
    const int64_t KB = K / 16, B = N * KB;
    if (B >= ((int64_t)1 << 32)) return FGMP_ERR_SHAPE;
    if (ws_bytes < ws_weights_bytes(N, K)) return FGMP_ERR_WORKSPACE;
    fgmp_status stt;
    if ((stt = fgmp_require_sm100()) != FGMP_OK) return stt;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint8_t* ws = (uint8_t*)workspace;
    SelectState* st = reinterpret_cast<SelectState*>(ws);
    uint8_t* sc_tmp = ws + STATE_BYTES + fgmp_align1k((size_t)B * 4);
    const uint4* W = reinterpret_cast<const uint4*>(W_bf16);
    const int ratio = sc.fp8_log2_ratio;
    const float s8_given = sc.scale_fp8;
    FGMP_LAUNCH(FGMP_K_W_AUX, s, state_init_kernel<<<1, 256, 0, s>>>(st, sc.scale_fp4, 0ull));
    if (sc.scale_fp4 == 0.f) {
        FGMP_LAUNCH(FGMP_K_W_AMAX, s, w_amax_kernel<<<grid_for(N * (K / 8), 256, 8), 256, 0, s>>>(W, ldw / 8, N, K / 8, st));
        FGMP_LAUNCH(FGMP_K_W_AUX, s, w_scale_kernel<<<1, 32, 0, s>>>(st));
    }
    const int g = grid_for(B, 256, 4);
    if (sm == FGMP_SCORE_LP_ERROR) {
        if (cm == FGMP_CLIP_SW_BRUTE) FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<0, true><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
        else                          FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<0, false><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
    } else {
        if (cm == FGMP_CLIP_SW_BRUTE) FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<1, true><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
        else                          FGMP_LAUNCH(FGMP_K_W_SCORE, s, w_score_kernel<1, false><<<g, 256, 0, s>>>(W, ldw / 8, fisher_elem, ldf, N, KB, ratio, s8_given, st, sc_tmp, scores));
    }
    return fgmp_launch_status();
}

size_t fgmp_ws_global_tau(int64_t total) { return STATE_BYTES + fgmp_align1k((size_t)total * 4); }

extern "C" fgmp_status fgmp_global_tau(const float* const* score_arrays, const int64_t* counts, int n_tensors,
                                       double fp8_fraction, float* tau_out,
                                       void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!score_arrays || !counts || n_tensors < 1 || !tau_out || !workspace) return FGMP_ERR_INVALID_ARG;
    if (!(fp8_fraction >= 0.0) || fp8_fraction > 1.0) return FGMP_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255) return FGMP_ERR_SHAPE;
    int64_t B = 0;
    for (int i = 0; i < n_tensors; ++i) {
        if (!score_arrays[i] || counts[i] < 1) return FGMP_ERR_INVALID_ARG;
        B += counts[i];
    }
    if (B >= ((int64_t)1 << 32)) return FGMP_ERR_SHAPE;
    if (ws_bytes < fgmp_ws_global_tau(B)) return FGMP_ERR_WORKSPACE;
    fgmp_status stt;
    if ((stt = fgmp_require_sm100()) != FGMP_OK) return stt;
    uint8_t* ws = (uint8_t*)workspace;
    SelectState* st = reinterpret_cast<SelectState*>(ws);
    float* scores = reinterpret_cast<float*>(ws + STATE_BYTES);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // all scores side by side: the threshold is a rank statistic of their union
    int64_t off = 0;
    for (int i = 0; i < n_tensors; ++i) {
        if (cudaMemcpyAsync(scores + off, score_arrays[i], (size_t)counts[i] * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
            return FGMP_ERR_CUDA;
        off += counts[i];
    }
    int64_t k = (int64_t)floor(fp8_fraction * (double)B + 0.5);
    if (k > B) k = B;
    FGMP_LAUNCH(FGMP_K_W_AUX, s, state_init_kernel<<<1, 256, 0, s>>>(st, 1.0f, (unsigned long long)k));
    if (k == 0 || k == B) {
        FGMP_LAUNCH(FGMP_K_W_AUX, s, calib_finish_kernel<<<1, 32, 0, s>>>(st, tau_out, k == 0 ? 1 : 2));
    } else {
        run_select(scores, B, st, s);
        FGMP_LAUNCH(FGMP_K_SELECT, s, next_below_kernel<<<grid_for(B, 256, 8), 256, 0, s>>>(scores, B, st));
        FGMP_LAUNCH(FGMP_K_W_AUX, s, calib_finish_kernel<<<1, 32, 0, s>>>(st, tau_out, 0));
    }
    return fgmp_launch_status();
}
