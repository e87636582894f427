// fgmp_linear for decode-sized batches (M <= 16 tokens): a weight-streaming kernel that
// reads the packed weights exactly once (Section 4.1 of the paper: the four block-pair
// products, FP32 accumulation), optionally with the activation quantizer of Section 4.2 in
// its prologue (fgmp_linear_fused).
//
// At this size the layer is bound by the weight stream, not by arithmetic, and every block pair
// has an exact fp16 form: an E2M1 code times its E4M3 microscale has 6 significant bits, an E4M3
// code times the power of two between the tensor scales has 4.  So both operands go through
// mma.sync m16n8k16 (fp16 in, fp32 accumulation) as their true values over the tensor scales.
// 16 weight rows are the M side of an MMA, a token octet the N side.  The order of the contraction
// index is free as long as both operands agree, so an MMA step takes four consecutive elements of
// one block per lane: lane (g, t) owns, for hq = 0..3, block column 4t + hq of rows 32jr + 8k + g,
// k = 0..3, of the unit, and its four MMA steps per 16-row tile walk through that block.  A lane
// therefore meets whole blocks, and the format of a block is a per-lane choice between two
// conversion instructions (cvt e2m1x2 / cvt e4m3x2, predicated on the block's flag) followed by the
// same multiply with the block's scale byte (the microscale, or 2^ratio for an FP8 block): the
// mixing of formats costs conversions, not extra MMAs, and all sums stay in registers.
// The record of a unit is stored in exactly this order (fgmp_common.cuh), so every shared-memory read
// of a warp is one contiguous, conflict-free piece; the activation record of a chunk likewise.
//
// Work is split stream-K style over (128-row tile, 256-element K chunk) units so that all SMs
// stream the same number of bytes; a unit is up to three bulk copies (its fixed-size record, the
// second halves of its FP8 blocks, the activation record of its chunk) into a ring of stages.
// The 16 warps form four groups; consecutive units of a CTA go to consecutive groups, so four units
// are being multiplied at any time and the latencies of one (barrier, shared-memory loads, the
// dependent MMAs) hide behind the others.  Inside a group warp jr takes rows 32jr .. 32jr+31.  There
// is no producer warp: the warp that is last to finish a unit refills its stage.  Tiles shared by
// several CTAs are reduced in a fixed order by the CTA that arrives last.  Every sum is taken in a
// fixed order: results are reproducible bit for bit.
#include "fgmp_common.cuh"
#include "fgmp_actq.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <cuda_fp16.h>
#include <mutex>
#include <type_traits>

namespace {

constexpr int MATH_WARPS = 16, MATH_THREADS = 32 * MATH_WARPS;
constexpr int DEC_THREADS = MATH_THREADS;
constexpr uint32_t OVF_CAP = 2560;              // overflow bytes of a unit that fit a stage (320 FP8 blocks); more are read from global
constexpr uint32_t STG_OVF = REC_BYTES;
constexpr uint32_t STG_A = STG_OVF + OVF_CAP;                                                    // 21120
constexpr uint32_t DEC_STAGE_BYTES = STG_A + AREC_BYTES;                                         // 29312
constexpr int DEC_STAGES = 6;                   // at most; a launch uses DecParams::stages of them
constexpr uint32_t EPI_FLOATS = 4 * 128 * 16;   // [warp / 4][row][token] fp32: the partial sums of a tile
constexpr int MAX_SPAN = 8192;                  // units of one CTA whose overflow starts fit the shared-memory table
constexpr size_t dec_smem(int stages, int64_t span) { return (size_t)stages * DEC_STAGE_BYTES + EPI_FLOATS * 4 + ((size_t)(span + 1) * 4 + 15) / 16 * 16 + 1024 /*alignment*/ + 512 /*barriers*/; }
static_assert(dec_smem(DEC_STAGES, 64) <= 232448, "shared memory of one CTA");
static_assert((STG_A % 128) == 0 && (DEC_STAGE_BYTES % 128) == 0, "bulk-copy alignment");

// control words of the workspace (int32, from byte 256): see fgmp_linear_fused
enum { CW_EPOCH = 0, CW_DONE = 1, CW_CLAIM = 2, CW_QCOUNT = 3, CW_QREADY = 4 };

struct DecParams {
    const uint8_t* wblob; const uint8_t* ablob;
    PackedLayout LW, LA;
    float* Y; void* Ybf; int64_t ldy; int y_is_bf16;
    int64_t M, N, K;
    int64_t total;            // tiles * chunks
    int64_t chunks;
    int* status; uint32_t* counters; float* partials; int maxseg;
    int stages;               // depth of the unit ring, 2 .. DEC_STAGES
    // activation quantizer in the prologue (fused launches only)
    const uint8_t* X; int64_t ldx;        // bf16 [M, ldx]
    const float* fisher;
    ActQuantScalars q; int q_mode;        // q_mode: fgmp_score_mode
    uint8_t* arec;                        // where the fp16 records of the chunks go (and are streamed from)
    uint8_t* q_codes4; uint8_t* q_sf; uint8_t* q_mask; uint8_t* q_codes8; fgmp_packed_header* q_header;   // optional packed output
    uint32_t* cw;                         // control words
};

struct StageMeta { uint32_t step, staged; };

// Profiling builds (-DFGMP_TIMELINE) stamp the global timer at the phases of every CTA into a buffer
// registered with fgmp_debug_timeline (16 x uint64 per CTA); ordinary builds contain none of this.
#ifdef FGMP_TIMELINE
__device__ unsigned long long* g_timeline = nullptr;
#define FGMP_STAMP(slot) do { if (g_timeline && threadIdx.x == 0) g_timeline[(size_t)blockIdx.x * 16 + (slot)] = globaltimer_ns(); } while (0)
#define FGMP_STAMP_ANY(slot) do { if (g_timeline) g_timeline[(size_t)blockIdx.x * 16 + (slot)] = globaltimer_ns(); } while (0)
#else
#define FGMP_STAMP(slot) do { } while (0)
#define FGMP_STAMP_ANY(slot) do { } while (0)
#endif     // overflow start (16-byte steps), bytes of it in the stage

__device__ __forceinline__ int64_t cta_of_unit(int64_t i, int64_t G, int64_t total) { return ((i + 1) * G - 1) / total; }

__device__ __forceinline__ void math_bar() { asm volatile("bar.sync 1, %0;" ::"n"(MATH_THREADS) : "memory"); }

// eight E2M1 codes (one word) times a scale (both halves of sc2) -> four fp16 pairs, exact
__device__ __forceinline__ void dq_nvfp4(uint32_t c32, uint32_t sc2, uint32_t (&x)[4])
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

// The same eight elements of a block that is NVFP4 (codes in c32) or, if is8 != 0, FP8 (E4M3 codes in e8a,
// e8b): the lane's flag picks the conversion, the multiply with the block's scale pair is common.
__device__ __forceinline__ void dq_mixed(uint32_t c32, uint32_t e8a, uint32_t e8b, uint32_t is8, uint32_t sc2, uint32_t (&x)[4])
{
    uint32_t q0, q1, q2, q3;
    asm("{\n\t.reg .pred p;\n\t.reg .b8 b0, b1, b2, b3;\n\t.reg .b16 h0, h1, h2, h3;\n\t"
        "setp.ne.u32 p, %7, 0;\n\t"
        "mov.b32 {b0, b1, b2, b3}, %4;\n\tmov.b32 {h0, h1}, %5;\n\tmov.b32 {h2, h3}, %6;\n\t"
        "@!p cvt.rn.f16x2.e2m1x2 %0, b0;\n\t@p cvt.rn.f16x2.e4m3x2 %0, h0;\n\t"
        "@!p cvt.rn.f16x2.e2m1x2 %1, b1;\n\t@p cvt.rn.f16x2.e4m3x2 %1, h1;\n\t"
        "@!p cvt.rn.f16x2.e2m1x2 %2, b2;\n\t@p cvt.rn.f16x2.e4m3x2 %2, h2;\n\t"
        "@!p cvt.rn.f16x2.e2m1x2 %3, b3;\n\t@p cvt.rn.f16x2.e4m3x2 %3, h3;\n\t}"
        : "=&r"(q0), "=&r"(q1), "=&r"(q2), "=&r"(q3) : "r"(c32), "r"(e8a), "r"(e8b), "r"(is8));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[0]) : "r"(q0), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[1]) : "r"(q1), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[2]) : "r"(q2), "r"(sc2));
    asm("mul.f16x2 %0, %1, %2;" : "=r"(x[3]) : "r"(q3), "r"(sc2));
}

// Bounded wait for a word in global memory to take a value that another CTA publishes.
__device__ __noinline__ bool wait_global_equals(const uint32_t* addr, uint32_t value, volatile int* abort_flag, int* status, int where)
{
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
        if (v == value) return true;
        if (*abort_flag) return false;
        if (globaltimer_ns() - t0 > MBAR_WAIT_LIMIT_NS) {
            *abort_flag = 1;
            atomicCAS(status, 0, (int)FGMP_ERR_TIMEOUT);
            atomicExch(status + 1, where);
            return false;
        }
        __nanosleep(100);
    }
}

// One work item of the prologue quantizer: chunk c (256 elements), token octet o: warp w takes token
// 8o + w/2 and the eight blocks 16c + 8(w%2) .. +7, four lanes per block.
template <int MODE>
__device__ __forceinline__ void quantize_item(const DecParams& p, int64_t c, int o)
{
    const uint32_t w = threadIdx.x >> 5, lane = threadIdx.x & 31u, li = lane & 3u;
    const int64_t m = 8 * o + (int64_t)(w >> 1);
    const uint32_t j = 8u * (w & 1u) + (lane >> 2);
    const int64_t kb = 16 * c + j;
    uint8_t* dst = p.arec + (size_t)c * AREC_BYTES + fgmp_arec_offset((uint32_t)m, j, li >> 1) + (li & 1u) * 8u;
    if (m >= p.M) {                                   // token rows beyond the batch are zero
        *reinterpret_cast<uint2*>(dst) = make_uint2(0u, 0u);
        return;
    }
    const uint2 x = __ldg(reinterpret_cast<const uint2*>(p.X + ((size_t)m * p.ldx + (size_t)kb * 16 + 4 * li) * 2));
    const float4 f = __ldg(reinterpret_cast<const float4*>(p.fisher + kb * 16 + 4 * li));
    const BlockQuarter r = quantize_block_quarter<MODE>(x, f, p.q);
    *reinterpret_cast<uint2*>(dst) = r.h;
    if (p.q_codes4) {
        const int64_t MW = p.LA.MW;
        *reinterpret_cast<uint16_t*>(p.q_codes4 + (m * p.K) / 2 + kb * 8 + li * 2) = (uint16_t)r.c4;
        if (li == 0) p.q_sf[fgmp_sf_offset(m, kb, p.K)] = (uint8_t)r.sc;
        if (r.is8) *reinterpret_cast<uint32_t*>(p.q_codes8 + m * p.K + kb * 16 + 4 * li) = r.c8;
        const uint32_t bal = __ballot_sync(0xffffffffu, r.is8 && li == 0);
        if (lane == 0) {
            uint32_t byte = 0;
#pragma unroll
            for (int b = 0; b < 8; ++b) byte |= ((bal >> (4 * b)) & 1u) << b;
            const int64_t kb0 = kb;                   // lane 0: first block of the warp's eight
            uint8_t* mb = p.q_mask + (size_t)m * MW * 4 + (kb0 >> 3);
            mb[0] = (uint8_t)byte;
            if (kb0 + 8 == p.LA.KB && (p.LA.KB & 31) != 0) { mb[1] = 0; mb[2] = 0; }   // rest of the row's last mask word
        }
    }
}

__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// NH = token octets in use: 1 for M <= 8, else 2.  FUSED: the activation quantizer runs in the prologue.
// NG = groups of 16 / NG warps that work on different units at the same time; a warp takes rows 32jr .. 32jr+31
// and NG of the four classes of block columns (j % 4).
template <int NH, bool FUSED, int NG>
__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(DecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    // 1 KiB aligned; an offset from the array keeps the pointer known to be shared memory (plain ld.shared / st.shared)
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int S = p.stages;
    float* epi = reinterpret_cast<float*>(smem + (size_t)S * DEC_STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(epi + EPI_FLOATS);             // full[DEC_STAGES]
    uint32_t* done = reinterpret_cast<uint32_t*>(bars + DEC_STAGES);            // warps that have finished with a stage
    StageMeta* smeta = reinterpret_cast<StageMeta*>(done + DEC_STAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smeta + DEC_STAGES);
    volatile uint32_t* s_misc = reinterpret_cast<volatile uint32_t*>(abort_flag + 1);   // [0] tag, [1..2] claimed item, [3] last-arrival flag
    uint32_t* table = const_cast<uint32_t*>(s_misc + 8);                        // overflow starts of this CTA's units (+ 1)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars);
    FGMP_STAMP(0);
    constexpr uint32_t A_BYTES = NH == 2 ? AREC_BYTES : AREC_BYTES / 2;

    // this CTA's span of (tile, chunk) units
    const int64_t G = gridDim.x, C = p.chunks;
    const int64_t u_begin = ((int64_t)blockIdx.x * p.total) / G, u_end = ((int64_t)(blockIdx.x + 1) * p.total) / G;
    const int n_units = (int)(u_end - u_begin);
    const uint32_t* uptr = reinterpret_cast<const uint32_t*>(p.wblob + p.LW.off_uptr);
    const uint8_t* recs = p.wblob + p.LW.off_rec;
    const uint8_t* ovfs = p.wblob + p.LW.off_ovf;
    const uint8_t* arec = FUSED ? p.arec : p.ablob + p.LA.off_arec;

    // the copies of unit i (index inside the span) into its stage, by one thread
    auto stage_dst = [&](int stage) { return smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES); };
    auto issue_rec = [&](int i, int stage) { bulk_load(stage_dst(stage), recs + (size_t)(u_begin + i) * REC_BYTES, REC_BYTES, full0 + 8 * stage); };
    auto issue_ovf = [&](int i, int stage, bool expect) {
        const uint32_t step0 = table[i], bytes = (table[i + 1] - step0) * 16u;
        const uint32_t staged = bytes < OVF_CAP ? bytes : OVF_CAP;
        smeta[stage].step = step0; smeta[stage].staged = staged;
        if (expect && staged) mbar_expect_tx_only(full0 + 8 * stage, staged);
        if (staged) bulk_load(stage_dst(stage) + STG_OVF, ovfs + (size_t)step0 * 16, staged, full0 + 8 * stage);
        return staged;
    };
    auto issue_a = [&](int i, int stage) {
        bulk_load(stage_dst(stage) + STG_A, arec + (size_t)((u_begin + i) % C) * AREC_BYTES, A_BYTES, full0 + 8 * stage);
    };

    // ------------------------------------------------------------ set-up: barriers, the weight blob's header, and the
    // first stages' weight copies.  The packed weights are not written by whatever runs before this kernel, so all
    // of this may overlap the end of that kernel (programmatic dependent launch).
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); done[s] = 0; }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // nothing is read through the blob's tables before its header has been seen to describe this call
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const uint2 mv = __ldg(reinterpret_cast<const uint2*>(hw));
        const bool okh = mv.x == FGMP_MAGIC && mv.y == 6u && __ldg(&hw->rows) == p.N && __ldg(&hw->K) == p.K &&
                         __ldg(&hw->kind) == 1u && __ldg(&hw->error) == 0;
        if (!okh) { *abort_flag = 1; atomicCAS(p.status, 0, (int)FGMP_ERR_INVALID_ARG); atomicExch(p.status + 1, 9); }
    }
    __syncthreads();
    FGMP_STAMP(1);
    const int pre = min(S, n_units);
    if (!*abort_flag) {
        for (int i = threadIdx.x; i <= n_units; i += DEC_THREADS) table[i] = __ldg(uptr + u_begin + i);
        if (threadIdx.x == 0)
            for (int s = 0; s < pre; ++s) { mbar_expect_tx_only(full0 + 8 * s, REC_BYTES + A_BYTES); issue_rec(s, s); }
    }
    __syncthreads();
    if (!*abort_flag && threadIdx.x == 0)
        for (int s = 0; s < pre; ++s) issue_ovf(s, s, true);
    FGMP_STAMP(2);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Launched as a programmatic dependent of the preceding kernel in the stream, this kernel may have
    // started before that one finished: everything above touches neither its output nor the workspace.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    FGMP_STAMP(3);
    if (FUSED) {
        if (threadIdx.x == 0) {
            uint32_t e;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(e) : "l"(p.cw + CW_EPOCH) : "memory");
            s_misc[0] = e + 1u;
        }
        __syncthreads();
    }
    const uint32_t tag = FUSED ? s_misc[0] : 0u;

    if (!*abort_flag) {
        if (FUSED) {
            // The quantizer's work items are handed out through a counter, so that every item is taken by a CTA
            // that is running: no CTA ever waits for one that has not started.  The counter and the count of
            // finished items wrap to zero with the call's last access.
            const uint32_t octets = p.M > 8 ? 2u : 1u;
            const uint32_t n_items = (uint32_t)C * octets;
            for (uint32_t it = 0;; ++it) {
                if (threadIdx.x == 0) s_misc[1 + (it & 1u)] = atomicInc(p.cw + CW_CLAIM, n_items + (uint32_t)G - 1u);
                math_bar();
                const uint32_t item = s_misc[1 + (it & 1u)];
                if (item >= n_items) break;
                if (item == 0 && threadIdx.x == 0 && p.q_header) {
                    fgmp_packed_header* h = p.q_header;
                    h->magic = FGMP_MAGIC; h->version = 6; h->rows = p.M; h->K = p.K; h->scale_fp4 = p.q.s4;
                    h->fp8_log2_ratio = p.q.ratio; h->n_fp8 = -1; h->tau_eff = 0.f; h->kind = 0; h->capacity = 0;
                    h->error = 0;
                }
                if (p.q_mode == 0) quantize_item<0>(p, (int64_t)(item / octets), (int)(item % octets));
                else               quantize_item<1>(p, (int64_t)(item / octets), (int)(item % octets));
                __threadfence();
                math_bar();
                if (threadIdx.x == 0 && atomicInc(p.cw + CW_QCOUNT, n_items - 1u) == n_items - 1u)
                    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.cw + CW_QREADY), "r"(tag) : "memory");
            }
        }
        // the activation records of the first stages; their barriers' one arrival comes last
        FGMP_STAMP(4);
        if (threadIdx.x == 0) {
            bool oka = true;
            if (FUSED) {
                // every chunk's record is in place once the last work item of the quantizer has been handed in
                oka = wait_global_equals(p.cw + CW_QREADY, tag, abort_flag, p.status, 8);
                asm volatile("fence.proxy.async;" ::: "memory");   // records were written with ordinary stores, the bulk copy reads them
            } else {
                const fgmp_packed_header* ha = reinterpret_cast<const fgmp_packed_header*>(p.ablob);
                const uint2 mv = __ldg(reinterpret_cast<const uint2*>(ha));
                if (!(mv.x == FGMP_MAGIC && mv.y == 6u && __ldg(&ha->rows) == p.M && __ldg(&ha->K) == p.K && __ldg(&ha->kind) == 0u)) {
                    *abort_flag = 1; atomicCAS(p.status, 0, (int)FGMP_ERR_INVALID_ARG); atomicExch(p.status + 1, 10);
                    oka = false;
                }
            }
            if (oka) for (int s = 0; s < pre; ++s) { issue_a(s, s); mbar_arrive(full0 + 8 * s); }
        }
        FGMP_STAMP(5);

        // ------------------------------------------------------------ the units of this CTA, group by group
        constexpr int GROUPS = NG, GROUP_WARPS = MATH_WARPS / NG;
        const uint32_t part = (uint32_t)warp >> 2, jr = (uint32_t)warp & 3u;      // part: which partial tile this warp's sums go to
        const uint32_t gq = part * NG / 4u;                                       // group
        const int hq0 = NG == 4 ? 0 : (NG == 2 ? 2 * (int)(part & 1u) : (int)part);
        const uint32_t g = (uint32_t)lane >> 2, t = (uint32_t)lane & 3u;
        const uint32_t sf_off = REC_SF + jr * 512u + (uint32_t)lane * 16u;
        const uint32_t tcol = (2 * t) & 3u, tpiece = t >> 1;
        const float alpha = FUSED ? __fmul_rn(p.q.s4, __ldg(&reinterpret_cast<const fgmp_packed_header*>(p.wblob)->scale_fp4))
                                  : __fmul_rn(__ldg(&reinterpret_cast<const fgmp_packed_header*>(p.ablob)->scale_fp4),
                                              __ldg(&reinterpret_cast<const fgmp_packed_header*>(p.wblob)->scale_fp4));
        bool ok = true;
        for (int sbeg = 0; sbeg < n_units;) {
            const int64_t tile = (u_begin + sbeg) / C;
            const int send = (int)min((int64_t)n_units, (tile + 1) * C - u_begin);
            // acc[mt][nh] = rows 32jr + 16mt + {g, g + 8} x tokens 8nh + {2t, 2t+1}, this group's units of the tile
            float acc[2][NH][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) acc[mt][nh][0] = acc[mt][nh][1] = acc[mt][nh][2] = acc[mt][nh][3] = 0.f;
            for (int i = sbeg + (int)((gq - (uint32_t)sbeg) & (uint32_t)(NG - 1)); i < send; i += GROUPS) {
                const int stage = i % S; const uint32_t phase = (uint32_t)(i / S) & 1u;
                if (ok) ok = mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 5);
                if (!ok) break;
                if (i == 0) FGMP_STAMP(6);
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint4 scv = *reinterpret_cast<const uint4*>(sb + sf_off);
                const bool any8 = __any_sync(0xffffffffu, ((scv.x | scv.y | scv.z | scv.w) & 0x80808080u) != 0u);
                // where this lane's overflow entries start, per hq (only with FP8 blocks in the unit)
                uint32_t idx4 = 0;
                if (any8) {
                    const uint32_t pack = __popc(scv.x & 0x80808080u) | (__popc(scv.y & 0x80808080u) << 8) |
                                          (__popc(scv.z & 0x80808080u) << 16) | (__popc(scv.w & 0x80808080u) << 24);
                    uint32_t incl = pack;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += y;
                    }
                    idx4 = incl - pack;
                }
                const uint32_t staged = smeta[stage].staged;
                const uint8_t* ovf_g = ovfs + (size_t)smeta[stage].step * 16;
#pragma unroll 1
                for (int hq = hq0; hq < hq0 + NG; ++hq) {
                    const uint32_t w = 4 * jr + (uint32_t)hq;
                    const uint32_t sc4 = *reinterpret_cast<const uint32_t*>(sb + sf_off + 4 * hq);
                    const uint4 s01 = *reinterpret_cast<const uint4*>(sb + REC_W4 + w * 1024u + (uint32_t)lane * 16u);
                    const uint4 s23 = *reinterpret_cast<const uint4*>(sb + REC_W4 + w * 1024u + 512u + (uint32_t)lane * 16u);
                    const uint32_t a_off = STG_A + (uint32_t)(hq * 2) * 512u + (uint32_t)lane * 16u;
                    // scale pairs: byte k of sc4 (flag bit cleared) in both halves, E4M3 -> fp16
                    uint32_t sc2[4];
                    {
                        const uint32_t s7 = sc4 & 0x7f7f7f7fu;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t two = __byte_perm(s7, 0u, 0x4400u | (uint32_t)(k << 4) | (uint32_t)k);
                            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2[k]) : "h"((uint16_t)two));
                        }
                    }
                    const uint32_t slot[4][2] = {{s01.x, s01.y}, {s01.z, s01.w}, {s23.x, s23.y}, {s23.z, s23.w}};
                    // the MMAs of one half (elements 8h .. 8h+7 of every block): x[k] = four fp16 pairs of slot k
                    auto half_mma = [&](int h, const uint32_t (&x)[4][4]) {
                        uint4 b[NH];
#pragma unroll
                        for (int nh = 0; nh < NH; ++nh) b[nh] = *reinterpret_cast<const uint4*>(sb + a_off + nh * 4096 + h * 512);
#pragma unroll
                        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                            for (int sl = 0; sl < 2; ++sl)
#pragma unroll
                                for (int nh = 0; nh < NH; ++nh)
                                    mma_f16_16816(acc[mt][nh], x[2 * mt][2 * sl], x[2 * mt + 1][2 * sl], x[2 * mt][2 * sl + 1], x[2 * mt + 1][2 * sl + 1],
                                                  sl ? b[nh].z : b[nh].x, sl ? b[nh].w : b[nh].y);
                    };
                    if (!any8) {
                        // no FP8 block in the warp's part of the unit: every slot holds sixteen E2M1 codes
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint32_t x[4][4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) dq_nvfp4(slot[k][h], sc2[k], x[k]);
                            half_mma(h, x);
                        }
                    } else {
                        // second halves of this lane's FP8 blocks: consecutive entries of the unit's overflow list
                        const uint32_t flags = sc4 & 0x80808080u;
                        uint32_t idx = ((idx4 >> (8 * hq)) & 0xffu) + *reinterpret_cast<const uint16_t*>(sb + REC_WSTART + 2 * w);
                        uint2 hi8[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            hi8[k] = make_uint2(0u, 0u);
                            if (flags & (0x80u << (8 * k))) {
                                hi8[k] = (idx * 8u + 8u <= staged) ? *reinterpret_cast<const uint2*>(sb + STG_OVF + idx * 8u)
                                                                   : __ldg(reinterpret_cast<const uint2*>(ovf_g + (size_t)idx * 8));
                                ++idx;
                            }
                        }
                        // NVFP4: codes 0..7 in slot word 0, 8..15 in word 1; FP8: codes 0..3, 4..7 in the slot, 8..11, 12..15 in the overflow entry
                        {
                            uint32_t x[4][4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) dq_mixed(slot[k][0], slot[k][0], slot[k][1], flags & (0x80u << (8 * k)), sc2[k], x[k]);
                            half_mma(0, x);
                        }
                        {
                            uint32_t x[4][4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) dq_mixed(slot[k][1], hi8[k].x, hi8[k].y, flags & (0x80u << (8 * k)), sc2[k], x[k]);
                            half_mma(1, x);
                        }
                    }
                }
                // this warp is done with the stage; the group's last warp to say so refills it with the unit S further on
                __syncwarp();
                if (lane == 0) {
                    uint32_t old;
                    asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(smem_u32(done + stage)) : "memory");
                    if (old == GROUP_WARPS - 1) {
                        done[stage] = 0;
                        const int nxt = i + S;
                        if (nxt < n_units) {
                            const uint32_t step0 = table[nxt], bytes = (table[nxt + 1] - step0) * 16u;
                            mbar_expect_tx(full0 + 8 * stage, REC_BYTES + A_BYTES + (bytes < OVF_CAP ? bytes : OVF_CAP));
                            issue_rec(nxt, stage); issue_ovf(nxt, stage, false); issue_a(nxt, stage);
                        }
                    }
                }
            }

            // ---- end of a segment (this CTA's units of one tile): the groups' sums are added, then the tile is
            // written or, if other CTAs share it, handed in; the last CTA to arrive adds the parts in order.
            // (After a failed wait the barriers below are still passed by everyone; nothing is written.)
            if (send == n_units) { FGMP_STAMP(7); if (threadIdx.x == DEC_THREADS - 32) FGMP_STAMP_ANY(8); }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int rh = 0; rh < 2; ++rh) {
                    const uint32_t r = 32 * jr + 16 * (uint32_t)mt + 8 * (uint32_t)rh + g;
                    float2* pt = reinterpret_cast<float2*>(epi + part * 2048u + r * 16u + (((tpiece ^ (r >> 1)) & 3u) << 2) + tcol);
                    pt[0] = make_float2(acc[mt][0][2 * rh], acc[mt][0][2 * rh + 1]);
                    if (NH == 2)
                        *reinterpret_cast<float2*>(reinterpret_cast<uintptr_t>(pt) ^ 32) = make_float2(acc[mt][NH - 1][2 * rh], acc[mt][NH - 1][2 * rh + 1]);
                }
            math_bar();
            const bool good = !*abort_flag;
            const uint32_t row = threadIdx.x >> 2, tq = threadIdx.x & 3u;      // this thread: tokens 4tq .. 4tq+3 of one row
            const bool live = tq < 2u * NH;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (live) {
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float4 x = *reinterpret_cast<const float4*>(epi + h * 2048 + row * 16u + (((tq ^ (row >> 1)) & 3u) << 2));
                    v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
                }
            }
            const bool whole = (u_begin + sbeg == tile * C) && (u_begin + send == (tile + 1) * C);
            bool write_out = whole;
            if (!whole) {
                const int64_t c_first = cta_of_unit(tile * C, G, p.total);
                const int64_t c_last = cta_of_unit((tile + 1) * C - 1, G, p.total);
                const int nseg = (int)(c_last - c_first + 1), slot_i = (int)(blockIdx.x - c_first);
                if (live && good) __stcg(reinterpret_cast<float4*>(p.partials + (((size_t)tile * p.maxseg + slot_i) * 128 + row) * 16 + 4 * tq), v);
                __threadfence();
                math_bar();
                // the counter wraps to zero with the last arrival, so the workspace is ready for the next call
                if (threadIdx.x == 0) s_misc[3] = (good && atomicInc(p.counters + tile, (uint32_t)(nseg - 1)) == (uint32_t)(nseg - 1)) ? 1u : 0u;
                math_bar();
                write_out = false;
                if (s_misc[3]) {
                    __threadfence();
                    v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (live)
                        for (int sgi = 0; sgi < nseg; ++sgi) {
                            const float4 x = __ldcg(reinterpret_cast<const float4*>(p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16 + 4 * tq));
                            v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
                        }
                    write_out = true;
                }
            }
            const int64_t n = tile * 128 + row;
            if (write_out && good && live && n < p.N) {
                const float y[4] = {v.x * alpha, v.y * alpha, v.z * alpha, v.w * alpha};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int64_t m = 4 * tq + i;
                    if (m < p.M) {
                        if (p.y_is_bf16) reinterpret_cast<__nv_bfloat16*>(p.Ybf)[m * p.ldy + n] = __float2bfloat16_rn(y[i]);
                        else p.Y[m * p.ldy + n] = y[i];
                    }
                }
            }
            math_bar();                                // the next segment's sums overwrite the tile
            sbeg = send;
        }
    }

    __syncthreads();
    FGMP_STAMP(9);
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    } else if (FUSED && threadIdx.x == 0) {
        // the CTA that finishes last moves the call number on: the next call publishes under a new tag
        if (atomicInc(p.cw + CW_DONE, (uint32_t)G - 1u) == (uint32_t)G - 1u)
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.cw + CW_EPOCH), "r"(tag) : "memory");
    }
}

struct DecPlan { int64_t tiles, chunks, total; int grid; int maxseg; int64_t span; };

DecPlan decode_plan(int64_t N, int64_t K)
{
    DecPlan d;
    d.tiles = (N + 127) / 128; d.chunks = K / 256; d.total = d.tiles * d.chunks;
    const int sms = fgmp_sm_count();
    d.grid = (int)(d.total < sms ? d.total : sms);
    // a tile of `chunks` units meets at most this many CTA spans of >= floor(total/grid) units
    const int64_t span = d.total / d.grid;
    d.maxseg = (int)((d.chunks + span - 1) / span + 1);
    d.span = (d.total + d.grid - 1) / d.grid;           // the longest span of a CTA
    return d;
}

std::mutex g_dec_mu;                 // guards the per-device caches below
bool g_attr_set[64] = {};

fgmp_status set_attrs_once()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FGMP_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_dec_mu);
    if (!g_attr_set[dev]) {
        const int most = 232448;
#define FGMP_SET(NG_) \
        if (cudaFuncSetAttribute(decode_kernel<1, false, NG_>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess || \
            cudaFuncSetAttribute(decode_kernel<2, false, NG_>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess || \
            cudaFuncSetAttribute(decode_kernel<1, true, NG_>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess || \
            cudaFuncSetAttribute(decode_kernel<2, true, NG_>, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess) \
            return FGMP_ERR_CUDA;
        FGMP_SET(1) FGMP_SET(2) FGMP_SET(4)
#undef FGMP_SET
        g_attr_set[dev] = true;
    }
    return FGMP_OK;
}

// Workspace of the decode path, all inside the control area that must be zero before the first call and
// that every call leaves zero (the call number excepted): status at 0, control words at 256, one
// stream-K counter per tile from 1024; partial sums behind the control area, then (fused calls) the
// activation records.
DecParams base_params(const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                      void* workspace, const DecPlan& d)
{
    uint8_t* ws = (uint8_t*)workspace;
    DecParams p{};
    p.wblob = (const uint8_t*)packed_weights;
    p.LW = fgmp_layout(N, K, 1, 0); p.LA = fgmp_layout(M, K, 0, 0);
    p.Y = (float*)Y; p.Ybf = Y; p.ldy = ldy; p.y_is_bf16 = y_is_bf16;
    p.M = M; p.N = N; p.K = K; p.total = d.total; p.chunks = d.chunks;
    p.status = reinterpret_cast<int*>(ws);
    p.cw = reinterpret_cast<uint32_t*>(ws + 256);
    p.counters = reinterpret_cast<uint32_t*>(ws + 1024);
    p.partials = reinterpret_cast<float*>(ws + FGMP_WS_CONTROL_BYTES);
    p.maxseg = d.maxseg;
    // Ring depth: long spans are bound by the weight stream and want every stage; short ones are bound by
    // set-up, which a smaller footprint shortens.
    p.stages = DEC_STAGES;
    while (p.stages > 2 && dec_smem(p.stages, d.span) > 232448) --p.stages;      // very long spans: their table takes the room of a stage
    return p;
}

template <bool FUSED>
fgmp_status launch_decode(const DecParams& p, const DecPlan& d, bool programmatic, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)d.grid); cfg.blockDim = dim3(DEC_THREADS); cfg.dynamicSmemBytes = dec_smem(p.stages, d.span); cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = programmatic ? 1 : 0;
    const int ng = 4;       // measured on Llama-2 shapes: four groups of four warps are the fastest split
#define FGMP_GO(NG_) \
    if (p.M <= 8) { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<1, FUSED, NG_>, p)); } \
    else          { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<2, FUSED, NG_>, p)); }
    if (ng == 1) { FGMP_GO(1) } else if (ng == 4) { FGMP_GO(4) } else { FGMP_GO(2) }
#undef FGMP_GO
    return fgmp_launch_status();
}

}  // namespace

bool fgmp_decode_supported(int64_t M, int64_t N, int64_t K)
{
    if (!(M >= 1 && M <= 16 && N >= 1 && K >= 256 && (K % 256) == 0 &&
          1024 + ((N + 127) / 128) * 4 <= (int64_t)FGMP_WS_CONTROL_BYTES)) return false;
    const int64_t total = ((N + 127) / 128) * (K / 256);
    const int sms = fgmp_sm_count();
    return (total + sms - 1) / sms <= MAX_SPAN;
}

size_t fgmp_ws_decode(int64_t M, int64_t N, int64_t K)
{
    if (!fgmp_decode_supported(M, N, K)) return 0;
    const DecPlan d = decode_plan(N, K);
    return (size_t)FGMP_WS_CONTROL_BYTES + (size_t)d.tiles * d.maxseg * 128 * 16 * 4;
}

size_t fgmp_ws_linear_fused(int64_t M, int64_t N, int64_t K)
{
    if (!fgmp_decode_supported(M, N, K)) return fgmp_ws_linear(M, N, K);
    return fgmp_align1k(fgmp_ws_decode(M, N, K)) + (size_t)(K / 256) * AREC_BYTES;
}

// clear_first: zero the control area on the stream before the kernel (for scratch whose state the
// caller cannot vouch for); otherwise the kernel is launched as a programmatic dependent of the
// kernel before it in the stream, so that its set-up and first weight copies overlap that kernel's end.
fgmp_status fgmp_linear_decode(const void* packed_acts, const void* packed_weights, void* Y, int y_is_bf16, int64_t ldy,
                               int64_t M, int64_t N, int64_t K, void* workspace, bool clear_first, cudaStream_t s)
{
    const DecPlan d = decode_plan(N, K);
    DecParams p = base_params(packed_weights, Y, y_is_bf16, ldy, M, N, K, workspace, d);
    p.ablob = (const uint8_t*)packed_acts;
    fgmp_status st = set_attrs_once();
    if (st != FGMP_OK) return st;
    if (clear_first && cudaMemsetAsync(workspace, 0, 1024 + (size_t)d.tiles * 4, s) != cudaSuccess) return FGMP_ERR_CUDA;
    return launch_decode<false>(p, d, !clear_first, s);
}

extern "C" fgmp_status fgmp_linear_fused(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                         fgmp_scales sc, fgmp_score_mode sm, float tau, const void* packed_weights,
                                         void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                                         void* packed_acts_out, size_t packed_bytes,
                                         void* workspace, size_t ws_bytes, void* cuda_stream)
{
    if (!X_bf16 || !fisher_chan || !packed_weights || !Y || !workspace) return FGMP_ERR_INVALID_ARG;
    if ((int)sm < 0 || (int)sm > 1 || tau != tau) return FGMP_ERR_INVALID_ARG;
    if (!(sc.scale_fp4 > 0.f) || !isfinite(sc.scale_fp4)) return FGMP_ERR_INVALID_ARG;
    if (sc.fp8_log2_ratio < -7 || sc.fp8_log2_ratio > 7) return FGMP_ERR_INVALID_ARG;
    if (M < 1 || N < 1 || K < 64 || (K % 64) != 0 || ldy < N || ldx < K || (ldx % 8) != 0) return FGMP_ERR_SHAPE;
    if (((uintptr_t)X_bf16 & 15) || ((uintptr_t)fisher_chan & 15) || ((uintptr_t)packed_weights & 1023) ||
        ((uintptr_t)workspace & 1023) || ((uintptr_t)Y & 15) || ((uintptr_t)packed_acts_out & 1023)) return FGMP_ERR_SHAPE;
    if (ws_bytes < fgmp_ws_linear_fused(M, N, K)) return FGMP_ERR_WORKSPACE;
    if (packed_acts_out && packed_bytes < fgmp_layout(M, K, 0, 0).total) return FGMP_ERR_WORKSPACE;
    if (!fgmp_decode_supported(M, N, K)) {
        // larger batches: the two calls (the quantizer is then a small part of the step)
        if (!packed_acts_out) return FGMP_ERR_INVALID_ARG;
        fgmp_status st2 = fgmp_quantize_activations(X_bf16, ldx, fisher_chan, M, K, sc, sm, tau, packed_acts_out, packed_bytes,
                                                    nullptr, 0, cuda_stream);
        if (st2 != FGMP_OK) return st2;
        return fgmp_linear(packed_acts_out, packed_weights, Y, y_is_bf16, ldy, M, N, K, workspace, ws_bytes, cuda_stream);
    }
    fgmp_status st;
    if ((st = fgmp_require_sm100()) != FGMP_OK) return st;
    if ((st = set_attrs_once()) != FGMP_OK) return st;
    const DecPlan d = decode_plan(N, K);
    DecParams p = base_params(packed_weights, Y, y_is_bf16, ldy, M, N, K, workspace, d);
    p.X = (const uint8_t*)X_bf16; p.ldx = ldx; p.fisher = fisher_chan;
    // the same scalars, computed the same way, as fgmp_quantize_activations uses
    p.q.s4 = sc.scale_fp4;
    p.q.k6 = 1.0f / (6.0f * sc.scale_fp4);
    p.q.s8 = ldexpf(sc.scale_fp4, sc.fp8_log2_ratio);
    p.q.inv8 = 1.0f / p.q.s8;
    p.q.tau = tau; p.q.ratio = sc.fp8_log2_ratio; p.q.r8 = ldexpf(1.0f, sc.fp8_log2_ratio);
    p.q_mode = (int)sm;
    if (packed_acts_out) {
        uint8_t* blob = (uint8_t*)packed_acts_out;
        p.q_codes4 = blob + p.LA.off_codes4; p.q_sf = blob + p.LA.off_sf; p.q_mask = blob + p.LA.off_mask;
        p.q_codes8 = blob + p.LA.off_codes8; p.q_header = reinterpret_cast<fgmp_packed_header*>(blob);
        p.arec = blob + p.LA.off_arec;
    } else {
        p.arec = (uint8_t*)workspace + fgmp_align1k(fgmp_ws_decode(M, N, K));
    }
    return launch_decode<true>(p, d, true, (cudaStream_t)cuda_stream);
}

#ifdef FGMP_TIMELINE
extern "C" int fgmp_debug_timeline(unsigned long long* buffer)
{
    return cudaMemcpyToSymbol(g_timeline, &buffer, sizeof(buffer)) == cudaSuccess ? 0 : -4;
}
#endif

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
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_dec_mu);
        if (!scratch_of_device[dev]) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return FGMP_ERR_CUDA;
            scratch_of_device[dev] = ptr;
        }
        scratch = scratch_of_device[dev];
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the status word and the tile counters at the start of the scratch are zeroed first; the
    // partial sums behind them are always written before they are read
    st = fgmp_linear_decode(packed_acts, packed_weights, Y, y_is_bf16, ldy, M, N, K, scratch, true, s);
    if (st != FGMP_OK) return st;
    if (status_out && cudaMemcpyAsync(status_out, scratch, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return FGMP_ERR_CUDA;
    return FGMP_OK;
}
