// fgmp_linear for decode-sized batches (M <= 16 tokens): a weight-streaming kernel that
// reads the packed weights exactly once (Section 4.1 of the paper: the four block-pair
// products, FP32 accumulation), optionally with the activation quantizer of Section 4.2 in
// its prologue (fgmp_linear_fused).
//
// At this size the layer is bound by the weight stream.  Converting packed codes to a common number
// format in the SIMT pipes costs more instructions per byte than the stream leaves time for (an E2M1
// pair takes a byte extraction, a conversion and a scale multiply), so the bulk of the products must
// not be converted at all.  Decomposition (exact), with the FP8 blocks as the exceptions:
//   (1) NVFP4 weight block x NVFP4 activation block: tcgen05.mma kind::mxf4nvf4 straight from the
//       packed codes, E4M3 block scales in tensor memory, FP32 accumulation there; weights are the
//       128-row operand, the 16 tokens are N.  A block that must not take part gets a zero scale: the
//       record stores scale 0 for FP8 weight blocks, the activation record for FP8 activation blocks,
//       and the scales of every token are zeroed in "hot" block columns (those in which some token of
//       the batch is FP8), which are left to (3) as a whole.
//   (2) FP8 weight block x any activation block: mma.sync m16n8k16 on exact fp16 values (an E4M3 code
//       has 4 significant bits; the activation record holds every activation over its tensor scale in
//       fp16, exact for either format).  A record lists its FP8 blocks by block column, so sixteen
//       blocks that meet the same 16 activation elements form the M side; the sums are added to their
//       rows in a [row][token] tile private to the warp.
//   (3) NVFP4 weight block x any activation block in a hot column: the column's weights are dequantized
//       in registers (exact in fp16: 6 significant bits) for mma.sync, 32 rows per warp, sums in registers.
// Every block pair is in exactly one of the three.  With 10 % FP8 blocks that concentrate in few block
// columns (outlier channels) (2) and (3) are small; with unstructured activation masks (3) grows towards
// the whole tensor and the kernel is as fast as its SIMT conversions allow.
//
// Work is split stream-K style over (128-row tile, 256-element K chunk) units so that all SMs
// stream the same number of bytes; a unit is three bulk copies (its fixed-size record, the list of
// its FP8 blocks, the activation record of its chunk) into a ring of stages.  Tiles shared by several
// CTAs are reduced in a fixed order by the CTA that arrives last.  Every sum is taken in a fixed
// order: results are reproducible bit for bit.
//
// Warp roles (576 threads): warp 0 = producer, warp 1 = MMA issuer and owner of the tensor memory,
// warps 2-9 = (2): two sets of four warps that take alternate units, four block columns per warp (a warp
// copies what it needs of a unit into registers and gives the stage back at once), warps 10-13 = (3), 32
// rows each, warps 14-17 = block scales into tensor memory unit by unit and, at the end of a tile, the
// epilogue (one lane quadrant each).
#include "fgmp_common.cuh"
#include "fgmp_actq.cuh"
#include "fgmp_host.h"
#include "fgmp_ptx.cuh"
#include <cuda_fp16.h>
#include <mutex>
#include <type_traits>

namespace {

constexpr int DEC_WARPS = 18, DEC_THREADS = 32 * DEC_WARPS;
constexpr int W_PROD = 0, W_MMA = 1, W_FP8 = 2, W_HOT = 10, W_EPI = 14;
constexpr int FP8_WARPS = W_HOT - W_FP8;        // two sets of four: a set takes every second unit
constexpr int Q_THREADS = 32 * 16;              // warps 2..17 share out the prologue quantizer
constexpr int TOK = 16;                         // MMA N (token rows, zero padded)
constexpr uint32_t LIST_CAP = 3968;             // bytes of a unit's FP8 list that fit a stage (about 330 blocks); more is read from global
constexpr uint32_t STG_LIST = REC_BYTES;                                                         // 18560
constexpr uint32_t STG_A = STG_LIST + LIST_CAP;                                                  // 22528, 1 KiB aligned
constexpr uint32_t DEC_STAGE_BYTES = 33792;
constexpr int DEC_STAGES = 4;
constexpr int NTILES = FP8_WARPS + 1;           // [row][token] fp32 tiles: one per (2) warp, one shared by the (3) warps
constexpr uint32_t TILE_FLOATS = 128 * TOK;
constexpr uint32_t SF_COL0 = 32;                // tensor memory: 2 x 16 accumulator columns, then 32 scale columns per stage
constexpr uint32_t DEC_TMEM_COLS = 256;
constexpr size_t DEC_SMEM = (size_t)DEC_STAGES * DEC_STAGE_BYTES + NTILES * TILE_FLOATS * 4 + 1024 /*alignment*/ + 512 /*barriers*/;
static_assert(STG_A % 1024 == 0 && STG_A + AREC_BYTES <= DEC_STAGE_BYTES, "stage layout");
static_assert(DEC_SMEM <= 232448, "shared memory of one CTA");
static_assert(SF_COL0 + 32 * DEC_STAGES <= DEC_TMEM_COLS, "tensor memory columns");

// kind::mxf4nvf4, E2M1 x E2M1, UE4M3 scales, K-major operands, M = 128, N = 16, dense K = 64
constexpr uint32_t IDESC_NVF4 = (1u << 7) | (1u << 10) | ((uint32_t)(TOK >> 3) << 17) | (0u << 23) | ((uint32_t)(128 >> 4) << 24);

// shared-memory matrix descriptors as (low word | start address >> 4, constant high word)
constexpr uint32_t SW128_LO = 1u << 16, SW128_HI = (1024u >> 4) | (1u << 14) | (2u << 29);   // 128B swizzle, 8-row groups 1 KiB apart
__device__ __forceinline__ uint64_t desc64(uint32_t lo, uint32_t hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}

// control words of the workspace (int32, from byte 256): see fgmp_linear_fused
enum { CW_DONE = 1, CW_CLAIM = 2, CW_QCOUNT = 3, CW_QREADY = 4 };

struct DecParams {
    const uint8_t* wblob; const uint8_t* ablob;
    PackedLayout LW, LA;
    float* Y; void* Ybf; int64_t ldy; int y_is_bf16;
    int64_t M, N, K;
    int64_t total;            // tiles * chunks
    int64_t chunks;
    int* status; uint32_t* counters; float* partials; int maxseg;
    // activation quantizer in the prologue (fused launches only)
    const uint8_t* X; int64_t ldx;        // bf16 [M, ldx]
    const float* fisher;
    ActQuantScalars q; int q_mode;        // q_mode: fgmp_score_mode
    uint8_t* arec;                        // where the records of the chunks go (and are streamed from)
    uint8_t* q_codes4; uint8_t* q_sf; uint8_t* q_mask; uint8_t* q_codes8; fgmp_packed_header* q_header;   // optional packed output
    uint32_t* cw;                         // control words
};

struct StageMeta { uint32_t step, staged; };     // list start (16-byte steps), bytes of it in the stage

// Profiling builds (-DFGMP_TIMELINE) stamp the global timer at the phases of every CTA into a buffer
// registered with fgmp_debug_timeline (16 x uint64 per CTA); ordinary builds contain none of this.
#ifdef FGMP_TIMELINE
__device__ unsigned long long* g_timeline = nullptr;
#define FGMP_STAMP_ANY(slot) do { if (g_timeline) g_timeline[(size_t)blockIdx.x * 16 + (slot)] = globaltimer_ns(); } while (0)
#else
#define FGMP_STAMP_ANY(slot) do { } while (0)
#endif

__device__ __forceinline__ int64_t cta_of_unit(int64_t i, int64_t G, int64_t total) { return ((i + 1) * G - 1) / total; }

__device__ __forceinline__ void quant_bar() { asm volatile("bar.sync 1, %0;" ::"n"(Q_THREADS) : "memory"); }

// A correction tile holds [128 rows][16 tokens] fp32, a row = 64 bytes = four 16-byte pieces of
// four tokens; piece index is XOR-ed with (row >> 1) & 3 so that 32 lanes reading one piece of 32
// consecutive rows (the epilogue) do not collide on banks.  Float index of (row, token):
__device__ __forceinline__ uint32_t tile_idx(uint32_t row, uint32_t token)
{
    return row * 16u + ((((token >> 2) ^ (row >> 1)) & 3u) << 2) + (token & 3u);
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

// One work item of the prologue quantizer: chunk c (256 elements) of the eight token rows of octet o.  Run by
// the 16 warps 2..17: warp wq takes token 8o + wq/2 and the eight blocks 8(wq%2) .. +7 of the chunk, four lanes
// per block.  s_hot: one word of shared memory.  Each octet has its own word for the chunk's hot block columns.
template <int MODE>
__device__ __forceinline__ void quantize_chunk(const DecParams& p, int64_t c, int o, uint32_t* s_hot)
{
    const uint32_t tq = threadIdx.x - 64u;                 // index among the quantizer's threads
    const uint32_t wq = tq >> 5, lane = tq & 31u, li = lane & 3u;
    const uint32_t j = 8u * (wq & 1u) + (lane >> 2);
    const int64_t kb = 16 * c + j;
    uint8_t* rec = p.arec + (size_t)c * AREC_BYTES;
    if (tq == 0) *s_hot = 0u;
    quant_bar();
    const uint32_t m = 8u * (uint32_t)o + (wq >> 1);
    const bool live = (int64_t)m < p.M;
    uint2 xin = make_uint2(0u, 0u);
    float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) {
        xin = __ldg(reinterpret_cast<const uint2*>(p.X + ((size_t)m * p.ldx + (size_t)kb * 16 + 4 * li) * 2));
        f = __ldg(reinterpret_cast<const float4*>(p.fisher + kb * 16 + 4 * li));
    }
    {
        uint8_t* a4 = rec + AREC_A4 + fgmp_rec_w4_offset(m, j) + 2u * li;
        uint8_t* at = rec + fgmp_arec_at_offset(m, j) + 8u * li;
        if (!live) {                                        // token rows beyond the batch are zero
            *reinterpret_cast<uint16_t*>(a4) = 0;
            *reinterpret_cast<uint2*>(at) = make_uint2(0u, 0u);
            if (li == 0) rec[AREC_SF + m * 16u + j] = 0;
        } else {
        const BlockQuarter r = quantize_block_quarter<MODE>(xin, f, p.q);
        *reinterpret_cast<uint16_t*>(a4) = (uint16_t)r.c4;
        *reinterpret_cast<uint2*>(at) = r.h;
        if (li == 0) rec[AREC_SF + m * 16u + j] = (uint8_t)r.sc;
        const uint32_t bal = __ballot_sync(0xffffffffu, r.is8 && li == 0);
        uint32_t byte = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) byte |= ((bal >> (4 * b)) & 1u) << b;
        if (lane == 0 && byte) atomicOr(s_hot, byte << (8u * (wq & 1u)));
        if (p.q_codes4) {
            const int64_t MW = p.LA.MW;
            *reinterpret_cast<uint16_t*>(p.q_codes4 + ((int64_t)m * p.K) / 2 + kb * 8 + li * 2) = (uint16_t)r.c4;
            if (li == 0) p.q_sf[fgmp_sf_offset(m, kb, p.K)] = (uint8_t)r.sc;
            if (r.is8) *reinterpret_cast<uint32_t*>(p.q_codes8 + (int64_t)m * p.K + kb * 16 + 4 * li) = r.c8;
            if (lane == 0) {
                uint8_t* mb = p.q_mask + (size_t)m * MW * 4 + (kb >> 3);    // lane 0: first block of the warp's eight
                mb[0] = (uint8_t)byte;
                if (kb + 8 == p.LA.KB && (p.LA.KB & 31) != 0) { mb[1] = 0; mb[2] = 0; }   // rest of the row's last mask word
            }
        }
        }
    }
    quant_bar();
    if (tq == 0) reinterpret_cast<uint32_t*>(rec + AREC_HOT)[o] = *s_hot;
}

// NH = token octets in use: 1 for M <= 8, else 2.  FUSED: the activation quantizer runs in the prologue.
template <int NH, bool FUSED>
__global__ void __launch_bounds__(DEC_THREADS, 1)
decode_kernel(DecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    // 1 KiB aligned; an offset from the array keeps the pointer known to be shared memory (plain ld.shared / st.shared)
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int S = DEC_STAGES;
    float* tiles = reinterpret_cast<float*>(smem + (size_t)S * DEC_STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + NTILES * TILE_FLOATS);
    // bars: [0,S) full, [S,2S) empty, [2S,3S) scales in tensor memory, then acc_full[2], acc_empty[2],
    // corrections of a segment done [2], tiles free [1]
    StageMeta* smeta = reinterpret_cast<StageMeta*>(bars + 3 * S + 8);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smeta + S);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* s_misc = reinterpret_cast<volatile uint32_t*>(abort_flag + 1);   // [1..2] claimed item, [3] hot columns of a chunk

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) FGMP_STAMP_ANY(0);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * S, sfr0 = empty0 + 8 * S;
    const uint32_t accf0 = sfr0 + 8 * S, acce0 = accf0 + 16, cdone0 = acce0 + 16, tfree = cdone0 + 16;
    constexpr uint32_t A_BYTES = NH == 2 ? AREC_BYTES : AREC_AT + 4096u;

    // this CTA's span of (tile, chunk) units
    const int64_t G = gridDim.x, C = p.chunks;
    const int64_t u_begin = ((int64_t)blockIdx.x * p.total) / G, u_end = ((int64_t)(blockIdx.x + 1) * p.total) / G;
    const uint32_t* uptr = reinterpret_cast<const uint32_t*>(p.wblob + p.LW.off_uptr);
    const uint8_t* recs = p.wblob + p.LW.off_rec;
    const uint8_t* lists = p.wblob + p.LW.off_ovf;
    const uint8_t* arec = FUSED ? p.arec : p.ablob + p.LA.off_arec;

    // One unit's copies into a stage (lane 0 of the producer warp): record and list, then the
    // activation record of the unit's chunk
    auto issue_w = [&](int64_t u, int stage, uint32_t step0, uint32_t step1) {
        const uint32_t bytes = (step1 - step0) * 16u;
        const uint32_t staged = bytes < LIST_CAP ? bytes : LIST_CAP;
        smeta[stage].step = step0; smeta[stage].staged = staged;
        const uint32_t fb = full0 + 8 * stage;
        const uint32_t dst = smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES);
        mbar_expect_tx(fb, REC_BYTES + staged + A_BYTES);
        bulk_load(dst, recs + (size_t)u * REC_BYTES, REC_BYTES, fb);
        if (staged) bulk_load(dst + STG_LIST, lists + (size_t)step0 * 16, staged, fb);
    };
    auto issue_a = [&](int64_t u, int stage) {
        bulk_load(smem_u32(smem + (size_t)stage * DEC_STAGE_BYTES) + STG_A, arec + (size_t)(u % C) * AREC_BYTES, A_BYTES, full0 + 8 * stage);
    };

    // ------------------------------------------------------------ set-up.  The packed weights are not written by
    // whatever runs before this kernel, so the producer's part (barriers, the weight blob's header, the first
    // stages' weight copies) may overlap the end of that kernel (programmatic dependent launch).
    int64_t pf_base = u_begin;
    uint32_t pf = 0;
    int pre = 0;
    if (warp == W_PROD) {
        if (lane == 0) {
            for (int s = 0; s < S; ++s) {
                mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1 + 8); mbar_init(sfr0 + 8 * s, 4);
            }
            for (int b = 0; b < 2; ++b) {
                mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 128); mbar_init(cdone0 + 8 * b, FP8_WARPS + 4);
            }
            mbar_init(tfree, 4);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        // nothing is read through the blob's tables before its header has been seen to describe this call
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        int okh = 1;
        if (lane == 0) {
            const uint2 mv = __ldg(reinterpret_cast<const uint2*>(hw));
            okh = mv.x == FGMP_MAGIC && mv.y == 7u && __ldg(&hw->rows) == p.N && __ldg(&hw->K) == p.K &&
                  __ldg(&hw->kind) == 1u && __ldg(&hw->error) == 0 && __ldg(&hw->fp8_scale_free) == 0;
            if (!okh) { *abort_flag = 1; atomicCAS(p.status, 0, (int)FGMP_ERR_INVALID_ARG); atomicExch(p.status + 1, 9); }
        }
        okh = __shfl_sync(0xffffffffu, okh, 0);
        if (okh) {
            if (pf_base + lane <= p.total) pf = __ldg(uptr + pf_base + lane);
            pre = (int)min((int64_t)S, u_end - u_begin);
            for (int s = 0; s < pre; ++s) {
                const uint32_t step0 = __shfl_sync(0xffffffffu, pf, s), step1 = __shfl_sync(0xffffffffu, pf, s + 1);
                if (lane == 0) issue_w(u_begin + s, s, step0, step1);
            }
        }
    }
    if (warp == W_MMA) tmem_alloc(smem_u32(tmem_slot), DEC_TMEM_COLS);
    if (warp >= W_FP8 && warp < W_EPI) {               // the tiles start at zero
        float4* z = reinterpret_cast<float4*>(tiles);
        for (int i = (warp - W_FP8) * 32 + lane; i < (int)(NTILES * TILE_FLOATS / 4); i += (W_EPI - W_FP8) * 32) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) FGMP_STAMP_ANY(1);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Launched as a programmatic dependent of the preceding kernel in the stream, this kernel may have
    // started before that one finished: everything above touches neither its output nor the workspace.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0) FGMP_STAMP_ANY(2);
    if (FUSED) {
        // the first of the quantizer's work items is asked for right away
        if (threadIdx.x == 64 && !*abort_flag) s_misc[1] = atomicInc(p.cw + CW_CLAIM, 2u * (uint32_t)C + (uint32_t)G - 1u);
        __syncthreads();
    }
    const bool dead = *abort_flag != 0;                // the weight blob does not belong to this call: nothing else is read

    if (FUSED && !dead && warp >= W_FP8) {
        // The quantizer's work items (chunks) are handed out through a counter, so that every item is taken by
        // a CTA that is running: no CTA ever waits for one that has not started.  The counter and the count of
        // finished items wrap to zero with the call's last access.
        const uint32_t n_items = 2u * (uint32_t)C;          // (chunk, token octet)
        for (uint32_t it = 0;; ++it) {
            const uint32_t item = s_misc[1 + (it & 1u)];
            if (item >= n_items) break;
            // the next item is asked for while this one is worked on
            if (threadIdx.x == 64) s_misc[1 + ((it + 1u) & 1u)] = atomicInc(p.cw + CW_CLAIM, n_items + (uint32_t)G - 1u);
            if (item == 0 && threadIdx.x == 64 && p.q_header) {
                fgmp_packed_header* h = p.q_header;
                h->magic = FGMP_MAGIC; h->version = 7; h->rows = p.M; h->K = p.K; h->scale_fp4 = p.q.s4;
                h->fp8_log2_ratio = p.q.ratio; h->n_fp8 = (p.q.tau == INFINITY) ? 0 : -1; h->tau_eff = 0.f; h->kind = 0; h->capacity = 0;
                h->error = 0; h->scale_fp8 = p.q.s8; h->fp8_scale_free = 0;
            }
            if (p.q_mode == 0) quantize_chunk<0>(p, (int64_t)(item >> 1), (int)(item & 1u), const_cast<uint32_t*>(s_misc + 3));
            else               quantize_chunk<1>(p, (int64_t)(item >> 1), (int)(item & 1u), const_cast<uint32_t*>(s_misc + 3));
            // The item's stores become visible with the counter: the barrier orders them before the one thread's
            // release, and the last arrival's acquire sees every earlier release of the counter.
            quant_bar();
            if (threadIdx.x == 64) {
                uint32_t old;
                asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.cw + CW_QCOUNT), "r"(n_items - 1u) : "memory");
                if (old == n_items - 1u)
                    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.cw + CW_QREADY), "r"(1u) : "memory");
            }
        }
    }

    if (threadIdx.x == 64) FGMP_STAMP_ANY(3);          // this CTA's share of the quantizer is done
    if (dead) {
    } else if (warp == W_PROD) {
        // ------------------------------------------------------------ producer (whole warp; lane 0 issues)
        int ok = 1;
        if (lane == 0) {
            if (FUSED) {
                // every chunk's record is in place once the last work item of the quantizer has been handed in
                ok = wait_global_equals(p.cw + CW_QREADY, 1u, abort_flag, p.status, 8) ? 1 : 0;
                asm volatile("fence.proxy.async;" ::: "memory");   // records were written with ordinary stores, the bulk copy reads them
            } else {
                const fgmp_packed_header* ha = reinterpret_cast<const fgmp_packed_header*>(p.ablob);
                const uint2 mv = __ldg(reinterpret_cast<const uint2*>(ha));
                if (!(mv.x == FGMP_MAGIC && mv.y == 7u && __ldg(&ha->rows) == p.M && __ldg(&ha->K) == p.K && __ldg(&ha->kind) == 0u && __ldg(&ha->fp8_scale_free) == 0)) {
                    *abort_flag = 1; atomicCAS(p.status, 0, (int)FGMP_ERR_INVALID_ARG); atomicExch(p.status + 1, 10);
                    ok = 0;
                }
            }
            if (ok) for (int s = 0; s < pre; ++s) issue_a(u_begin + s, s);
            FGMP_STAMP_ANY(4);                         // all activation records are in place
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        int stage = pre % S; uint32_t phase = (uint32_t)(pre / S) & 1u;
        for (int64_t u = u_begin + pre; u < u_end && ok; ++u) {
            if (u + 1 - pf_base > 31) {                // next 32 list starts
                pf_base = u;
                pf = (pf_base + lane <= p.total) ? __ldg(uptr + pf_base + lane) : 0u;
            }
            const uint32_t step0 = __shfl_sync(0xffffffffu, pf, (int)(u - pf_base));
            const uint32_t step1 = __shfl_sync(0xffffffffu, pf, (int)(u + 1 - pf_base));
            if (lane == 0) {
                ok = mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1) ? 1 : 0;  /*lane*/
                if (ok) { issue_w(u, stage, step0, step1); issue_a(u, stage); }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (++stage == S) { stage = 0; phase ^= 1; }
        }
    } else if (warp == W_MMA) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop; lane 0 alone issues the tcgen05 instructions, so that every
        // commit tracks every MMA before it.
        const uint32_t smem0 = smem_u32(smem);
        int stage = 0; uint32_t phase = 0; bool ok = true;
        int seg = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_end = min(u_end, (tile + 1) * C);
            const int acc = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            if (!(ok = mbar_wait_warp(acce0 + 8 * acc, acc_phase ^ 1, abort_flag, p.status, 2))) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TOK);
            uint32_t accum = 0;
            for (; u < seg_end && ok; ++u) {
                if (!(ok = mbar_wait_warp(full0 + 8 * stage, phase, abort_flag, p.status, 3))) break;
                if (!(ok = mbar_wait_warp(sfr0 + 8 * stage, phase, abort_flag, p.status, 8))) break;   // the scales are in tensor memory
                if (u == u_begin && lane == 0) FGMP_STAMP_ANY(5);
                if (u == u_end - 1 && lane == 0) FGMP_STAMP_ANY(6);
                tc_fence_after();
                const uint32_t sb = smem0 + (uint32_t)stage * DEC_STAGE_BYTES;
                const uint32_t sf_t = tmem_base + SF_COL0 + (uint32_t)stage * 32;   // [0,16) weights, [16,32) tokens
                const uint32_t w4_lo = ((sb + REC_W4) >> 4) | SW128_LO, a4_lo = ((sb + STG_A + AREC_A4) >> 4) | SW128_LO;
                if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        umma_nvf4(d_tmem, desc64(w4_lo + 2 * j, SW128_HI), desc64(a4_lo + 2 * j, SW128_HI), IDESC_NVF4,
                                  sf_t + 4 * j, sf_t + 16 + 4 * j, accum);
                        accum = 1;
                    }
                    umma_commit(empty0 + 8 * stage);
                }
                accum = 1;
                __syncwarp();
                if (++stage == S) { stage = 0; phase ^= 1; }
            }
            if (ok && lane == 0) umma_commit(accf0 + 8 * acc);
            __syncwarp();
        }
    } else if (warp < W_HOT) {
        // ------------------------------------------------------------ (2): FP8 weight blocks of block columns bq, bq+4, bq+8, bq+12
        // of every second unit.  The E4M3 codes go into the MMA as they are; the factor 2^ratio between the
        // FP8 and NVFP4 tensor scales is applied once to the tile sums in the epilogue.
        const int bq = (warp - W_FP8) & 3, par = (warp - W_FP8) >> 2;
        const uint32_t g = lane >> 2, t = lane & 3;
        float* mytile = tiles + (warp - W_FP8) * TILE_FLOATS;
        const uint32_t tcol = (2 * t) & 3u, tpiece = t >> 1;
        // tile[row][tokens] += sums of one group.  Within one column every block has its own row, so the
        // read-modify-writes of a group touch distinct addresses: all loads first, then all stores.
        // (tlA, tlB: the rows' places in the tile as the list gives them, 0xffff = no block)
        const uint32_t tx = tpiece << 2;
        auto group_add = [&](const float (&c)[4], const float (&d)[4], uint32_t tlA, uint32_t tlB) {
            const uint32_t iA = (tlA ^ tx) + tcol, iB = (tlB ^ tx) + tcol;      // tokens 2t, 2t+1; tokens 8+2t, 9+2t are 8 floats on
            float2 vA0 = make_float2(0.f, 0.f), vA1 = vA0, vB0 = vA0, vB1 = vA0;
            if (tlA != 0xffffu) {
                vA0 = *reinterpret_cast<const float2*>(mytile + iA);
                if (NH == 2) vA1 = *reinterpret_cast<const float2*>(mytile + (iA ^ 8u));
            }
            if (tlB != 0xffffu) {
                vB0 = *reinterpret_cast<const float2*>(mytile + iB);
                if (NH == 2) vB1 = *reinterpret_cast<const float2*>(mytile + (iB ^ 8u));
            }
            if (tlA != 0xffffu) {
                *reinterpret_cast<float2*>(mytile + iA) = make_float2(vA0.x + c[0], vA0.y + c[1]);
                if (NH == 2) *reinterpret_cast<float2*>(mytile + (iA ^ 8u)) = make_float2(vA1.x + d[0], vA1.y + d[1]);
            }
            if (tlB != 0xffffu) {
                *reinterpret_cast<float2*>(mytile + iB) = make_float2(vB0.x + c[2], vB0.y + c[3]);
                if (NH == 2) *reinterpret_cast<float2*>(mytile + (iB ^ 8u)) = make_float2(vB1.x + d[2], vB1.y + d[3]);
            }
            __syncwarp();                  // a later group may add to the same rows
        };
        // blocks iA = e + g and iB = e + g + 8 of a group as the M side of the mma.sync (tokens 0-7 and 8-15 as N);
        // c/d[0..1]: block iA, tokens 2t, 2t+1 / 8+2t, 9+2t; [2..3]: block iB
        auto group_mma = [&](uint32_t rawA, uint32_t rawB, const uint2& bt0, const uint2& bt1, float (&c)[4], float (&d)[4]) {
            uint32_t a0, a1, a2, a3;
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a0) : "h"((uint16_t)rawA));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a2) : "h"((uint16_t)(rawA >> 16)));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a1) : "h"((uint16_t)rawB));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(a3) : "h"((uint16_t)(rawB >> 16)));
            c[0] = c[1] = c[2] = c[3] = 0.f; d[0] = d[1] = d[2] = d[3] = 0.f;
            mma_f16_16816(c, a0, a1, a2, a3, bt0.x, bt0.y);
            if (NH == 2) mma_f16_16816(d, a0, a1, a2, a3, bt1.x, bt1.y);
        };

        bool ok = true;
        int seg = 0;
        const int n_units = (int)(u_end - u_begin);
        for (int sbeg = 0; sbeg < n_units && ok; ++seg) {
            const int64_t tile = (u_begin + sbeg) / C;
            const int send = (int)min((int64_t)n_units, (tile + 1) * C - u_begin);
            // the epilogue has taken (and cleared) the previous segment's sums
            if (seg > 0 && !(ok = mbar_wait_warp(tfree, (uint32_t)(seg - 1) & 1u, abort_flag, p.status, 7))) break;
            for (int i = sbeg + ((par ^ sbeg) & 1); i < send; i += 2) {
                const int stage = i % S; const uint32_t phase = (uint32_t)(i / S) & 1u;
                if (!(ok = mbar_wait_warp(full0 + 8 * stage, phase, abort_flag, p.status, 5))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint8_t* sa = sb + STG_A;
                const uint32_t staged = smeta[stage].staged;
                const uint8_t* list_g = lists + (size_t)smeta[stage].step * 16;
                const uint16_t* kbs = reinterpret_cast<const uint16_t*>(sb + REC_KBSTART);
                const uint32_t ntot = kbs[16];
                const uint32_t hoff = fgmp_list_halves_offset(ntot);
                const bool all = hoff + ntot * 8 <= staged;        // the whole list is in the stage (the usual case)
                uint32_t st[4], en[4], rowA[8], rowB[8], rawA[8], rawB[8];     // [4 gr + cc]: group gr (blocks 16 gr ..) of column cc
                uint2 bt0[4], bt1[4];
                bool plain = all;                                  // ... and no column has more than two groups of 16
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const uint32_t j = (uint32_t)bq + 4u * cc;
                    st[cc] = kbs[j]; en[cc] = kbs[j + 1];
                    plain = plain && (en[cc] - st[cc] <= 32u);
                    bt0[cc] = *reinterpret_cast<const uint2*>(sa + fgmp_arec_at_offset(g, j) + 8 * t);
                    bt1[cc] = make_uint2(0u, 0u);
                    if (NH == 2) bt1[cc] = *reinterpret_cast<const uint2*>(sa + fgmp_arec_at_offset(g + 8, j) + 8 * t);
                }
                if (plain) {
                    // Everything the four columns need, into registers.  Lane t has elements 4t .. 4t+3 of a block:
                    // from its slot in the record (t < 2) or from the list (t >= 2).
#pragma unroll
                    for (int gr = 0; gr < 2; ++gr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            const uint32_t iA = st[cc] + 16u * gr + g, iB = iA + 8;
                            const bool hasA = iA < en[cc], hasB = iB < en[cc];
                            const uint32_t mA = hasA ? *reinterpret_cast<const uint32_t*>(sb + STG_LIST + 4 * iA) : 0xffffffffu;
                            const uint32_t mB = hasB ? *reinterpret_cast<const uint32_t*>(sb + STG_LIST + 4 * iB) : 0xffffffffu;
                            const uint32_t oA = t < 2 ? REC_W4 + (mA & 0xffffu) + 4 * t : STG_LIST + hoff + iA * 8 + 4 * (t - 2);
                            const uint32_t oB = t < 2 ? REC_W4 + (mB & 0xffffu) + 4 * t : STG_LIST + hoff + iB * 8 + 4 * (t - 2);
                            rawA[4 * gr + cc] = hasA ? *reinterpret_cast<const uint32_t*>(sb + oA) : 0u;
                            rawB[4 * gr + cc] = hasB ? *reinterpret_cast<const uint32_t*>(sb + oB) : 0u;
                            rowA[4 * gr + cc] = mA >> 16;
                            rowB[4 * gr + cc] = mB >> 16;
                        }
                } else {
                    // a list that does not fit the stage, or a column with more than 32 FP8 blocks (rare): group by
                    // group straight from the stage or from global memory, before the stage is given back
                    auto fetch = [&](uint32_t i_, uint32_t& row, uint32_t& raw) {
                        const uint32_t m_ = (all || 4 * i_ + 4 <= staged) ? *reinterpret_cast<const uint32_t*>(sb + STG_LIST + 4 * i_)
                                                                          : __ldg(reinterpret_cast<const uint32_t*>(list_g + 4 * i_));
                        row = m_ >> 16;
                        if (t < 2) {
                            raw = *reinterpret_cast<const uint32_t*>(sb + REC_W4 + (m_ & 0xffffu) + 4 * t);
                        } else {
                            const uint32_t o = hoff + i_ * 8 + 4 * (t - 2);
                            raw = (all || o + 4 <= staged) ? *reinterpret_cast<const uint32_t*>(sb + STG_LIST + o)
                                                           : __ldg(reinterpret_cast<const uint32_t*>(list_g + o));
                        }
                    };
#pragma unroll 1
                    for (int cc = 0; cc < 4; ++cc) {
                        const uint32_t j = (uint32_t)bq + 4u * cc;
                        const uint32_t st_ = kbs[j], en_ = kbs[j + 1];
                        const uint2 b0 = *reinterpret_cast<const uint2*>(sa + fgmp_arec_at_offset(g, j) + 8 * t);
                        uint2 b1 = make_uint2(0u, 0u);
                        if (NH == 2) b1 = *reinterpret_cast<const uint2*>(sa + fgmp_arec_at_offset(g + 8, j) + 8 * t);
                        for (uint32_t e = st_; e < en_; e += 16) {
                            uint32_t rA = 0xffffu, rB = 0xffffu, wA = 0u, wB = 0u;
                            if (e + g < en_) fetch(e + g, rA, wA);
                            if (e + g + 8 < en_) fetch(e + g + 8, rB, wB);
                            float c[4], d[4];
                            group_mma(wA, wB, b0, b1, c, d);
                            group_add(c, d, rA, rB);
                        }
                    }
                }
                // the stage is no longer needed
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (plain) {
#pragma unroll
                    for (int gr = 0; gr < 2; ++gr)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) {
                            if (gr == 1 && en[cc] - st[cc] <= 16u) continue;      // (the same for every lane)
                            float c[4], d[4];
                            group_mma(rawA[4 * gr + cc], rawB[4 * gr + cc], bt0[cc], bt1[cc], c, d);
                            group_add(c, d, rowA[4 * gr + cc], rowB[4 * gr + cc]);
                        }
                }
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) mbar_arrive(cdone0 + 8 * (seg & 1));
            sbeg = send;
        }
    } else if (warp < W_EPI) {
        // ------------------------------------------------------------ (3): hot block columns, rows 32jr .. 32jr+31
        // Lane (g, t) has elements 4t .. 4t+3 of the column's block in rows 32jr + 16mt + {g, g + 8}: two code
        // bytes and the block's microscale (zero for an FP8 weight block, which (2) covers).
        const uint32_t jr = (uint32_t)(warp - W_HOT);
        const uint32_t g = lane >> 2, t = lane & 3;
        float* tile3 = tiles + FP8_WARPS * TILE_FLOATS;
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
                if (!(ok = mbar_wait_warp(full0 + 8 * stage, phase, abort_flag, p.status, 6))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint8_t* sa = sb + STG_A;
                const uint2 hw2 = *reinterpret_cast<const uint2*>(sa + AREC_HOT);      // one word per token octet
                const uint32_t hot = hw2.x | hw2.y;
                uint32_t todo = hot & 0xffffu;
                while (todo) {
                    const uint32_t j = (uint32_t)__ffs(todo) - 1u;
                    todo &= todo - 1;
                    uint2 b[NH];
#pragma unroll
                    for (int nh = 0; nh < NH; ++nh) b[nh] = *reinterpret_cast<const uint2*>(sa + fgmp_arec_at_offset(g + 8 * nh, j) + 8 * t);
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        uint32_t x[2][2];
#pragma unroll
                        for (int rh = 0; rh < 2; ++rh) {
                            const uint32_t r = 32 * jr + 16 * (uint32_t)mt + 8 * (uint32_t)rh + g;
                            const uint32_t codes = *reinterpret_cast<const uint16_t*>(sb + REC_W4 + fgmp_rec_w4_offset(r, j) + 2 * t);
                            const uint32_t sfb = sb[REC_SF + fgmp_rec_sf_offset(r, j)];
                            uint32_t q0, q1, sc2;
                            // (one byte at a time: unpacking a word into byte registers of which only some are used
                            // gave wrong values on this toolchain)
                            asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(q0) : "r"(codes & 0xffu));
                            asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(q1) : "r"(codes >> 8));
                            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(sc2) : "h"((uint16_t)(sfb | (sfb << 8))));
                            asm("mul.f16x2 %0, %1, %2;" : "=r"(x[rh][0]) : "r"(q0), "r"(sc2));
                            asm("mul.f16x2 %0, %1, %2;" : "=r"(x[rh][1]) : "r"(q1), "r"(sc2));
                        }
#pragma unroll
                        for (int nh = 0; nh < NH; ++nh) mma_f16_16816(acc[mt][nh], x[0][0], x[1][0], x[0][1], x[1][1], b[nh].x, b[nh].y);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * stage);
                if (++stage == S) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            // the epilogue has taken the previous segment's sums; now this segment's go in:
            // acc[mt][nh] = rows 32jr + 16mt + {g, g + 8} x tokens 8nh + {2t, 2t+1}
            if (seg > 0 && !(ok = mbar_wait_warp(tfree, (uint32_t)(seg - 1) & 1u, abort_flag, p.status, 7))) break;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) {
                    const uint32_t r = 32 * jr + 16 * (uint32_t)mt + g, m = 8 * (uint32_t)nh + 2 * t;
                    tile3[tile_idx(r, m)] = acc[mt][nh][0];
                    tile3[tile_idx(r, m + 1)] = acc[mt][nh][1];
                    tile3[tile_idx(r + 8, m)] = acc[mt][nh][2];
                    tile3[tile_idx(r + 8, m + 1)] = acc[mt][nh][3];
                }
            __syncwarp();
            if (lane == 0) mbar_arrive(cdone0 + 8 * (seg & 1));
        }
    } else {
        // ------------------------------------------------------------ epilogue: tensor-memory lane quadrant warp % 4
        const int q = warp & 3;
        const fgmp_packed_header* hw = reinterpret_cast<const fgmp_packed_header*>(p.wblob);
        const float s4a = FUSED ? p.q.s4 : __ldg(&reinterpret_cast<const fgmp_packed_header*>(p.ablob)->scale_fp4);
        const float alpha = __fmul_rn(s4a, __ldg(&hw->scale_fp4));
        const float r8 = __int_as_float((127 + __ldg(&hw->fp8_log2_ratio)) << 23);     // FP8 tensor scale / NVFP4 tensor scale of the weights
        const int row = 32 * q + lane;
        bool ok = true;
        int seg = 0;
        int stage = 0; uint32_t phase = 0;
        for (int64_t u = u_begin; u < u_end && ok; ++seg) {
            const int64_t tile = u / C;
            const int64_t seg_begin = u, seg_end = min(u_end, (tile + 1) * C);
            // Block scales of the segment's units into tensor memory, lane quadrant warp % 4: lane i holds, for MMA
            // step j, the four scale bytes of rows i, 32+i, 64+i, 96+i in columns 4j..4j+3 -- 16 bytes of scale tile j
            // of the record; the token scales follow in columns 16..31 (16 tokens: lanes 0..15, first column of
            // every step), zeroed in the chunk's hot block columns.
            for (; u < seg_end; ++u) {
                if (!(ok = mbar_wait_warp(full0 + 8 * stage, phase, abort_flag, p.status, 4))) break;
                const uint8_t* sb = smem + (size_t)stage * DEC_STAGE_BYTES;
                const uint8_t* sa = sb + STG_A;
                const uint2 hw2 = *reinterpret_cast<const uint2*>(sa + AREC_HOT);      // one word per token octet
                const uint32_t hot = hw2.x | hw2.y;
                uint32_t r[16];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 x = *reinterpret_cast<const uint4*>(sb + REC_SF + 512 * j + lane * 16);
                    r[4 * j] = x.x; r[4 * j + 1] = x.y; r[4 * j + 2] = x.z; r[4 * j + 3] = x.w;
                }
                const uint32_t sf_t = tmem_base + ((uint32_t)(q * 32) << 16) + SF_COL0 + (uint32_t)stage * 32;
                tmem_st16(sf_t, r);
                const uint4 ts = *reinterpret_cast<const uint4*>(sa + AREC_SF + (lane & 15) * 16);
                const uint32_t tsw[4] = {ts.x, ts.y, ts.z, ts.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // bits 4j .. 4j+3 of the cold columns spread to the four bytes of the step's scale word
                    const uint32_t keep = ((((~hot >> (4 * j)) & 0xfu) * 0x00204081u) & 0x01010101u) * 0xffu;
                    r[4 * j] = lane < 16 ? (tsw[j] & keep) : 0u;
                    r[4 * j + 1] = 0u; r[4 * j + 2] = 0u; r[4 * j + 3] = 0u;
                }
                tmem_st16(sf_t + 16, r);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(sfr0 + 8 * stage);
                if (++stage == S) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            const int accb = seg & 1; const uint32_t acc_phase = (uint32_t)((seg >> 1) & 1);
            if (!(ok = mbar_wait_warp(accf0 + 8 * accb, acc_phase, abort_flag, p.status, 11))) break;
            tc_fence_after();
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
            uint32_t rr[16];
            tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(accb * TOK), rr);
            tc_fence_before();
            mbar_arrive(acce0 + 8 * accb);
            float v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(rr[j]);
            // corrections (2) and (3) of the segment: this row of every tile, in tile order; the rows of (2)
            // are cleared for the next segment on the way
            if (!(ok = mbar_wait_warp(cdone0 + 8 * accb, acc_phase, abort_flag, p.status, 12))) break;
            float c2[16];                              // (2): sums of the FP8 weight codes, still without 2^ratio
#pragma unroll
            for (int j = 0; j < 16; ++j) c2[j] = 0.f;
#pragma unroll
            for (int w = 0; w < NTILES; ++w) {
                float4* src = reinterpret_cast<float4*>(tiles + w * TILE_FLOATS + row * TOK);
                float4 x[4];
#pragma unroll
                for (int j = 0; j < 2 * NH; ++j) x[j] = src[(j ^ (row >> 1)) & 3];       // tokens 4j .. 4j+3
#pragma unroll
                for (int j = 0; j < 2 * NH; ++j) {
                    if (w < FP8_WARPS) { c2[4 * j] += x[j].x; c2[4 * j + 1] += x[j].y; c2[4 * j + 2] += x[j].z; c2[4 * j + 3] += x[j].w; }
                    else               { v[4 * j] += x[j].x; v[4 * j + 1] += x[j].y; v[4 * j + 2] += x[j].z; v[4 * j + 3] += x[j].w; }
                    if (w < FP8_WARPS) src[(j ^ (row >> 1)) & 3] = make_float4(0.f, 0.f, 0.f, 0.f);   // the tile of (3) is overwritten
                }
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += c2[j] * r8;
            __syncwarp();
            if (lane == 0) mbar_arrive(tfree);

            const int64_t n = tile * 128 + row;
            bool write_out = whole;
            if (!whole) {
                // partial tile: publish, and let the warp that arrives last add everything up.  When all the
                // others were seen to have arrived, this warp is the last without asking and skips the counter.
                float* dst = p.partials + (((size_t)tile * p.maxseg + slot) * 128 + row) * 16;
                // (32 bytes per store: whole sectors)
#pragma unroll
                for (int j = 0; j < 8 * NH; j += 8)
                    asm volatile("st.global.cg.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                 ::"l"(dst + j), "r"(__float_as_uint(v[j])), "r"(__float_as_uint(v[j + 1])), "r"(__float_as_uint(v[j + 2])),
                                   "r"(__float_as_uint(v[j + 3])), "r"(__float_as_uint(v[j + 4])), "r"(__float_as_uint(v[j + 5])),
                                   "r"(__float_as_uint(v[j + 6])), "r"(__float_as_uint(v[j + 7])) : "memory");
                // The counter wraps to zero with the last arrival (or is put back by the warp that skipped
                // it), so the workspace is ready for the next call without being cleared.
                uint32_t old = __shfl_sync(0xffffffffu, seen, 0);
                if (old != (uint32_t)(nseg - 1)) {
                    // the warp's stores are ordered before lane 0's release of the counter; its acquire sees the others'
                    __syncwarp();
                    if (lane == 0)
                        asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(p.counters + tile * 8 + q), "r"((uint32_t)(nseg - 1)) : "memory");
                    old = __shfl_sync(0xffffffffu, old, 0);
                } else if (lane == 0) {
                    p.counters[tile * 8 + q] = 0u;
                }
                if (old == (uint32_t)(nseg - 1)) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
                    for (int sgi = 0; sgi < nseg; ++sgi) {       // one sum in slot order
                        const float* src = p.partials + (((size_t)tile * p.maxseg + sgi) * 128 + row) * 16;
#pragma unroll
                        for (int j = 0; j < 8 * NH; j += 8) {
                            uint32_t y8[8];
                            asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                         : "=r"(y8[0]), "=r"(y8[1]), "=r"(y8[2]), "=r"(y8[3]), "=r"(y8[4]), "=r"(y8[5]), "=r"(y8[6]), "=r"(y8[7])
                                         : "l"(src + j) : "memory");
#pragma unroll
                            for (int e = 0; e < 8; ++e) v[j + e] += __uint_as_float(y8[e]);
                        }
                    }
                    write_out = true;
                }
            }
            if (u == u_end && threadIdx.x == W_EPI * 32) FGMP_STAMP_ANY(whole ? 7 : 8);    // last segment: sums complete / handed in
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
    }

    __syncthreads();
    if (threadIdx.x == 0) FGMP_STAMP_ANY(9);
    if (*abort_flag) {
        const unsigned long long t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    } else if (FUSED && threadIdx.x == 0) {
        // the CTA that finishes last takes the "records ready" word back, so that the control area is as the next call needs it
        if (atomicInc(p.cw + CW_DONE, (uint32_t)G - 1u) == (uint32_t)G - 1u)
            asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.cw + CW_QREADY), "r"(0u) : "memory");
    }
    if (warp == W_MMA) {
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

std::mutex g_dec_mu;                 // guards the per-device caches below
bool g_attr_set[64] = {};

fgmp_status set_attrs_once()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FGMP_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_dec_mu);
    if (!g_attr_set[dev]) {
        if (cudaFuncSetAttribute(decode_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(decode_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DEC_SMEM) != cudaSuccess)
            return FGMP_ERR_CUDA;
        g_attr_set[dev] = true;
    }
    return FGMP_OK;
}

// Workspace of the decode path, all inside the control area that must be zero before the first call and
// that every call leaves zero: status at 0, control words at 256, stream-K
// counters from 1024 (32 bytes per tile); partial sums behind the control area, then (fused calls
// without a packed output) the activation records.
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
    return p;
}

template <bool FUSED>
fgmp_status launch_decode(const DecParams& p, const DecPlan& d, bool programmatic, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)d.grid); cfg.blockDim = dim3(DEC_THREADS); cfg.dynamicSmemBytes = DEC_SMEM; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = programmatic ? 1 : 0;
    if (p.M <= 8) { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<1, FUSED>, p)); }
    else          { FGMP_LAUNCH(FGMP_K_DECODE, s, cudaLaunchKernelEx(&cfg, decode_kernel<2, FUSED>, p)); }
    return fgmp_launch_status();
}

}  // namespace

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
    if (clear_first && cudaMemsetAsync(workspace, 0, 1024 + (size_t)d.tiles * 32, s) != cudaSuccess) return FGMP_ERR_CUDA;
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
    if (!fgmp_scales_valid(sc) || fgmp_fp8_free(sc)) return FGMP_ERR_INVALID_ARG;   // a free FP8 scale: the two calls and fgmp_linear_classes
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
