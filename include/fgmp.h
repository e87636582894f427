/*
 * libfgmp -- the FGMP linear layer (fine-grained mixed-precision NVFP4/FP8 weights and
 * activations) for NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes only.
 *
 * Orientation (Section 3: Y = W x X, blocks run along the dot-product dimension):
 *   activations X [M, K], weights W [N, K], output Y [M, N]; K is contiguous in X and W.
 * A block is 16 consecutive elements along K (Section 4: block size = NVFP4 microscale
 * block = vector length 16).  Each block is stored either as NVFP4 (16 E2M1 codes + one
 * E4M3 microscale, times an FP32 tensor scale) or as FP8 E4M3 (times an FP32 tensor
 * scale, no microscale), with one metadata bit per block (Section 4, Section 5.1).
 *
 * Conventions for every entry point
 *   - every data pointer is a DEVICE pointer owned by the caller, unless it says "host";
 *   - the library allocates no device memory: scratch comes in through `workspace`
 *     (size from fgmp_workspace_bytes); a workspace may be reused once the call that used
 *     it has completed on its stream;
 *   - calls are asynchronous on `cuda_stream` (a cudaStream_t, may be NULL for the default
 *     stream); the return value reports argument validation and launch errors only;
 *   - requirements: K % 64 == 0, K >= 64, rows >= 1, bf16 inputs finite, input pointers
 *     16-byte aligned, leading dimensions multiples of 8 elements;
 *   - a packed tensor is an opaque device blob (layout below) produced by the two
 *     quantizers and consumed by fgmp_linear / fgmp_unpack; it must be 1024-byte aligned.
 *
 * Packed blobs (sections 1024-byte aligned).  A "unit" = one tile of 128 rows x one chunk of 256
 * K elements (16 blocks); C = ceil(K/256) chunks per tile.
 *
 * Activations: header | codes4 | sf | mask | arec | codes8
 *   header  256 B : fgmp_packed_header (device-written)
 *   codes4        : rows * K/2 bytes, row-major; two E2M1 codes per byte, even element in
 *                   the low nibble; all-zero for FP8 blocks
 *   sf            : E4M3 microscales in 512-byte tiles of 128 rows x 4 blocks:
 *                   byte of (row r, block kb) = ((r/128) * (K/64) + kb/4) * 512
 *                                               + (r%32)*16 + ((r%128)/32)*4 + kb%4;
 *                   0x00 for FP8 blocks
 *   mask          : rows * ceil(K/16/32) uint32; bit j of word w of a row = block 32w+j,
 *                   1 = FP8
 *   arec          : (rows <= 16 only) C records of 10752 bytes, one per chunk, holding what the
 *                   decode-sized GEMM streams, for 16 token rows (rows >= M are zero):
 *                   2048 B: the E2M1 codes as a 16-row x 128-byte tile, the 16-byte pieces of row m
 *                   XOR-swizzled with m%8 (zero in FP8 blocks) | 256 B: E4M3 microscales [token][block
 *                   column], 0x00 for FP8 blocks | 16 B: two uint32 (one per token octet; their OR is used) whose
 *                   bit j says that block column j of some token is FP8, padding | 256 B padding | 8192 B: every element over the tensor
 *                   scale in fp16 (exact for either format): token octet m/8 in its own 4096 bytes, there
 *                   256 bytes per block column, there 32 bytes per token
 *   codes8        : a dense rows*K byte plane of which only the FP8 blocks are written (the
 *                   blob is sized for the worst case of every block being FP8).  Footprint of packed
 *                   activations: 1.57 bytes per element reserved (codes4 0.5 + sf 1/16 + mask 1/128 + codes8 1),
 *                   of which a quantizer pass with FP8 fraction p writes and a GEMM reads
 *                   (1-p)*9/16 + p + 1/128 bytes per element (0.61 at p = 0.1): the plane costs address space,
 *                   not traffic, and keeps the single-pass quantizer free of a compaction step
 *
 * Weights: header | mask | uptr | records | lists
 *   record        : 18560 bytes per unit, unit (t, c) at index t*C + c:
 *                   16384 B of 8-byte slots as a 128-row x 128-byte tile, the 16-byte pieces of row r
 *                   XOR-swizzled with r%8 (the K-major layout the tensor core reads): the 16 E2M1 codes
 *                   of an NVFP4 block, or E4M3 codes 0..7 of an FP8 block (zero beyond N)
 *                   | 2048 B of E4M3 microscales, 0x00 for FP8 blocks, in the order they go to tensor
 *                   memory: byte of (row r, block column j) = (j/4)*512 + (r%32)*16 + (r/32)*4 + j%4
 *                   | 128 B: uint16 x 17, FP8 blocks of the unit before block column j; entry 16 = all
 *   list          : per unit, its FP8 blocks ordered by (block column, row): one uint32 for each (padded
 *                   to 16 bytes; low half = byte offset of the block's slot in the tile, high half =
 *                   16 * row + 4 * ((row / 2) % 4)), then E4M3 codes 8..15 of each (8 bytes, padded to 16)
 *   uptr          : uint32 [units + 1]: start of a unit's list in 16-byte steps
 *                   fgmp_weights_bytes(N, K, max_fp8_blocks) leaves room for that many FP8 blocks.
 */
#ifndef FGMP_H
#define FGMP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FGMP_OK = 0,
    FGMP_ERR_INVALID_ARG = -1, /* NULL pointer, bad enum, non-finite or non-positive scale   */
    FGMP_ERR_SHAPE = -2,       /* K % 64, leading dimension, alignment                       */
    FGMP_ERR_WORKSPACE = -3,   /* workspace or output blob too small                         */
    FGMP_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed                          */
    FGMP_ERR_ARCH = -5,        /* current device is not compute capability 10.x              */
    FGMP_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired (see fgmp_check)        */
    FGMP_ERR_CAPACITY = -7     /* more FP8 blocks than the packed blob has room for          */
} fgmp_status;

/* Which block score decides the precision.
 *   FGMP_SCORE_LP_ERROR : sum_i f_i (v_i - Q_NVFP4(v_i))^2          (Eq. 6)
 *   FGMP_SCORE_HP_TO_LP : sum_i f_i (Q_NVFP4(v_i) - Q_FP8(v_i))^2   (Eq. 7-8)          */
typedef enum { FGMP_SCORE_LP_ERROR = 0, FGMP_SCORE_HP_TO_LP = 1 } fgmp_score_mode;

/* NVFP4 microscale of weight blocks: dynamic max, or the sensitivity-weighted brute-force
 * search over all 126 positive finite E4M3 scales (Eq. 11).  Activations always use
 * dynamic max (Section 3.3). */
typedef enum { FGMP_CLIP_NONE = 0, FGMP_CLIP_SW_BRUTE = 1 } fgmp_clip_mode;

typedef struct {
    float scale_fp4;    /* FP32 tensor scale of the NVFP4 part; 0 = derive amax/(6*448)
                           on the device (weights only)                                     */
    int fp8_log2_ratio; /* FP8 tensor scale = scale_fp4 * 2^ratio, -7 <= ratio <= 7 (used
                           when scale_fp8 is 0)                                             */
    float scale_fp8;    /* 0, or an FP32 tensor scale of the FP8 part of its own (Section
                           5.1: FP8 blocks carry no microscale, only a per-tensor scale),
                           in any ratio to scale_fp4.  Operands packed with such a scale
                           are multiplied by fgmp_linear_classes; fgmp_linear, whose single
                           accumulator needs the power-of-two ratio, refuses them.          */
} fgmp_scales;

/* First 256 bytes of a packed blob (device memory). */
typedef struct {
    uint32_t magic;          /* 'FGMP' = 0x504d4746                                         */
    uint32_t version;        /* layout version, 7                                           */
    int64_t rows, K;
    float scale_fp4;         /* tensor scale actually used                                  */
    int32_t fp8_log2_ratio;
    int64_t n_fp8;           /* number of FP8 blocks (activations: 0 if tau = +inf, else -1) */
    float tau_eff;           /* weights, fraction mode: smallest selected score             */
    uint32_t kind;           /* 0 = activations, 1 = weights                                */
    int64_t capacity;        /* weights: room for the FP8 lists, in 16-byte steps            */
    int32_t error;           /* 0, or FGMP_ERR_CAPACITY                                     */
    float scale_fp8;         /* FP8 tensor scale actually used                              */
    int32_t fp8_scale_free;  /* 1 if scale_fp8 was given on its own (fgmp_scales.scale_fp8) */
    int32_t reserved[47];
} fgmp_packed_header;

enum { FGMP_OP_QUANTIZE_WEIGHTS = 0, FGMP_OP_QUANTIZE_ACTIVATIONS = 1, FGMP_OP_LINEAR = 2,
       FGMP_OP_CALIBRATE_TAU = 3,
       FGMP_OP_GLOBAL_TAU = 4,      /* M = total number of scores; N, K ignored */
       FGMP_OP_LINEAR_QUANTIZE = 5, FGMP_OP_LINEAR_FUSED = 6, FGMP_OP_LINEAR_CLASSES = 7 };

/* ---- sizes (pure host functions; return 0 for invalid shapes) ---- */
size_t fgmp_weights_bytes(int64_t N, int64_t K, int64_t max_fp8_blocks);
size_t fgmp_acts_bytes(int64_t M, int64_t K);
/* scratch needed by one call of `op` (FGMP_OP_*); M or N is ignored where it has no meaning */
size_t fgmp_workspace_bytes(int op, int64_t M, int64_t N, int64_t K);

/* ---- offline: weight packing (Section 3.1-3.3; Eq. 8, 9, 11) ----
 * W_bf16 [N, ldw] bf16, fisher_elem [N, ldf] fp32 (per-element diagonal Fisher information,
 * the g^2 of Eq. 6).  Per block: microscale (dynamic max or Eq. 11 search), score under that
 * scale (Eq. 6 or Eq. 8).  fp8_fraction >= 0: exactly floor(fraction * N*K/16 + 0.5) blocks
 * with the largest scores are kept in FP8 (Eq. 9: the top-R percentile of one tensor; equal
 * scores are taken in row-major block order) and tau is ignored; fp8_fraction < 0: a block
 * is FP8 iff score > tau.  The blob must have room for the result
 * (packed_bytes >= fgmp_weights_bytes(N, K, max_fp8_blocks)); if threshold mode finds
 * more FP8 blocks than the blob has room for, header.error = FGMP_ERR_CAPACITY and the blob
 * is invalid: fgmp_unpack refuses it, and fgmp_linear given such a blob (or one whose header
 * does not carry the N and K of the call) reads none of it and records FGMP_ERR_INVALID_ARG in
 * the workspace status (fgmp_check).
 * tau_eff_out (device float, may be NULL) receives the smallest selected score. */
fgmp_status fgmp_quantize_weights(const void* W_bf16, int64_t ldw, const float* fisher_elem, int64_t ldf,
                                  int64_t N, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                                  fgmp_clip_mode cm, double fp8_fraction, float tau,
                                  void* packed_out, size_t packed_bytes, float* tau_eff_out,
                                  void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- online: activation quantizer (Section 4.2) ----
 * X_bf16 [M, ldx] bf16, fisher_chan [K] fp32 (average squared gradient per input channel).
 * Per block: dynamic-max NVFP4 scale, NVFP4 rounding, the score, FP8 iff score > tau
 * (tau is calibrated offline and fixed; +inf = all NVFP4, negative = all FP8), then the
 * block is written in its format.  sc.scale_fp4 must be > 0.  No workspace needed
 * (workspace may be NULL). */
fgmp_status fgmp_quantize_activations(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                      int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm, float tau,
                                      void* packed_out, size_t packed_bytes,
                                      void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- offline: activation threshold for a target FP8 fraction (Eq. 9, local threshold) ----
 * Scores every block of a calibration batch X and writes to tau_out (device float) the
 * value midway (in fp32) between the k-th and (k+1)-th largest score, k = floor(fraction *
 * blocks + 0.5), so that exactly k blocks of this batch exceed it unless scores tie. */
fgmp_status fgmp_calibrate_tau(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                               int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                               double fp8_fraction, float* tau_out,
                               void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- offline: one threshold for several tensors (Eq. 10, global threshold) ----
 * Section 3.2 prefers a single threshold per tensor kind over per-layer ones: the blocks of all
 * layers compete for the FP8 budget, so sensitive layers end up with a larger FP8 share.
 * fgmp_weight_scores writes the block scores of one weight tensor (the scores fgmp_quantize_weights
 * ranks: under the clipped microscale if cm = FGMP_CLIP_SW_BRUTE; scores[n * K/16 + kb], device,
 * 16-byte aligned; workspace as for fgmp_quantize_weights); fgmp_activation_scores does the same
 * for a calibration batch.  fgmp_global_tau then takes the scores of n_tensors tensors
 * (score_arrays: HOST array of device pointers, counts: HOST array of lengths) and writes to tau_out
 * (device float) the value midway (in fp32) between the k-th and (k+1)-th largest of their union,
 * k = floor(fraction * total + 0.5): exactly k blocks exceed it unless scores tie (k = 0 gives +inf,
 * k = total gives -1).  Pass it as `tau` with fp8_fraction < 0 to fgmp_quantize_weights, or as the
 * activation threshold.  workspace: fgmp_workspace_bytes(FGMP_OP_GLOBAL_TAU, total, 0, 0). */
fgmp_status fgmp_weight_scores(const void* W_bf16, int64_t ldw, const float* fisher_elem, int64_t ldf,
                               int64_t N, int64_t K, fgmp_scales sc, fgmp_score_mode sm, fgmp_clip_mode cm,
                               float* scores, void* workspace, size_t ws_bytes, void* cuda_stream);
fgmp_status fgmp_global_tau(const float* const* score_arrays, const int64_t* counts, int n_tensors,
                            double fp8_fraction, float* tau_out,
                            void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- offline: the baseline policies of Section 3.4 ----
 * The "Quantization Error" policy (Eq. 12) is the score of Eq. 8 with every sensitivity weight equal to
 * one: pass a vector (activations) or matrix (weights) of ones as the Fisher argument, with
 * FGMP_SCORE_HP_TO_LP.  The "Output Error" policy (Eq. 13) weights element i by the average squared
 * magnitude of input channel i of the OTHER operand: this call computes that vector, mean_sq[c] = mean
 * over rows of X[r, c]^2 (X bf16 [rows, K] row-major, any K >= 1, rows <= 2^24; fp32, rows added in
 * order), for the weights' policy from a calibration batch of activations, for the activations' policy
 * from the weight matrix; broadcast it over the rows of the weights' Fisher matrix.  Both policies use
 * the local threshold (fraction mode / fgmp_calibrate_tau). */
fgmp_status fgmp_channel_mean_sq(const void* X_bf16, int64_t ldx, int64_t rows, int64_t K,
                                 float* mean_sq, void* cuda_stream);

/* ---- workspace of fgmp_linear ----
 * The first FGMP_WS_CONTROL_BYTES of a workspace hold the status word that fgmp_check reads and,
 * for decode-sized batches, the counters of tiles that several thread blocks share.  They must be
 * zero when fgmp_linear first uses the workspace: clear them once with this call (a memset on the
 * stream; workspace 1024-byte aligned).  Every fgmp_linear that ends without a device-side error
 * leaves them as the next call needs them, whatever the shapes of the two calls (prefill-sized
 * calls keep their scratch behind the control area), so that a decode step needs no clearing pass
 * of its own; after an error reported by fgmp_check, clear the workspace again before reusing it. */
#define FGMP_WS_CONTROL_BYTES 65536
fgmp_status fgmp_workspace_init(void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- the mixed-precision GEMM (Section 4.1) ----
 * Y[m, n] = sum over blocks of dot16(A[m, kb], W[n, kb]) with each block pair multiplied in
 * its own formats (FP4xFP4, FP4xFP8, FP8xFP4, FP8xFP8), microscales and tensor scales
 * applied, accumulated in FP32.  Y is fp32 (y_is_bf16 = 0) or bf16 [M, ldy].  The workspace
 * must have been cleared once with fgmp_workspace_init.  For 1 <= M <= 16, K % 256 == 0 and
 * N <= 258048 the weight-streaming kernel runs, launched as a programmatic dependent of the kernel
 * before it in the stream (its set-up and its first reads of packed_weights overlap that kernel's
 * end; it reads the packed activations and the workspace only after that kernel has completed).  So
 * packed_weights must be complete before the kernel that precedes this call in the stream starts --
 * always true for weights packed by fgmp_quantize_weights, whose last kernel writes only header fields
 * that are read late; a caller who fills or copies a weight blob with a kernel of their own must not
 * make that kernel the immediate predecessor (any other operation in between is enough). */
fgmp_status fgmp_linear(const void* packed_acts, const void* packed_weights,
                        void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                        void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- the same GEMM with one accumulation per class of block pair (Section 4.1: the four dot-product
 * units; Section 5.1: FP8 blocks under a per-tensor scale of their own) ----
 * For operands whose FP8 tensor scale is not tied to the NVFP4 one by a power of two (fgmp_scales.scale_fp8 > 0
 * at packing time; operands with tied scales are accepted too).  The four classes FP4xFP4, FP4xFP8, FP8xFP4 and
 * FP8xFP8 are accumulated separately in FP32 -- four passes of the tensor-core GEMM over operands in which the
 * blocks of the other format are zero -- and each sum is multiplied by the product of its own two tensor scales
 * before it is added to Y.  About four times the cost of fgmp_linear: the price of the free scale.
 * Y is fp32 [M, ldy] (y_is_bf16 must be 0).  workspace: fgmp_workspace_bytes(FGMP_OP_LINEAR_CLASSES, M, N, K),
 * cleared once with fgmp_workspace_init; any M >= 1. */
fgmp_status fgmp_linear_classes(const void* packed_acts, const void* packed_weights,
                                void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                                void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- one decode step in one launch: activation quantizer + GEMM (Section 4.2 into Section 4.1) ----
 * For decode-sized batches (the shapes of fgmp_linear's weight-streaming kernel: 1 <= M <= 16,
 * K % 256 == 0) this is fgmp_quantize_activations(X, ...) followed by fgmp_linear, as one kernel: the
 * thread blocks first share out the quantizer's work (256-element chunks of eight token rows; four lanes
 * per block, the same single-precision steps in the same order, so codes, scales and masks are those of
 * fgmp_quantize_activations bit for bit), while the first weight records are already on their way, and
 * start multiplying once every chunk has been handed in.  Y is what fgmp_linear returns for those packed
 * activations, bit for bit.
 *   packed_acts_out (may be NULL): receives the packed activations (size fgmp_acts_bytes(M, K)) for a
 *     caller that wants them (fgmp_unpack, or a later fgmp_linear with other weights); if NULL only the
 *     fp16 records the GEMM streams are kept, in the workspace.
 *   workspace: fgmp_workspace_bytes(FGMP_OP_LINEAR_FUSED, M, N, K), cleared once with
 *     fgmp_workspace_init.  Beside fgmp_linear's words the control area holds the work-item counters of
 *     the quantizer and a "records ready" word; the counters wrap to zero by themselves and the block that
 *     finishes last clears the word, so nothing has to be cleared between calls; after an
 *     error reported by fgmp_check clear the workspace again.  Calls that share a workspace must not
 *     overlap on the GPU.
 *   The kernel is launched as a programmatic dependent like fgmp_linear's (same condition on
 *   packed_weights); X and the workspace are read only after the preceding kernel has completed.
 * Larger M runs the two calls (packed_acts_out is then required). */
fgmp_status fgmp_linear_fused(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                              fgmp_scales sc, fgmp_score_mode sm, float tau, const void* packed_weights,
                              void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                              void* packed_acts_out, size_t packed_bytes,
                              void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- fgmp_linear with the next layer's activation quantizer in its epilogue (Section 4.2) ----
 * The paper's post-processing unit quantizes the output activations of a layer, block by block, to
 * FP4 or FP8 from the FP32 partial sums, so that they reach memory only in packed form.  This call is
 * fgmp_linear with a bf16 output followed by fgmp_quantize_activations on that output -- the packed
 * result is the same bit for bit -- without the bf16 tensor ever being written or read: every
 * accumulator is scaled, rounded to bf16 and quantized in registers by the GEMM's epilogue.
 * packed_out is a packed activation tensor of M rows and N columns (N is the next layer's K; size from
 * fgmp_acts_bytes(M, N)); fisher_chan_next [N], sc_next, sm and tau_next are the arguments
 * fgmp_quantize_activations would get.  N % 64 == 0.  Decode-sized batches (the shapes that take the
 * weight-streaming kernel, whose threads hold output rows rather than token rows) run as the two
 * launches, with the bf16 outputs (at most 16 x N) passing through the workspace.
 * workspace: fgmp_workspace_bytes(FGMP_OP_LINEAR_QUANTIZE, M, N, K), cleared once like fgmp_linear's. */
fgmp_status fgmp_linear_quantize(const void* packed_acts, const void* packed_weights,
                                 int64_t M, int64_t N, int64_t K,
                                 const float* fisher_chan_next, fgmp_scales sc_next, fgmp_score_mode sm,
                                 float tau_next, void* packed_out, size_t packed_bytes,
                                 void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- fgmp_linear for callers that cannot allocate (the paper has no counterpart) ----
 * Some callers have no way to hand the library a workspace: code that runs where cudaMalloc is
 * forbidden (inside a region that must not touch the allocator, a host that pre-sized its
 * memory pool and gave all of it away, a plugin interface with no scratch argument).  This
 * variant of fgmp_linear for decode-sized batches (1 <= M <= 16 tokens, K % 256 == 0) keeps its
 * scratch -- status word, stream-K tile counters and partial sums -- in a fixed array inside the
 * library image instead: FGMP_STATIC_SCRATCH_BYTES of device memory on every GPU that loads the
 * library, held until the process exits.  It calls no allocation routine of any kind.
 *   - Inputs and outputs are passed as for fgmp_linear; results are bit-identical to it.
 *   - Shapes whose scratch need (fgmp_workspace_bytes(FGMP_OP_LINEAR, M, N, K)) exceeds
 *     FGMP_STATIC_SCRATCH_BYTES return FGMP_ERR_WORKSPACE; M > 16 or K % 256 != 0 returns
 *     FGMP_ERR_SHAPE.  Llama-2-70B FC1/FC2 (28672 x 8192) needs 3.6 MiB and fits; N > 258048 is not a decode shape.
 *   - The first call on each device looks up the array's device address (a host-side query,
 *     made with that device current); make that first call outside any stream capture.
 *   - All calls on one GPU share the array and each call starts by clearing the part that
 *     must be zero, so calls must not overlap on the GPU: two calls in flight at once (two
 *     streams, two host threads) race on the scratch and give wrong results.  Calls ordered
 *     on one stream are fine.
 *   - status_out (device, 2 x int32, may be NULL) receives what fgmp_check would report for
 *     this call: word 0 = FGMP_OK or FGMP_ERR_TIMEOUT, copied on the stream after the kernel. */
#define FGMP_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
fgmp_status fgmp_linear_static(const void* packed_acts, const void* packed_weights,
                               void* Y, int y_is_bf16, int64_t ldy, int64_t M, int64_t N, int64_t K,
                               int32_t* status_out, void* cuda_stream);

/* Synchronizes the stream and returns the device-side status recorded in a workspace used
 * by fgmp_linear (FGMP_OK, FGMP_ERR_TIMEOUT, or FGMP_ERR_INVALID_ARG for a packed tensor whose
 * header does not match the call). */
fgmp_status fgmp_check(const void* workspace, void* cuda_stream);

/* ---- parity support: packed -> canonical arrays (device) ----
 * codes4 [rows*K/2] (0 for FP8 blocks), codes8 [rows*K] (0 for FP4 blocks), scales
 * [rows*K/16] E4M3 (0 for FP8 blocks), mask [rows*ceil(K/16/32)], scores is not stored.
 * Any output pointer may be NULL.  The tensor scales are not among the outputs: they are in the blob's
 * header (scale_fp4, fp8_log2_ratio, scale_fp8), 256 bytes that the caller can copy. */
fgmp_status fgmp_unpack(const void* packed, int64_t rows, int64_t K, uint8_t* codes4, uint8_t* codes8,
                        uint8_t* scales, uint32_t* mask, void* cuda_stream);

/* ---- measurement support: tensor-core rate per operand kind ----
 * Runs, on every SM, mma_per_cta tcgen05 instructions of M = 128, N = 256 on operands resident in
 * shared memory (nothing is loaded or stored; mma_per_cta <= 2^21): kind 0 = bf16 (K = 16 per instruction), 1 = FP8 E4M3
 * (K = 32), 2 = NVFP4 with E4M3 block scales (K = 64); kind + 4 = the same on CTA pairs (cta_group::2, M = 256 per
 * pair, the leader issues mma_per_cta instructions; an odd SM stays idle).  The caller times the call on the stream;
 * flops = 2 * 128 * 256 * K * mma_per_cta * (number of CTAs launched: the SMs, or the SMs in pairs).  These are the rates the block-pair
 * products of Section 4.1 can run at at best, i.e. the denominators of the prefill roofline.
 * workspace: >= 256 bytes, zeroed, 256-byte aligned (status word, read by fgmp_check). */
fgmp_status fgmp_tensor_peak(int kind, int64_t mma_per_cta, void* workspace, size_t ws_bytes, void* cuda_stream);

/* ---- self-test of the failure path (the paper has no counterpart) ----
 * Every wait inside the kernels is bounded: when it runs out the kernel records FGMP_ERR_TIMEOUT in
 * the status word of its workspace and returns, instead of hanging the GPU.  This call exercises that
 * path without any GEMM: a single thread block waits up to limit_ns (1e3 .. 1e8) for a barrier that
 * nothing completes.  Afterwards fgmp_check(workspace) returns FGMP_ERR_TIMEOUT, fgmp_workspace_init
 * clears it, and the workspace serves fgmp_linear again.  workspace: >= 256 bytes, 256-byte aligned. */
fgmp_status fgmp_selftest_wait_timeout(void* workspace, size_t ws_bytes, int64_t limit_ns, void* cuda_stream);

/* Block scores only (parity support and calibration): scores [M*K/16] fp32, activations. */
fgmp_status fgmp_activation_scores(const void* X_bf16, int64_t ldx, const float* fisher_chan,
                                   int64_t M, int64_t K, fgmp_scales sc, fgmp_score_mode sm,
                                   float* scores, void* cuda_stream);

/* ---- measurement support (the paper has no counterpart) ----
 * Between fgmp_profile_begin and fgmp_profile_end (host calls, same thread as the launches)
 * the library counts every kernel it launches, per kernel id, and brackets the launches of
 * the ids selected in `timed_kernel_mask` (bit i = id i) with CUDA events on their launch
 * stream.  fgmp_profile_end synchronizes those events and fills launches[i] and ms_total[i]
 * (host arrays of length n; ms_total is 0 for ids that were not selected).  Both return the
 * number of kernel ids; fgmp_kernel_name(i) names id i. */
int fgmp_profile_begin(unsigned timed_kernel_mask);
int fgmp_profile_end(int n, long long* launches, float* ms_total);
const char* fgmp_kernel_name(int id);

const char* fgmp_status_string(fgmp_status s);
int fgmp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FGMP_H */
