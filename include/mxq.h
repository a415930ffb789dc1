/*
 * mxq.h -- C ABI of libmxq: the MXFP4 weight-only-quantised linear layer that
 * dominates every draft step of ML-SpecQD (arXiv 2503.13565), for one NVIDIA
 * B200 (sm_100a).
 *
 * General rules, valid for every call below unless it says otherwise:
 *   - Pointers named *_dev (and every pointer not named *_host) are DEVICE
 *     pointers owned by the caller; the library allocates nothing, frees
 *     nothing and keeps no pointer after the call returns.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream).  No call synchronises.
 *   - The return value is an MXQ_* status.  Argument errors are found on the
 *     host before anything is enqueued, so a non-zero status other than
 *     MXQ_ERR_CUDA means nothing ran.  Nothing throws or aborts.
 *   - Base pointers must be 16-byte aligned (MXQ_ERR_ALIGN otherwise).
 *   - K must be a positive multiple of 32 and N >= 1 (MXQ_ERR_SHAPE otherwise).
 *
 * The MXFP4 tensor pair (Sec. III-D-3 of the paper: an FP4 weight tensor plus
 * one 8-bit scale per 32 elements):
 *   codes  uint8 [N][K/2]  row-major; byte j of a row holds element 2j in its
 *                          low nibble and element 2j+1 in its high nibble.  A
 *                          nibble is an E2M1 code  s e1 e0 m  (bias 1), i.e.
 *                          one of 0, 0.5, 1, 1.5, 2, 3, 4, 6 with a sign.
 *   scales uint8 [N][K/32] row-major; E8M0: the byte b stands for 2^(b-127);
 *                          0xFF stands for NaN.
 * Sixteen consecutive code bytes are one block of 32 weights and share one
 * scale byte.  The dequantised weight is  w^ = (+-)value(code) * 2^(b-127).
 */
#ifndef MXQ_H
#define MXQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MXQ_VERSION 100 /* major*100 + minor */

enum mxq_status {
    MXQ_OK = 0,
    MXQ_ERR_NULL = 1,      /* a required pointer is NULL                               */
    MXQ_ERR_SHAPE = 2,     /* a size is out of range (K % 32, M not in 1..16, ...)      */
    MXQ_ERR_ALIGN = 3,     /* a base pointer is not 16-byte aligned                    */
    MXQ_ERR_DTYPE = 4,     /* unknown MXQ_F32 / MXQ_BF16 selector                      */
    MXQ_ERR_WORKSPACE = 5, /* workspace missing or smaller than *_workspace_bytes()     */
    MXQ_ERR_CUDA = 6       /* the CUDA runtime reported an error at launch             */
};

enum mxq_dtype { MXQ_F32 = 0, MXQ_BF16 = 1 };

#define MXQ_MAX_M 16 /* token rows per mxq_linear call                          */
#define MXQ_MAX_T 64 /* speculated tokens per sequence in mxq_greedy_accept*    */

/* Library version (MXQ_VERSION of the build). */
int mxq_version(void);

/* Static, human-readable text for a status code; never NULL. */
const char *mxq_status_string(int status);

/* Programmatic dependent launch.  When enabled (the default) mxq_linear kernels are
 * launched so that their weight prefetch may overlap the tail of the previous kernel
 * in the stream; they read X and write Y only after that kernel has completed, so
 * results do not change.  Returns the previous setting.  Host-side, process-wide. */
int mxq_set_pdl(int enabled);

/* Bytes of a codes / scales tensor for an [N][K] weight matrix: N*K/2 and N*K/32
 * (together 4.25 bits per weight, Sec. III-D-3).  0 if the shape is invalid. */
size_t mxq_codes_bytes(int64_t N, int64_t K);
size_t mxq_scales_bytes(int64_t N, int64_t K);

/* Direct cast BF16 -> MXFP4 (Sec. III-D-3, steps i and ii).
 *   W_bf16  [N][K] BF16 row-major, contiguous (read)
 *   codes   [N][K/2], scales [N][K/32] (written; layout above)
 *   nonfinite_blocks  optional uint32 counter (may be NULL); incremented once per
 *           block that contained an Inf or a NaN.  The caller zeroes it.
 * Per block of 32 along K: the scale is 2^(floor(log2 max|v|) - 2), never below
 * 2^-127 (an all-zero block gets 2^-127); each element divided by the scale is
 * rounded to the nearest E2M1 value, ties to the even code, magnitudes above 6
 * clamp to 6; the sign bit of the input is always kept (so -0 stays -0).  A block
 * holding Inf/NaN gets scale 0xFF and all-zero codes. */
int mxq_quantize(const void *W_bf16, int64_t N, int64_t K, uint8_t *codes, uint8_t *scales,
                 uint32_t *nonfinite_blocks, void *stream);

/* Exact inverse map (the value each code/scale pair stands for, Sec. III-D-3), for
 * tools and tests.  W_bf16_out [N][K] BF16.  Every w^ with scale byte <= 252 is
 * BF16-representable and written exactly; 0xFF gives NaN; 253/254 may overflow to Inf. */
int mxq_dequantize(const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K, void *W_bf16_out,
                   void *stream);

/* Workspace (bytes) with which mxq_linear runs fastest for this shape; 0 where none is used.  The workspace is
 * OPTIONAL: mxq_linear accepts NULL / 0 or a smaller buffer and is then merely slower for 3 or more token rows (and for
 * 2 on matrices of 8 M weights or more).
 * With it, MXQ_KERNEL_UMMA rewrites the M token rows as FP8 parts once per call (a small kernel ahead of the
 * weight kernel, which then fetches them with bulk copies) instead of once per CTA.  Device memory, 16-byte
 * aligned, no initialisation needed; contents are scratch.  Calls that may run concurrently (different streams)
 * need a workspace each. */
size_t mxq_linear_workspace_bytes(int M, int64_t N, int64_t K);

/* The kernels behind mxq_linear, fastest first.
 *   MXQ_KERNEL_FP4     tcgen05 block-scaled MMA with packed 4-bit operands on both sides: the codes and scales
 *                      go to the tensor core as they are, the 1..4 token rows as 16 exact radix-4 digit planes
 *                      each (needs K % 128 == 0, M <= 4)
 *   MXQ_KERNEL_UMMA    tcgen05 block-scaled MMA with the codes expanded in flight by the copy engine and each
 *                      token row split exactly into three E5M2 rows (needs K % 128 == 0, a 32-byte aligned `codes`)
 *   MXQ_KERNEL_MMA     decodes the codes into FP16 mma.sync fragments (needs K % 128 == 0)
 *   MXQ_KERNEL_GENERIC any valid shape, on the CUDA cores
 * Left to itself (MXQ_KERNEL_AUTO) mxq_linear picks by measured speed among the kernels that cover the call: FP4
 * for M = 1 (and for M = 2 on matrices of more row tiles of 128 than the GPU has SMs); UMMA otherwise, except on the
 * largest matrices at M > 2 where it can run neither one tile per CTA nor one CTA per SM: those go to MMA. */
enum mxq_kernel {
    MXQ_KERNEL_AUTO = -1, MXQ_KERNEL_GENERIC = 0, MXQ_KERNEL_MMA = 1, MXQ_KERNEL_UMMA = 2, MXQ_KERNEL_FP4 = 3
};

/* Overrides mxq_linear's choice (tests, comparisons): with a kernel of the list, mxq_linear uses the first of FP4,
 * UMMA, MMA, GENERIC that is not above it and covers the call; MXQ_KERNEL_AUTO restores the default.  Returns the
 * previous setting.  Host-side, process-wide.  The initial setting comes from the environment variable
 * MXQ_LINEAR_VARIANT (fp4 | umma | mma | generic), else MXQ_KERNEL_AUTO. */
int mxq_set_linear_kernel(int kernel);

/* Forces one layout parameter of the tcgen05 kernels where it is feasible (tests and comparisons; the heuristics
 * are the product).  `what`: one of mxq_layout_knob; `value` 0 restores the heuristic (-1 for
 * MXQ_LAYOUT_OPERAND_THROUGH_RING).  Host-side, process-wide, not synchronised with calls running on other host
 * threads (the same holds for mxq_set_pdl and mxq_set_linear_kernel, and for the per-device caches behind the
 * launches: configure from one thread, or before the worker threads start). */
enum mxq_layout_knob {
    MXQ_LAYOUT_SPLIT = 0,                /* CTAs per cluster (K split) of MXQ_KERNEL_FP4 / MXQ_KERNEL_UMMA              */
    MXQ_LAYOUT_RING = 1,                 /* ring slots                                                               */
    MXQ_LAYOUT_TILES = 2,                /* 128-row tiles per CTA                                                    */
    MXQ_LAYOUT_OPERAND_THROUGH_RING = 3, /* MXQ_KERNEL_UMMA with a workspace: 0 token operand resident, 1 through the ring */
    MXQ_LAYOUT_PRESPLIT_MIN_M = 4,       /* MXQ_KERNEL_UMMA: token rows from which the operand is split ahead (17: never) */
    MXQ_LAYOUT_BATCH_RING = 5,           /* mxq_linear_batch: ring slots per CTA                                      */
    MXQ_LAYOUT_BATCH_CTAS_PER_SM = 6     /* mxq_linear_batch: CTAs per SM (1..2)                                      */
};
int mxq_set_linear_layout(int what, int value);

/* How a kernel would run this shape on the current device (diagnostics; launches nothing).
 * kernel = MXQ_KERNEL_AUTO describes the one mxq_linear would pick under the current setting for a
 * suitably aligned `codes`; another value describes that kernel whether or not it would be picked.
 * info[12] int32; info[0] = the kernel described, or -1 if the requested kernel does not cover the shape.
 *   MXQ_KERNEL_FP4,     [1] CTAs; [2] ring slots; [3] CTAs per cluster (K split); [4] most stages a CTA owns
 *   MXQ_KERNEL_UMMA:    (a stage is 256 k for FP4, 128 k for UMMA); [5] 128-row tiles; [6] tensor-memory
 *                       columns; [7] dynamic shared memory bytes; [8] columns of the token operand; [9] K/32;
 *                       [10] tile groups (CTAs = groups x split; a CTA walks the tiles of its group);
 *                       [11] most tiles in a group.
 *   MXQ_KERNEL_MMA:     [1] CTAs; [2] ring stages; [3] K windows; [4] blocks per window; [5] blocks in the
 *                       last window; [6] most 16-row tiles a CTA owns; [7] dynamic shared memory bytes;
 *                       [8] 8-token column tiles; [9] K/32.
 *   MXQ_KERNEL_GENERIC: [1] CTAs.
 * Unused entries are 0. */
int mxq_linear_plan_info(int kernel, int M, int64_t N, int64_t K, int32_t *info);

/* Copies to *status_host, and then clears, the sticky device words in which the tcgen05 kernels record a
 * bounded wait that gave up (bit 0: data of a stage never arrived, bit 1: a stage was never released,
 * bit 2: the accumulator never completed, bit 3: a prefetched stage never landed; bits 0-3 for
 * MXQ_KERNEL_UMMA, bits 8-11 the same for MXQ_KERNEL_FP4, bits 16-20 for mxq_linear_bf16; bits 24-27 for
 * mxq_linear_batch: data of a stage never arrived, a ring slot was never released, an accumulator never completed,
 * the rewritten token rows never became ready; bit 28 for MXQ_KERNEL_MMA: the wait for a reduction slot).  0 in normal
 * operation; a non-zero word means the affected output tiles were written as NaN.  Synchronises with
 * the device (a blocking copy), so call it outside the hot loop. */
int mxq_linear_device_status(uint32_t *status_host);

/* Weight-only-quantised linear layer (the MXFP4 GEMM of Sec. III-D-3, Eq. 2):
 *     Y[m][n] = sum_k X[m][k] * w^[n][k],   1 <= M <= 16 token rows.
 *   X_bf16  [M][K] BF16 row-major (read)
 *   codes, scales  the MXFP4 pair for W[N][K] (read)
 *   Y       [M][N] row-major, float (MXQ_F32) or BF16 rounded to nearest even (MXQ_BF16)
 *   workspace / workspace_bytes  optional scratch, see mxq_linear_workspace_bytes (NULL / 0 allowed)
 * Products are formed exactly and accumulated in FP32; the block scale is applied to
 * 32-long partial sums (Eq. 2).  The summation order is fixed for a given shape, kernel selection and
 * presence of a workspace, so results are bit-reproducible run to run.  A row containing a 0xFF scale yields NaN. */
int mxq_linear(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
               void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream);

/* The same layer with the activations and the result in HOST memory (pinned memory
 * makes the copies asynchronous).  X_host [M][K] BF16 is copied to X_stage_dev
 * (>= M*K*2 bytes), the layer runs, and Y_stage_dev (>= M*N*elem bytes) is copied to
 * Y_host, all on `stream`.  The weights stay resident on the device.  Host buffers that are page-locked and
 * addressable by the GPU (cudaHostAlloc / cudaHostRegister; 16-byte aligned) are moved by the GPU itself: a small
 * kernel pulls X into X_stage_dev and the layer stores Y straight into Y_host (Y_stage_dev is then not written);
 * pageable buffers go through cudaMemcpyAsync.  Y_host is complete once `stream` has reached the end of the call. */
int mxq_linear_host(const void *X_host, int M, const uint8_t *codes, const uint8_t *scales, int64_t N,
                    int64_t K, void *Y_host, int y_dtype, void *X_stage_dev, void *Y_stage_dev,
                    void *workspace, size_t workspace_bytes, void *stream);

/* Workspace (bytes) for mxq_greedy_accept.  Device memory, 16-byte aligned.  Its first 4096 bytes are ticket counters:
 * zero them ONCE before the first call (cudaMemset); every call that completes leaves them zero again, so the same
 * workspace can be reused by later calls of any shape it is large enough for.  With counters that are not zero the
 * kernel never finds its last CTA and accept_len / next_token are not written, although the call returns MXQ_OK.  The
 * rest needs no initialisation.  Calls that may run concurrently (different streams) need a workspace each. */
size_t mxq_accept_workspace_bytes(int64_t B, int R, int64_t V);

/* Greedy verification of speculated tokens (Sec. III-A: tokens after the first
 * mismatch are dropped; Sec. III-B: G accepted tokens plus one of the target's own).
 *   logits  [B][R][V] row-major, MXQ_F32 or MXQ_BF16; row i of a sequence is the
 *           target's distribution for the position draft token i proposes to fill;
 *           R == T (no extra row) or R == T + 1
 *   draft   [B][T] int32, 1 <= T <= 64
 *   accept_len [B] int32: G = first i with draft[i] != argmax(logits[i]), else T
 *   next_token [B] int32: argmax(logits[G]) if G < R, else -1
 * argmax takes the lowest index among equal maxima and never selects a NaN; a row
 * with nothing above -inf yields 0. */
int mxq_greedy_accept(const void *logits, int logits_dtype, int64_t B, int R, int64_t V, const int32_t *draft,
                      int T, int32_t *accept_len, int32_t *next_token, void *workspace, size_t workspace_bytes,
                      void *stream);

/* mxq_greedy_accept for callers that cannot hand over a workspace because they cannot allocate
 * one.  (The paper has no counterpart: this entry point exists for the library's users, not for
 * the method.)  Who that is: code that runs inside someone else's process with the device memory
 * already given out -- an inference server that sized its pools at start-up and forbids further
 * cudaMalloc, a plugin that is handed input and output buffers and nothing else, a latency-critical
 * loop where the device-wide synchronisation an allocation implies is not acceptable.
 *
 * Same arguments and results as mxq_greedy_accept minus the workspace.  The scratch (ticket
 * counters and per-slice partial maxima) lives in an array built into the library,
 * mxq_greedy_accept_static_max_bytes() bytes (1 MiB) on every GPU that loads the library, for the
 * life of the process.  The call allocates and frees nothing.
 *   - A shape whose scratch (mxq_accept_workspace_bytes) exceeds that size is refused with
 *     MXQ_ERR_WORKSPACE; use mxq_greedy_accept with your own workspace instead.
 *   - The first call on each device asks the CUDA runtime once for the array's device address
 *     (with that device current) and remembers it; make that first call outside any stream
 *     capture.  A failure of that query returns MXQ_ERR_CUDA.
 *   - All calls on a device share the one array, and it keeps what the previous call left in it
 *     (each call re-zeroes the counters it needs on `stream` before launching).  Two calls that may
 *     run on the GPU at the same time -- different streams, or different host threads -- race on
 *     it and may return wrong results; serialise them, or give each its own workspace through
 *     mxq_greedy_accept. */
int mxq_greedy_accept_static(const void *logits, int logits_dtype, int64_t B, int R, int64_t V,
                             const int32_t *draft, int T, int32_t *accept_len, int32_t *next_token,
                             void *stream);

/* Size in bytes of the built-in scratch array of mxq_greedy_accept_static. */
size_t mxq_greedy_accept_static_max_bytes(void);

/* Same, with the verifier's tokens already known: verifier [B][R] int32. */
int mxq_greedy_accept_tokens(const int32_t *draft, const int32_t *verifier, int64_t B, int T, int R,
                             int32_t *accept_len, int32_t *next_token, void *stream);

/* The same layer with the weights NOT quantised: Y[m][n] = sum_k X[m][k] * W[n][k], W [N][K] BF16 row-major.  The
 * comparison point of the paper (Sec. III-D-3: 16 / 4.25 = 3.76 times the bytes of MXFP4; Sec. IV-D measures both),
 * so that the gain of the cast can be measured on this machine.  1 <= M <= 16, K even; FP32 accumulation of exact
 * products; K % 64 == 0 runs on the tensor cores, anything else on a plain kernel.  Bounded waits that give up are
 * reported by mxq_linear_device_status in bits 16-20. */
int mxq_linear_bf16(const void *X_bf16, int M, const void *W_bf16, int64_t N, int64_t K, void *Y, int y_dtype, void *stream);

/* Vocabulary projection fused with the greedy verification: logits = X . w^[V][K]^T (mxq_linear with N = V), the
 * argmax of every row and the walk over the draft in ONE launch; the logits are never written (Sec. III-A, III-B:
 * the verifier's tokens decide how many speculated tokens survive, and supply the next one).
 *   X_bf16  [R][K] BF16: the hidden states at the positions the T draft tokens propose to fill, R == T or T + 1,
 *           1 <= R <= 16.  T == 0, R == 1 is the plain draft step: next_token = argmax.
 *   draft   [T] int32 (device; may be NULL if T == 0)
 *   verifier [R] int32 out, optional (NULL to skip): argmax of every row
 *   accept_len [1], next_token [1] int32 out: as mxq_greedy_accept for one sequence
 *   workspace  device memory, >= mxq_lm_head_accept_workspace_bytes, 16-byte aligned; zero its first 4096 bytes once
 *              before the first use; every call leaves them zero again.  One per stream.
 * Argmax rules as in mxq_greedy_accept (lowest index among equal maxima, NaN and -inf never selected), applied to the
 * FP32 sums mxq_linear would have stored.  Where no tcgen05 kernel covers the call (K % 128 != 0, no tensor maps), and
 * for 11 or more rows on the largest vocabularies (where that is faster), the logits pass through the workspace: the
 * plain layer, one launch for the argmax of every row, one for the walk over the draft. */
size_t mxq_lm_head_accept_workspace_bytes(int R, int64_t V, int64_t K);
int mxq_lm_head_accept(const void *X_bf16, int R, const uint8_t *codes, const uint8_t *scales, int64_t V, int64_t K,
                       const int32_t *draft, int T, int32_t *verifier, int32_t *accept_len, int32_t *next_token,
                       void *workspace, size_t workspace_bytes, void *stream);

/* The layer with one more step fused into its output (Sec. III-D-2 names the residual add among the operators
 * fused into the linear layers; the gate / up pairing is the feed-forward block of the Llama-family models of
 * Sec. IV-A).  Arguments as mxq_linear, plus:
 *   mxq_linear_residual   Y[m][n] = residual[m][n] + sum_k X[m][k] w^[n][k].  residual [M][N] row-major in Y's type
 *                         (device, 16-byte aligned, read); it may be Y itself (in-place add).
 *   mxq_linear_swiglu     W holds the gate and up projections interleaved by rows: row 2i = gate row i, row 2i+1 = up
 *                         row i (N = 2F even).  Y[m][i] = silu(g) * u with g, u the FP32 sums of rows 2i and 2i+1 and
 *                         silu(g) = g / (1 + e^-g) evaluated in FP32; Y is [M][N/2].
 *   workspace  REQUIRED: device memory, >= mxq_linear_fused_workspace_bytes(M, N, K), 16-byte aligned, no
 *              initialisation needed, contents are scratch; one per stream.
 * On the tcgen05 kernels (K % 128 == 0) the step runs in the kernel's epilogue and the sums never reach memory;
 * elsewhere the plain layer writes its FP32 sums into the workspace and a small kernel finishes them.  Errors as
 * mxq_linear; MXQ_ERR_WORKSPACE for a workspace that is too small, MXQ_ERR_SHAPE for an odd N in mxq_linear_swiglu. */
size_t mxq_linear_fused_workspace_bytes(int M, int64_t N, int64_t K);
int mxq_linear_residual(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                        const void *residual, void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream);
int mxq_linear_swiglu(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                      void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream);

/* Several layers in ONE launch (Sec. III-B: a draft step is bound by the stream of its weights; Sec. III-D-2: the
 * operators of a layer fused around its linear layers).  A decoder layer is seven small matrices, and a kernel launch
 * per matrix costs more than its 1.4-3.7 us of weight traffic; here one persistent grid (two CTAs per SM) walks all
 * the layers of the call with one uninterrupted stream of weights, the token rows of every distinct X are rewritten as
 * tensor-core operands once, and tiles that fall into two CTAs' shares are summed in a fixed order.
 *   descs   HOST array of `count` (1..MXQ_MAX_BATCH) descriptors, read during the call only.  Per layer:
 *             X_bf16 [M][K], codes / scales the MXFP4 pair of W[N][K], Y and y_dtype as in mxq_linear;
 *             epilogue MXQ_EPI_NONE      Y [M][N]   = X . w^T
 *                      MXQ_EPI_RESIDUAL  Y [M][N]   = residual + X . w^T   (residual [M][N] in Y's type; may be Y itself)
 *                      MXQ_EPI_SWIGLU    Y [M][N/2] = silu(g) * u, rows 2i / 2i+1 of W being gate / up row i
 *           Layers run interleaved, so by default none may read (as X or residual) what another layer of the call
 *           writes.  A layer with flags = MXQ_BATCH_DEPENDS opens a new GROUP (at most MXQ_MAX_BATCH_GROUPS per call):
 *           it and the layers after it start only when every layer before it in the array has been stored, and may
 *           read those outputs (a BF16 Y as the next X, e.g. gate/up with MXQ_EPI_SWIGLU followed by down); the weight
 *           stream runs on across the group boundary.  A call of several groups is one grid whose CTAs wait for one
 *           another at the boundaries, so the whole grid (two CTAs per SM) must be able to become resident: do not run
 *           such a call while kernels of OTHER streams hold SMs for long (a wait that starves gives up after its limit
 *           and reports through mxq_linear_device_status; calls of one group never wait for a CTA that is not running).
 *           Within a group, layers that share an X pointer share its rewriting.  X, Y and residual may also be
 *           page-locked host memory that the GPU can address (cudaHostAlloc / cudaHostRegister): the kernel then reads
 *           the activations and writes the results across the bus itself.
 *   M       token rows, common to all layers of the call
 *   workspace  REQUIRED: device memory, 256-byte aligned, >= mxq_linear_batch_workspace_bytes(descs, count, M).  Zero
 *           its first 16384 bytes (counters) ONCE before the first use; every call that completes leaves them zero
 *           again; the rest needs no initialisation.  After a non-zero mxq_linear_device_status zero them again.  Calls
 *           in one stream may share a workspace; calls that may run concurrently need one each.
 * The persistent kernel covers M <= 8 with every K a multiple of 128; with 9 <= M <= 16 it runs twice, over the rows
 * [0, 8) and [8, M) (the rows of a layer are independent of one another); any other call runs its layers one after the
 * other through mxq_linear / mxq_linear_residual / mxq_linear_swiglu (same results as those).  Results are
 * bit-reproducible run to run and within mxq_linear's bound; the summation order differs from mxq_linear's.  Errors as
 * mxq_linear.  Bounded waits that give up are reported in bits 24-27 of mxq_linear_device_status. */
#define MXQ_MAX_BATCH 64
#define MXQ_MAX_BATCH_GROUPS 8
#define MXQ_BATCH_DEPENDS 1 /* this layer and the ones after it may read what the layers before it in the array wrote */
enum mxq_epilogue { MXQ_EPI_NONE = 0, MXQ_EPI_RESIDUAL = 1, MXQ_EPI_SWIGLU = 2 };
typedef struct mxq_linear_desc {
    const void *X_bf16;
    const uint8_t *codes;
    const uint8_t *scales;
    void *Y;
    const void *residual; /* MXQ_EPI_RESIDUAL only, else NULL */
    int64_t N, K;
    int32_t y_dtype;      /* MXQ_F32 / MXQ_BF16 */
    int32_t epilogue;     /* mxq_epilogue */
    int32_t flags;        /* 0, or MXQ_BATCH_DEPENDS */
    int32_t reserved;     /* 0 */
} mxq_linear_desc;
size_t mxq_linear_batch_workspace_bytes(const mxq_linear_desc *descs, int count, int M);
int mxq_linear_batch(const mxq_linear_desc *descs, int count, int M, void *workspace, size_t workspace_bytes,
                     void *stream);

/* How mxq_linear_batch would run the call on the current device (diagnostics; launches nothing).  info[8] int32:
 * [0] launches of the persistent kernel (1; 2 for 9..16 token rows, the rest then describes the first), 0 if the
 * layers would run one by one; [1] CTAs; [2] ring slots per
 * CTA; [3] dynamic shared memory bytes; [4] columns of the token operand; [5] units of work (128 rows x 256 k);
 * [6] tensor-memory columns per CTA; [7] accumulator slots in tensor memory. */
int mxq_linear_batch_info(const mxq_linear_desc *descs, int count, int M, int32_t *info);

/* Test hook for the bounded waits of mxq_linear_batch: the NEXT call of mxq_linear_batch (one-shot) leaves out the weight
 * copy of unit `unit` of its work sequence and limits every wait inside the kernel to `wait_us` microseconds.  The
 * CTA that owns the unit then gives up: the call still completes, mxq_linear_device_status reports bit 24 and the
 * tiles that CTA had not finished are NaN.  unit = -1, wait_us = 0 cancels. */
int mxq_debug_batch_fault(int unit, unsigned wait_us);

/* The bounds-checked build (the library compiled with -DMXQ_DEBUG_BOUNDS; python -m paper_2503_13565_b200.build
 * --checked writes it to libmxq_checked.so): in the linear kernels (mxq_linear with every kernel choice, the layer
 * epilogues, mxq_lm_head_accept, mxq_linear_batch, mxq_linear_bf16) every plain load and store of global memory whose
 * address is formed from an index -- X, codes, scales, Y, residual, workspace images, partial sums, correction lists,
 * tickets -- is tested against its buffer first.  An access outside it is counted, the first one recorded, and the
 * access itself redirected to a scratch area: a wrong index shows as a report, never as a fault.  (TMA copies are
 * clipped by the hardware against their tensor map.)  Same results, several times slower; meant to be run once over the
 * ragged-shape tests where no memory checker is at hand.
 * mxq_debug_bounds_report: report[0] = 1 if this library is the checked build (else 0 and the rest stays 0);
 *   report[1] = accesses refused since the last call; of the first one: report[2] = source file (0 mxq_linear.cu, 1
 *   mxq_linear_umma.cu, 2 mxq_linear_fp4.cu, 3 mxq_linear_mma.cu, 4 mxq_linear_batch.cu, 5 mxq_linear_bf16.cu),
 *   report[3] = source line, report[4] = byte offset from the buffer's base (modulo 2^64), report[5] = the buffer's size.
 *   Reading clears the record.  Synchronises with the device.
 * mxq_debug_bounds_selftest: checked build only (otherwise MXQ_ERR_SHAPE): one kernel stores 4 bytes at offset 100
 *   through the checked address of a 64-byte buffer that lies inside a larger array of the library's own (so that not
 *   even an unchecked store could leave it) and 4 bytes at offset 60; returns MXQ_OK if the array shows the second
 *   store and nothing else.  The refused store is then in mxq_debug_bounds_report. */
int mxq_debug_bounds_report(uint64_t *report);
int mxq_debug_bounds_selftest(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MXQ_H */
