// Host-side helpers: argument validation and launch plumbing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxq.h"

namespace mxq {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool shape_ok(int64_t N, int64_t K) { return N >= 1 && K >= 32 && (K % 32) == 0; }
inline int launch_status() { return cudaGetLastError() == cudaSuccess ? MXQ_OK : MXQ_ERR_CUDA; }

// number of SMs of the current device (cached per device)
int sm_count();
// whether mxq_linear launches carry the programmatic-dependent-launch attribute
bool pdl_enabled();

// mxq_set_linear_layout: layout parameters of the tcgen05 kernels forced by a test or a comparison (0 / -1 = the
// heuristic decides); see include/mxq.h
struct LayoutOverride {
    int split, ring, tiles;      // > 0: CTAs per cluster, ring slots, tiles per CTA (where feasible)
    int operand_through_ring;    // FP8-operand kernel with a workspace: 0 = token operand resident, 1 = through the ring, -1 = heuristic
    int presplit_min_m;          // FP8-operand kernel: token rows from which the operand is split ahead of the weight kernel (> 16: never)
    int batch_ring, batch_ctas_per_sm;   // mxq_linear_batch: ring slots per CTA, CTAs per SM
};
LayoutOverride layout_override();

// Vocabulary projection fused with the greedy verification (Sec. III-A, III-B).  With `keys` set a tcgen05 kernel
// does not store Y: every finished logit (token row m, vocabulary index n) competes for keys[m], the last CTA to
// deliver turns the keys into the verifier's tokens, walks the draft and leaves keys and ticket zero for the next call.
struct FusedAccept {
    unsigned long long *keys;   // running maxima as (ordered value, ~index), 0 = nothing yet, one per 128 bytes; nullptr: plain layer
    unsigned int *ticket;       // CTAs that have delivered
    const int32_t *draft;       // [T] speculated tokens
    int32_t *verifier;          // [R] out: argmax of every row (may be nullptr)
    int32_t *accept_len;        // [1] out: G
    int32_t *next_token;        // [1] out: the verifier's token at position G, -1 if there is no such row
    int T;
    // Layer epilogues (keys == nullptr; Sec. III-D-2: operators fused into the linear layers).  A finished sum is
    // stored after one more step:
    const void *residual;       // [M][N] in Y's type, added to the sum (may be Y itself); nullptr: none
    int swiglu;                 // rows 2i / 2i+1 of W are gate / up row i: Y[m][i] = silu(sum 2i) * sum(2i+1), Y is [M][N/2]
};
// which epilogue a tcgen05 kernel is compiled for
enum { kEpiStore = 0, kEpiAccept = 1, kEpiLayer = 2 };
inline int epilogue_kind(const FusedAccept &fa) { return fa.keys ? kEpiAccept : (fa.residual || fa.swiglu ? kEpiLayer : kEpiStore); }

struct LinearPlan;
// tensor-core path of mxq_linear (mxq_linear_mma.cu): false if the shape is not covered
bool linear_mma_plan(int M, int64_t N, int64_t K, LinearPlan &plan);
size_t linear_mma_workspace_bytes(const LinearPlan &plan);
cudaError_t linear_mma_launch(const LinearPlan &plan, const void *X, const uint8_t *codes, const uint8_t *scales,
                              void *Y, int y_dtype, void *workspace, cudaStream_t stream);

struct UmmaPlan;
// tcgen05 path of mxq_linear (mxq_linear_umma.cu): false if the shape is not covered
bool linear_umma_available();
// with_workspace: plan for a token operand split ahead of the weight kernel (from 3 token rows on)
// pow2_split: only cluster sizes that are powers of two (what the gate / up epilogue needs: the two rows of a pair
// then end up in one warp)
// one_wave: never more CTAs than fit on the GPU at once (the fused verification pays per CTA: keys, ticket)
bool linear_umma_plan(int M, int64_t N, int64_t K, UmmaPlan &plan, bool with_workspace, bool pow2_split = false, bool one_wave = false);
// workspace: optional; with linear_umma_workspace_bytes(M, K) bytes (0: not used for this M) the token operand is split
// once per call by a kernel of its own instead of by every CTA of the weight kernel
size_t linear_umma_workspace_bytes(int M, int64_t K);
cudaError_t linear_umma_launch(const UmmaPlan &plan, const void *X, const uint8_t *codes, const uint8_t *scales,
                               void *Y, int y_dtype, void *workspace, size_t workspace_bytes, cudaStream_t stream,
                               const FusedAccept *fused = nullptr);

struct Fp4Plan;
// tcgen05 path with packed 4-bit operands on both sides, M <= 4 (mxq_linear_fp4.cu)
bool linear_fp4_plan(int M, int64_t N, int64_t K, Fp4Plan &plan, bool pow2_split = false);
cudaError_t linear_fp4_launch(const Fp4Plan &plan, const void *X, const uint8_t *codes, const uint8_t *scales,
                              void *Y, int y_dtype, cudaStream_t stream, const FusedAccept *fused = nullptr);
int linear_fp4_take_status(uint32_t *out);
int linear_mma_take_status(uint32_t *out);    // the mma.sync kernel (mxq_linear_mma.cu)
int linear_batch_take_status(uint32_t *out);  // the persistent multi-layer kernel (mxq_linear_batch.cu)
int linear_bf16_take_status(uint32_t *out);   // the BF16-weight comparison kernel (mxq_linear_bf16.cu)

// Bounds-checked build (-DMXQ_DEBUG_BOUNDS): every translation unit with linear kernels keeps a record of global accesses
// that fell outside their buffer (out[0] = how many; of the first: out[1] source line, out[2] byte offset, out[3] extent);
// reading clears it.  In the ordinary build the functions report zeros.
int bounds_take_linear(unsigned long long *out);        // mxq_linear.cu
int bounds_take_linear_umma(unsigned long long *out);   // mxq_linear_umma.cu
int bounds_take_linear_fp4(unsigned long long *out);    // mxq_linear_fp4.cu
int bounds_take_linear_mma(unsigned long long *out);    // mxq_linear_mma.cu
int bounds_take_linear_batch(unsigned long long *out);  // mxq_linear_batch.cu
int bounds_take_linear_bf16(unsigned long long *out);   // mxq_linear_bf16.cu

}  // namespace mxq
