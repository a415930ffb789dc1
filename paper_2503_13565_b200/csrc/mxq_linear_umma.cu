// mxq_linear for 1..16 token rows on the 5th-generation tensor cores (tcgen05) with the MXFP4 weights as a NATIVE
// operand and the activations rewritten exactly as FP8 numbers.
//
// The layer (Sec. III-D-3, Eq. 2) is  Y[m][n] = sum_blocks 2^(b-127) * sum_{k in block} X[m][k] * value(code[n][k]).
// tcgen05.mma kind::mxf8f6f4.block_scale computes exactly that shape of sum in hardware: both operands carry
// one E8M0 scale per 32 elements along K, the 32 products of a block are added, multiplied by the two
// scales and accumulated in FP32 in tensor memory.  So the weights are never decoded by the CUDA cores:
//   A (128 weight rows x 32 k, E2M1)  <- TMA copies the packed codes straight from the canonical [N][K/2]
//                                        array (tensor map type 16U4_ALIGN16B expands 8 code bytes into the
//                                        16-byte slot the tensor core reads; 128-byte swizzle)
//   SFA (one scale byte per row)      <- 4-byte cp.async per row into the 512-byte scale-factor atom, then
//                                        tcgen05.cp into tensor memory
//   B (tokens x 32 k)                 <- X is BF16, which the MMA kind does not take.  Each BF16 value is split
//                                        EXACTLY into three E5M2 numbers (three significant bits each) with
//                                        block scales 2^S, 2^(S-3), 2^(S-6); the three parts are three rows of
//                                        B, and the epilogue adds their three accumulator columns.  A block of
//                                        X whose smallest non-zero element lies more than ~29 binades under its
//                                        largest (or that holds Inf/NaN) cannot be split exactly; a CTA that
//                                        meets one computes its share with scalar FP32 code instead.
//   D (128 rows x NB columns, FP32)   <- tensor memory; tcgen05.ld in the epilogue.
//
// Work decomposition, warp roles, pipeline, programmatic dependent launch and bounded waits are those of the
// packed-FP4 kernel (mxq_linear_fp4.cu), which is the faster one at M = 1; this one splits a token into 3 rows of
// the token operand instead of 16 and wins from M = 2 on.  A stage here is 128 k (16 KB of shared memory for 8 KB of
// packed codes); the activations are split in groups of 256 k, so one "ready" barrier covers two stages.
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxq_host.h"
#include "mxq_linear_umma.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

namespace {

__device__ unsigned int g_umma_status = 0;   // sticky: bit 0 full-wait, 1 empty-wait, 2 done-wait, 3 drain-wait gave up

constexpr uint32_t kFullArrivals = 1 + 32;   // the expect_tx arrive of the TMA lane + one cp.async arrive per producer lane

// Every partial sum is bounded by sum |x w^|, which cancellation can leave up to 1/2e-3 = 500 times larger than a
// result that still has to come out finite.  So the token operand's scales carry an extra 2^-kGuard, all sums are
// formed 2^kGuard too small, and the factor is restored once, at the final store.  (What this costs at the bottom of
// the FP32 range is far below the layer's absolute tolerance.)
constexpr int kGuard = 10;
constexpr float kGuardUp = 1024.f, kGuardDown = 1.f / 1024.f;

// ---- exact split of a scaled BF16 value into E5M2 parts ---------------------------------------------------
// Largest-magnitude E5M2 number not above |v| (same sign).  Below the E5M2 normal range a non-final part
// takes nothing (the next part sees the value 8 times larger); the final part uses the subnormal grid 2^-16.
__device__ __forceinline__ float e5m2_part(float v, bool last) {
    const float a = fabsf(v);
    float t = __uint_as_float(__float_as_uint(v) & 0xFFE00000u);
    if (a < 6.103515625e-05f) t = last ? truncf(v * 65536.f) * (1.f / 65536.f) : 0.f;
    return t;
}
__device__ __forceinline__ uint32_t pack_e5m2x2(float lo, float hi) {
    uint16_t out;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(out) : "f"(hi), "f"(lo));
    return out;
}

// One 8-element unit of X (token m, k offset kk inside the CTA's range): split into parts, store into B and SFB.
// All 32 lanes call it together (the block maximum crosses the four lanes of a 32-block by shuffle).
template <int NB>
// (b_bytes, sf_bytes: sizes of the two destinations, for the bounds-checked build)
__device__ __forceinline__ bool split_unit(const uint4 raw, bool act, int m, int kk, int lane, uint8_t *gB, uint8_t *gSFB, size_t b_bytes,
                                           size_t sf_bytes) {
    (void)b_bytes;
    (void)sf_bytes;
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    bool inexact = false;
    uint32_t emax = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        emax = max(emax, (w[i] >> 7) & 0xFFu);
        emax = max(emax, (w[i] >> 23) & 0xFFu);
    }
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 1));
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 2));
    if (emax == 255u) inexact = true;              // Inf or NaN in the block
    // scale byte of the first part: the block's largest element lands in the top E5M2 binade
    const uint32_t sb1 = max(emax, 21u + kGuard) - 15u;   // >= 6 + kGuard: the third part's byte, kGuard lower, stays >= 0
    const float down = __uint_as_float((254u - sb1) << 23);   // 2^(127 - sb1)
    uint32_t part[3][2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float t[3][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t word = w[h * 2 + (i >> 1)];
            const float x = (i & 1) ? __uint_as_float(word & 0xFFFF0000u) : __uint_as_float(word << 16);
            float v = x * down;
            t[0][i] = e5m2_part(v, false);
            v = (v - t[0][i]) * 8.f;
            t[1][i] = e5m2_part(v, false);
            v = (v - t[1][i]) * 8.f;
            t[2][i] = e5m2_part(v, true);
            if (v - t[2][i] != 0.f) inexact = true;
        }
#pragma unroll
        for (int p = 0; p < 3; ++p) part[p][h] = pack_e5m2x2(t[p][0], t[p][1]) | (pack_e5m2x2(t[p][2], t[p][3]) << 16);
    }
    if (act) {
        const int j = kk >> 7;
#pragma unroll
        for (int p = 0; p < 3; ++p) {
            const int row = 3 * m + p;
            uint8_t *dst = gB + (size_t)j * (NB * 128) + (row >> 3) * 1024 + ((kk >> 4) & 7) * 128 + (row & 7) * 16 + (kk & 15);
            *reinterpret_cast<uint2 *>(MXQ_AT(dst, 8, gB, b_bytes)) = make_uint2(part[p][0], part[p][1]);
            if ((lane & 3) == 0)
                *MXQ_AT(gSFB + (size_t)j * kUmmaSfStageBytes + (row & 31) * 16 + (row >> 5) * 4 + ((kk >> 5) & 3), 1, gSFB, sf_bytes) =
                    (uint8_t)(sb1 - kGuard - 3 * p);
        }
    }
    return inexact && act;
}

// The token operand of a whole call, split once, ahead of the weight kernel (from kUmmaPresplitMinM token rows on, and at
// two rows on large matrices, where every CTA splitting its own K range costs more than one more launch in the chain).  CTA = 256 k of every token;
// a warp takes tokens warp, warp + 8, ...  The result lies in the workspace as umma_ws_bytes describes.
constexpr int kSplitWarps = 8;
template <int NB>
__global__ void __launch_bounds__(kSplitWarps * 32)
split_tokens_kernel(const __nv_bfloat16 *__restrict__ X, int M, int64_t K, int ks, uint8_t *__restrict__ ws) {
    pdl_trigger();   // the weight kernel may start at once: it streams weights until this kernel has completed
    __shared__ int s_bad;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) s_bad = 0;
    uint8_t *gSFB = ws + umma_ws_flags_bytes(ks), *gB = gSFB + (size_t)ks * kUmmaSfStageBytes;
    const int kk = (int)blockIdx.x * (2 * kUmmaStageK) + lane * 8;
    const bool act = kk < K;
    if (warp == 0) pdl_wait();   // X may be the previous kernel's output; the workspace may still be read by the previous weight kernel
    __syncthreads();
    uint4 raw[(kUmmaMaxM + kSplitWarps - 1) / kSplitWarps];
#pragma unroll
    for (int q = 0; q < (kUmmaMaxM + kSplitWarps - 1) / kSplitWarps; ++q) {
        const int m = warp + q * kSplitWarps;
        raw[q] = make_uint4(0, 0, 0, 0);
        if (m < M && act) raw[q] = ld_dep_u4(MXQ_AT(X + (int64_t)m * K + kk, 16, X, (int64_t)M * K * 2));
    }
    bool inexact = false;
#pragma unroll
    for (int q = 0; q < (kUmmaMaxM + kSplitWarps - 1) / kSplitWarps; ++q) {
        const int m = warp + q * kSplitWarps;
        if (m < M)   // uniform across the warp
            inexact |= split_unit<NB>(raw[q], act, m, kk, lane, gB, gSFB, (size_t)ks * (NB * 128), (size_t)ks * kUmmaSfStageBytes);
    }
    if (inexact) s_bad = 1;
    __syncthreads();
    const int stage = (int)blockIdx.x * 2 + (int)threadIdx.x;
    if (threadIdx.x < 2 && stage < ks) *MXQ_AT(reinterpret_cast<uint32_t *>(ws) + stage, 4, ws, umma_ws_flags_bytes(ks)) = (uint32_t)s_bad;
}

template <int NB>
cudaError_t launch_split(const __nv_bfloat16 *X, int M, int64_t K, int ks, uint8_t *ws, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((ks + 1) / 2));
    cfg.blockDim = dim3(kSplitWarps * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, split_tokens_kernel<NB>, X, M, K, ks, ws);
}

// NB: columns of the B operand / accumulator = 3 parts x tokens, rounded up to 16, 32 or 48.
// Warp roles (192 threads): warp 0 issues the MMAs and owns tensor memory; warp 1 is the producer (TMA copies of
// the codes, cp.async of the scale bytes, barrier set-up); warps 2..5 split the activations stage by stage and,
// at the end, read the accumulator (one row per thread), exchange partial results and store.
// MULTI: whether a CTA may own more than one tile (false: exactly one, and the per-tile loops fold away).
template <int NB, bool MULTI, bool BRING, int EPI>
__global__ void __launch_bounds__(kUmmaThreads)
linear_umma_kernel(const __grid_constant__ CUtensorMap tmap, const __nv_bfloat16 *__restrict__ X, int M,
                  const uint8_t *__restrict__ codes, const uint8_t *__restrict__ scales, int64_t N, int64_t K,
                  void *__restrict__ Y, int y_dtype, int split, int ring, int ks, int chunk_max, int tmem_cols, int groups,
                  int tiles, int tiles_max, const uint8_t *__restrict__ presplit, const FusedAccept fa_arg) {
    // EPI: what happens to a finished sum: stored (kEpiStore), competing for the verifier's argmax (kEpiAccept, fa.keys
    // set) or stored after a residual add or the gate / up pairing (kEpiLayer); a template parameter so that the plain
    // layer's epilogue carries none of the others
    FusedAccept fa = fa_arg;
    if (EPI != kEpiAccept) fa.keys = nullptr;
    constexpr bool bring = BRING;   // the token operand is fetched stage by stage into the ring slots (needs presplit, one tile)
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");   // needed by the first copy, 1 us from now
    const uint32_t rank = split > 1 ? cluster_rank() : 0u;
    const uint32_t group = blockIdx.x / (uint32_t)split;
    // this CTA's tiles [tile_lo, tile_lo + ntile) and, for all of them, its K range
    const int tile_lo = (int)((group * (uint32_t)tiles) / (uint32_t)groups);
    const int ntile = MULTI ? (int)(((group + 1u) * (uint32_t)tiles) / (uint32_t)groups) - tile_lo : 1;
    const int64_t n0 = (int64_t)tile_lo * kUmmaTileRows;   // first weight row of the first tile
    // everything below fits in 32 bits (the plan refuses K >= 2^30 and more than 2^20 tiles)
    const int s_begin = (int)((rank * (uint32_t)ks) / (uint32_t)split), s_end = (int)(((rank + 1u) * (uint32_t)ks) / (uint32_t)split);
    const int nst = s_end - s_begin;   // stages of this CTA (>= 1 because split <= ks)
    const int kb_row = (int)((uint32_t)K >> 5);
    const int k_begin = s_begin * kUmmaStageK;
    const int k_len = nst * kUmmaStageK;

    // carve shared memory (1024-byte aligned for the 128-byte swizzle)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base;
    const uint32_t sSFA = sA + (uint32_t)ring * kUmmaStageBytes;
    const uint32_t sB = sSFA + (uint32_t)ring * kUmmaSfStageBytes;
    // the token operand: one image and one scale atom per stage of the CTA's K range, or (bring: the operand was split
    // ahead of this kernel and the CTA owns one tile) per ring slot, fetched with the slot's weights
    const uint32_t nbslot = bring ? (uint32_t)ring : (uint32_t)chunk_max;
    const uint32_t sSFB = sB + nbslot * (NB * 128);
    const uint32_t sRecv = sSFB + nbslot * kUmmaSfStageBytes;   // [tile][split][M][rows of this rank] floats
    const uint32_t sBar = sRecv + (split > 1 ? (uint32_t)(tiles_max * M) * kUmmaRecvRows * 4u : 0u);   // no exchange, no buffer
    // barriers: full[ring], empty[ring], done, recv, ready[pairs of stages]; then the tensor-memory address and flags
    const uint32_t full0 = sBar, empty0 = sBar + (uint32_t)ring * 8u, done_bar = sBar + (uint32_t)ring * 16u;
    const uint32_t recv_bar = done_bar + 8u, ready0 = done_bar + 16u;
    const int npair = (nst + 1) >> 1;   // the activations are split 256 k (two stages) at a time
    const uint32_t sMisc = ready0 + (uint32_t)((chunk_max + 1) >> 1) * 8u;
    uint8_t *gB = gbase + (sB - base), *gSFB = gbase + (sSFB - base);
    const float *gRecv = reinterpret_cast<const float *>(gbase + (sRecv - base));
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(gbase + (sMisc - base));
    volatile int &s_fail = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 4);
    const int row_lo = (int)(rank * kUmmaTileRows) / split, row_cnt = (int)((rank + 1) * kUmmaTileRows) / split - row_lo;

    // ---- prologue: barriers, tensor memory, and the first stages of weights (they do not depend on the previous
    //      kernel, so all of this runs before griddepcontrol.wait) -----------------------------------------------
    // The CTA's work is a sequence of units (tile, stage), tile-major; unit u goes through ring slot u % ring.
    const int nunit = ntile * nst;
    const int pre = nunit < ring ? nunit : ring;
    // The SM's requests are served roughly in order, so activations asked for behind a ring full of weight copies
    // arrive late, and everything after the split waits with them.  Only the first two units are requested up
    // front; the rest of the ring follows once the activations are in, or else at a trickle.
    const int pre0 = pre < 2 ? pre : 2;
    volatile int &s_xin = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 12);   // the activations have arrived
    // producer lane l owns rows l, l + 32, l + 64, l + 96 of a tile's scale bytes
    const uint8_t *srow0 = scales + (n0 + lane) * kb_row + s_begin * 4;
    const int64_t srow_step = (int64_t)32 * kb_row;
    const uint32_t sf_lane = sSFA + (uint32_t)lane * 16u;
    auto copy_scales = [&](int t, int i, uint32_t slot) {   // unit (t, i) into ring slot `slot` (all lanes of the producer warp)
        const uint32_t dst = sf_lane + slot * kUmmaSfStageBytes;
        const uint8_t *src = srow0 + (int64_t)t * (4 * srow_step) + i * 4;
        const int rows_here = (int)min((int64_t)kUmmaTileRows, N - n0 - (int64_t)t * kUmmaTileRows);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (lane + 32 * q < rows_here) cp_async4(dst + 4 * q, MXQ_AT(src, 4, scales, N * kb_row));
            src += srow_step;
        }
        cp_async_arrive(full0 + slot * 8);
    };
    auto copy_codes = [&](int t, int i, uint32_t slot) {    // one lane
        mbar_expect_tx(full0 + slot * 8, kUmmaStageTxBytes);
        tma_load_codes(sA + slot * kUmmaStageBytes, &tmap, (s_begin + i) * kUmmaStageK, (int)n0 + t * kUmmaTileRows, full0 + slot * 8);
    };
    const uint8_t *ws_sf = presplit ? presplit + umma_ws_flags_bytes(ks) : nullptr;
    const uint8_t *ws_b = presplit ? ws_sf + (size_t)ks * kUmmaSfStageBytes : nullptr;
    auto copy_tokens = [&](int i, uint32_t slot) {     // one lane; bring only: stage i of the token operand into ring slot `slot`
        mbar_expect_tx(full0 + slot * 8, NB * 128u + kUmmaSfStageBytes);
        bulk_load(sB + slot * (NB * 128u), MXQ_AT(ws_b + (size_t)(s_begin + i) * (NB * 128u), NB * 128u, ws_b, (size_t)ks * (NB * 128u)), NB * 128u,
                  full0 + slot * 8);
        bulk_load(sSFB + slot * kUmmaSfStageBytes,
                  MXQ_AT(ws_sf + (size_t)(s_begin + i) * kUmmaSfStageBytes, kUmmaSfStageBytes, ws_sf, (size_t)ks * kUmmaSfStageBytes), kUmmaSfStageBytes,
                  full0 + slot * 8);
    };
    if (warp == 1) {
        for (int b = lane; b < 2 * ring + 2 + npair; b += 32) {
            // full: the TMA lane + 32 producer lanes; empty, done, recv: 1; ready (one per 256 k): one arrival per token
            // (with the token operand split ahead of this kernel: the one thread that requests the copies)
            const uint32_t count = b < ring ? kFullArrivals + (bring ? 1u : 0u) : (b < 2 * ring + 2 || presplit ? 1u : (uint32_t)M);
            mbar_init(sBar + (uint32_t)b * 8u, count);
        }
        if (lane == 31) {
            s_fail = 0;
            *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 8) = 0;   // s_bad
            s_xin = 0;
            if (fa.keys)
                for (int q = 0; q < 16; ++q) reinterpret_cast<volatile unsigned long long *>(gbase + (sMisc - base) + 16)[q] = 0ull;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
            if (split > 1) mbar_expect_tx(recv_bar, (uint32_t)(ntile * split * M * row_cnt) * 4u);   // every rank sends M values per tile and row
            for (int u = 0, t = 0, i = 0; u < pre0; ++u) {
                copy_codes(t, i, (uint32_t)u);
                if (++i == nst) {
                    i = 0;
                    ++t;
                }
            }
        }
    } else if (warp == 0) {
        // let the next kernel start launching at once (its CTAs take the shared memory this kernel leaves free and start
        // their own weight stream); the MMA warp does it because it has nothing urgent to do yet
        pdl_trigger();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sMisc), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Only the activation warps read what the previous kernel wrote (X, or the split kernel's output) and write what the
    // next one reads (Y).  One of them waits for it, at once; the others -- and the producer, which fetches the split
    // kernel's output only after this point -- meet it at the CTA-wide barrier below (see the packed-FP4 kernel).
    if (warp == 2) pdl_wait();
    if (split > 1) cluster_arrive();   // "my barriers exist"; the matching wait is just before the first push to a peer
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;
    if (warp == 1) {
        for (int u = 0, t = 0, i = 0; u < pre; ++u) {
            if (u >= pre0) {
                for (int spin = 0; spin < 3 && !s_xin && !bring; ++spin) __nanosleep(100);
                if (lane == 0) copy_codes(t, i, (uint32_t)u);
            }
            if (bring && lane == 0) copy_tokens(i, (uint32_t)u);
            copy_scales(t, i, (uint32_t)u);
            if (++i == nst) {
                i = 0;
                ++t;
            }
        }
    }
    if (warp == 0) {
        // ---- MMA warp: the loop is warp-uniform, one elected lane issues -------------------------------------------
        // descriptors as 32-bit halves: only the start-address field changes from MMA to MMA
        // A = E2M1 (5), B = E5M2 (1), N = NB, E8M0 scales, M = 128
        const uint32_t idesc = (5u << 7) | (1u << 10) | (((uint32_t)NB >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
        const uint32_t a_hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32), b_hi = (uint32_t)(smem_desc(0, 128, 1024, 0) >> 32);
        const uint32_t s_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);
        const uint32_t a_lo0 = (uint32_t)smem_desc(sA, 16, 1024, 2), s_lo0 = (uint32_t)smem_desc(sSFA, 0, 128, 0);
        const uint32_t b_lo0 = (uint32_t)smem_desc(sB, 128, 1024, 0), sb_lo0 = (uint32_t)smem_desc(sSFB, 0, 128, 0);
        const uint32_t t_sf0 = tmem + (uint32_t)(NB * tiles_max);   // after the accumulators: two slots of 4 + 4 scale columns
        uint32_t slot = 0, phase = 0, par = 0;
        bool ok = true;
        for (int t = 0; t < ntile && ok; ++t) {
          const uint32_t t_acc = tmem + (uint32_t)(t * NB);   // this tile's accumulator columns
          uint32_t b_lo = b_lo0, sb_lo = sb_lo0, accumulate = 0;
          for (int i = 0; i < nst; ++i) {
            // the unit's weights and scales have landed and (first tile only; the others find it done) the stage's
            // share of the activations has been split
            if ((t == 0 && !bring && !mbar_wait_relaxed(ready0 + (uint32_t)(i >> 1) * 8u, 0)) || !mbar_wait_relaxed(full0 + slot * 8, phase)) {
                if (lane == 0) {
                    atomicOr(&g_umma_status, 1u);
                    s_fail = 1;
                }
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + slot * (kUmmaStageBytes >> 4);
            const uint32_t sa_lo = s_lo0 + slot * (kUmmaSfStageBytes >> 4);
            if (bring) {   // the token operand's stage sits in the ring slot
                b_lo = b_lo0 + slot * ((NB * 128) >> 4);
                sb_lo = sb_lo0 + slot * (kUmmaSfStageBytes >> 4);
            }
            const uint32_t t_sf = t_sf0 + par * 8u;   // alternating between consecutive units
            par ^= 1u;
            if (elect_one()) {
                fence_async_proxy();   // the weight scale atom was written by cp.async
                tc_copy_sf_lohi(t_sf, sa_lo, s_hi);
                tc_copy_sf_lohi(t_sf + 4, sb_lo, s_hi);
#pragma unroll
                for (int j = 0; j < 4; ++j)   // k [32 j, 32 j + 32) of the stage: scale j of the atom on both sides
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
                        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], da, db, %5, [%7], [%8], p;\n\t}"
                        ::"r"(t_acc), "r"(a_lo + j * 2), "r"(a_hi), "r"(b_lo + j * 16), "r"(b_hi),
                        "r"(idesc | ((uint32_t)j << 4) | ((uint32_t)j << 29)), "r"(j == 0 ? accumulate : 1u), "r"(t_sf), "r"(t_sf + 4u)
                        : "memory");
                tc_commit(empty0 + slot * 8);
            }
            accumulate = 1;
            b_lo += (NB * 128) >> 4;
            sb_lo += kUmmaSfStageBytes >> 4;
            if (++slot == (uint32_t)ring) {
                slot = 0;
                phase ^= 1u;
            }
          }
        }
        __syncwarp();
        if (elect_one()) tc_commit(done_bar);
        __syncwarp();
        // tensor memory goes back as soon as the epilogue warps have read it (they arrive on barrier 2 without waiting),
        // so that nothing but their stores is left at the end of the CTA
        asm volatile("bar.sync 2, 160;" ::: "memory");
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    } else if (warp == 1) {
        // ---- producer warp: refill ring slots as the MMAs release them ----------------------------------------------
        uint32_t slot = 0, phase = 0;   // unit `pre` reuses slot 0 (pre == ring whenever the loop runs)
        int t = pre / nst, i = pre - t * nst;
        for (int u = pre; u < nunit; ++u) {
            if (!mbar_wait_relaxed(empty0 + slot * 8, phase)) {
                if (lane == 0) {
                    atomicOr(&g_umma_status, 2u);
                    s_fail = 1;
                }
                break;
            }
            if (lane == 0) {
                copy_codes(t, i, slot);
                if (bring) copy_tokens(i, slot);
            }
            copy_scales(t, i, slot);
            if (++i == nst) {
                i = 0;
                ++t;
            }
            if (++slot == (uint32_t)ring) {
                slot = 0;
                phase ^= 1u;
            }
        }
    } else {
        // ---- the four activation / epilogue warps ---------------------------------------------------------------------
        const int ct = tid - 64;                                   // 0..127
        const int row = ((warp & 3) << 5) + lane;                  // accumulator row this thread may read (its warp's quarter)
        volatile int &s_bad = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 8);
        bool inexact = false;
        if (presplit) {
            // The token operand was split by split_tokens_kernel: fetch this CTA's stages, two at a time, each pair
            // completing the "ready" barrier the MMA warp waits on (unless the producer fetches them stage by stage into
            // the ring); the flags say whether every block split exactly.
            if (ct == 0 && !bring) {
                for (int p = 0; p < npair; ++p) {
                    const uint32_t n2 = (uint32_t)min(2, nst - 2 * p), bar = ready0 + (uint32_t)p * 8u;
                    mbar_expect_tx(bar, n2 * (NB * 128u + kUmmaSfStageBytes));
                    bulk_load(sB + (uint32_t)(2 * p) * (NB * 128u),
                              MXQ_AT(ws_b + (size_t)(s_begin + 2 * p) * (NB * 128u), n2 * (NB * 128u), ws_b, (size_t)ks * (NB * 128u)), n2 * (NB * 128u), bar);
                    bulk_load(sSFB + (uint32_t)(2 * p) * kUmmaSfStageBytes,
                              MXQ_AT(ws_sf + (size_t)(s_begin + 2 * p) * kUmmaSfStageBytes, n2 * kUmmaSfStageBytes, ws_sf, (size_t)ks * kUmmaSfStageBytes),
                              n2 * kUmmaSfStageBytes, bar);
                }
                s_xin = 1;   // lets the producer request the rest of the ring
            }
            const uint32_t *flags = reinterpret_cast<const uint32_t *>(presplit);
            for (int i = ct; i < nst; i += 128) inexact |= ld_dep_u32(MXQ_AT(flags + s_begin + i, 4, flags, umma_ws_flags_bytes(ks))) != 0u;
        } else {
            // Groups of 32 units (256 k of one token, one warp; a unit is 8 elements, one lane) in order of K, so that
            // the MMA warp can start on the first stages while later ones are being split.  Group G: pair of stages
            // G / M, token G % M; the last pair is half full when the CTA has an odd number of stages.  All of this
            // is uniform across a warp.
            const int ngroups = npair * M;
            const __nv_bfloat16 *xbase = X + k_begin;
            const int cw = ct >> 5;
            constexpr int kBatch = 4;   // loads in flight per thread
            for (int G0 = 0; G0 < ngroups; G0 += 4 * kBatch) {
                uint4 raw[kBatch];
                int mm[kBatch], kk[kBatch], pair[kBatch];
                bool act[kBatch];
#pragma unroll
                for (int b = 0; b < kBatch; ++b) {   // all loads of the batch first
                    const int G = G0 + 4 * b + cw;
                    mm[b] = kk[b] = pair[b] = 0;
                    act[b] = false;
                    raw[b] = make_uint4(0, 0, 0, 0);
                    if (G < ngroups) {
                        pair[b] = G / M;
                        mm[b] = G - pair[b] * M;
                        kk[b] = pair[b] * (2 * kUmmaStageK) + lane * 8;
                        act[b] = kk[b] < k_len;
                        if (act[b]) raw[b] = ld_dep_u4(MXQ_AT(xbase + (int64_t)mm[b] * K + kk[b], 16, X, (int64_t)M * K * 2));
                    }
                }
#pragma unroll
                for (int b = 0; b < kBatch; ++b)
                    if (G0 + 4 * b + cw < ngroups) {   // uniform across the warp
                        inexact |= split_unit<NB>(raw[b], act[b], mm[b], kk[b], lane, gB, gSFB, (size_t)nbslot * (NB * 128), (size_t)nbslot * kUmmaSfStageBytes);
                        if (G0 == 0 && b == 0 && ct == 0) s_xin = 1;   // lets the producer request the rest of the ring
                        fence_async_proxy();   // ordinary stores, read by the tensor core
                        __syncwarp();
                        if (lane == 0) mbar_arrive(ready0 + (uint32_t)pair[b] * 8u);
                    }
            }
        }
        if (inexact) s_bad = 1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int bad = s_bad;

        // ---- epilogue: accumulator row -> registers; the three parts of a token are three neighbouring columns -------
        constexpr int MT = NB / kUmmaParts;         // token slots per tile (5, 10 or 16)
        // layer epilogues: the residual values this thread will add to its first tile's sums, requested before the wait
        float res[MT];   // (unused, and optimised away, in the other epilogues)
        if (EPI == kEpiLayer && split == 1) {
            const int64_t n_first = (int64_t)tile_lo * kUmmaTileRows + row;
            layer_prefetch<MT>(fa, y_dtype, M, n_first, N, n_first < N, res);
        }
        if (!mbar_wait_relaxed(done_bar, 0)) {
            atomicOr(&g_umma_status, 4u);
            s_fail = 1;
        }
        tc_fence_after();
        // Tile by tile: this thread's row of the accumulator -> registers -> direct store (split == 1) or, for the sum over
        // the cluster in a fixed order, a push to the row's owner.  Rank q owns rows [q*128/split, (q+1)*128/split) of every
        // tile of the group: every CTA pushes its partial results for those rows into q's shared memory (slot = tile,
        // sender's rank) with stores that count on q's mbarrier; q waits for all of them and adds them in a fixed
        // order.  No CTA reads a peer's memory, and a CTA leaves only after everything addressed to it has arrived.
        const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int cnt_max = (kUmmaTileRows + split - 1) / split;
        const uint32_t owner = (uint32_t)(((row + 1) * split - 1) / kUmmaTileRows);
        const int rr = row - (int)(owner * kUmmaTileRows) / split;
        const uint32_t remote = peer_saddr(sRecv, owner), remote_bar = peer_saddr(recv_bar, owner);
        if (split > 1) cluster_wait();   // every CTA of the cluster has initialised its barriers (they arrived long ago)
        // fused verification: instead of being stored, a finished value competes for its token row's running maximum
        unsigned long long *s_keys = reinterpret_cast<unsigned long long *>(gbase + (sMisc - base) + 16);
        // (a thread meets its candidates in ascending index order, so "strictly greater" keeps the lowest index; NaN and
        // -inf never pass the test)
        float bestv[MT];
        uint32_t besti[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            bestv[m] = -INFINITY;
            besti[m] = 0xFFFFFFFFu;
        }
        for (int t = 0; t < ntile; ++t) {
            float yt[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) yt[m] = 0.f;
            if (!bad) {
#pragma unroll
                for (int c = 0; c < NB / 16; ++c) {
                    float d[16];
                    tc_load16(t_row + t * NB + c * 16, d);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int col = c * 16 + j;
                        if (col < MT * kUmmaParts) yt[col / kUmmaParts] += d[j];   // fixed order: parts 0, 1, 2
                    }
                }
            } else {
                // Scalar path for a K range whose X cannot be rewritten exactly (the MMA results are ignored).
                const int64_t n = n0 + (int64_t)t * kUmmaTileRows + row;
                float acc[kUmmaMaxM];
#pragma unroll
                for (int m = 0; m < kUmmaMaxM; ++m) acc[m] = 0.f;
                if (n < N) {
                    const uint4 *crow = reinterpret_cast<const uint4 *>(codes + n * (K / 2));
                    const uint8_t *srw = scales + n * kb_row;
                    for (int blk = k_begin / 32; blk < (k_begin + k_len) / 32; ++blk) {
                        const uint4 c = ld_stream_u4(MXQ_AT(crow + blk, 16, codes, N * (K / 2)));
                        const float sc = e8m0_to_float(*MXQ_AT(srw + blk, 1, scales, N * kb_row)) * kGuardDown;
                        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
                        float part[kUmmaMaxM];
#pragma unroll
                        for (int m = 0; m < kUmmaMaxM; ++m) part[m] = 0.f;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 wv = __half22float2(e2m1x2_to_half2((w[q] >> (8 * i)) & 0xFFu));
                                const int64_t k = (int64_t)blk * 32 + q * 8 + i * 2;
#pragma unroll
                                for (int m = 0; m < kUmmaMaxM; ++m)
                                    if (m < M) {
                                        const uint32_t xb = ld_dep_u32(MXQ_AT(X + (int64_t)m * K + k, 4, X, (int64_t)M * K * 2));
                                        part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                                        part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                                    }
                            }
#pragma unroll
                        for (int m = 0; m < kUmmaMaxM; ++m) acc[m] = fmaf(part[m], sc, acc[m]);
                    }
                }
#pragma unroll
                for (int m = 0; m < MT; ++m) yt[m] = acc[m];
            }
            if (t == ntile - 1) {
                // the accumulators have been read (or are not needed): the MMA warp may give tensor memory back
                tc_fence_before();
                asm volatile("bar.arrive 2, 160;" ::: "memory");
            }
            if (s_fail) {
#pragma unroll
                for (int m = 0; m < MT; ++m) yt[m] = __uint_as_float(0x7FC00000u);
            }
            if (split == 1) {
                const int64_t n = n0 + (int64_t)t * kUmmaTileRows + row;
                if (EPI == kEpiLayer) {
                    // (gate / up pairing: the partner row's sum sits in the neighbouring lane)
#pragma unroll
                    for (int m = 0; m < MT; ++m) yt[m] *= kGuardUp;
                    layer_emit<MT>(fa, Y, y_dtype, M, n, N, n < N, yt, res, 1);
                    if (t + 1 < ntile) layer_prefetch<MT>(fa, y_dtype, M, n + kUmmaTileRows, N, n + kUmmaTileRows < N, res);
                } else if (n < N)
#pragma unroll
                    for (int m = 0; m < MT; ++m)
                        if (m < M) {
                            if (fa.keys) {
                                const float v = yt[m] * kGuardUp;
                                if (v > bestv[m]) {
                                    bestv[m] = v;
                                    besti[m] = (uint32_t)n;
                                }
                            } else {
                                store_out(Y, y_dtype, (int64_t)m * N + n, yt[m] * kGuardUp, (int64_t)M * N);
                            }
                        }
            } else {
#pragma unroll
                for (int m = 0; m < MT; ++m)
                    if (m < M) st_async_f32(remote + (uint32_t)(((t * split + (int)rank) * M + m) * cnt_max + rr) * 4u, yt[m], remote_bar);
            }
        }
        if (split > 1) {
            float res_s[TokenScatter<MT>::PH];   // (power-of-two clusters: the residual values of this lane's share of the token rows)
            if (EPI == kEpiLayer && (split & (split - 1)) == 0)
                scatter_prefetch<MT>(fa, y_dtype, M, split, ct & (split - 1), (int64_t)tile_lo * kUmmaTileRows + row_lo + ct / split, N, res_s);
            if (!mbar_wait_relaxed(recv_bar, 0)) {
                atomicOr(&g_umma_status, 16u);
                s_fail = 1;
            }
            const float poison = s_fail ? __uint_as_float(0x7FC00000u) : 0.f;
            // (Funnelling the few results of a one-token call through one warp, so that only one warp has stores in flight
            // when the CTA ends, was measured: the serial sums cost more than the shorter launch-to-launch gap saves.)
            const int total = ntile * M * row_cnt;
            if ((split & (split - 1)) != 0) {
                for (int idx = ct; idx < total; idx += 128) {
                    const int t = idx / (M * row_cnt), rem = idx - t * (M * row_cnt);
                    const int m = rem / row_cnt, r = rem - m * row_cnt;
                    float acc = 0.f;
                    for (int j = 0; j < split; ++j) acc += gRecv[((t * split + j) * M + m) * cnt_max + r];
                    const int64_t n = n0 + (int64_t)t * kUmmaTileRows + row_lo + r;
                    if (n < N) {
                        if (EPI == kEpiLayer) {
                            // (gate / up calls are planned with power-of-two clusters and never come here)
                            const int64_t at = (int64_t)m * N + n;
                            store_out(Y, y_dtype, at, acc * kGuardUp + poison + load_in(fa.residual, y_dtype, at, (int64_t)M * N), (int64_t)M * N);
                        } else if (fa.keys) {
                            const unsigned long long key = argmax_key(acc * kGuardUp + poison, (uint32_t)n);
                            if (key) atomicMax(s_keys + m, key);   // (rare decomposition: straight into shared memory)
                        } else {
                            store_out(Y, y_dtype, (int64_t)m * N + n, acc * kGuardUp + poison, (int64_t)M * N);
                        }
                    }
                }
            } else {
                // power-of-two cluster: one thread per (row ct / split, sender ct % split), the senders of a row in neighbouring
                // lanes; the order of additions is fixed by the lane pattern
                const int r = ct / split, j = ct & (split - 1);
                for (int t = 0; t < ntile; ++t) {
                    const int64_t n = n0 + (int64_t)t * kUmmaTileRows + row_lo + r;
                    if (EPI != kEpiAccept) {
                        // plain store and layer epilogues: reduce-scatter over the token rows, every lane finishes its share
                        scatter_sum_store<MT, EPI>(gRecv + ((t * split + j) * M) * cnt_max + r, cnt_max, M, split, j, n, N, kGuardUp, poison,
                                                   fa, Y, y_dtype, res_s);
                        if (EPI == kEpiLayer && t + 1 < ntile) scatter_prefetch<MT>(fa, y_dtype, M, split, j, n + kUmmaTileRows, N, res_s);
                        continue;
                    }
                    // fused verification: all-to-all butterfly, every lane ends with all token rows (the running maxima are
                    // kept per token row); all loads, then all shuffles, then all uses: the token rows are independent of each other
                    float v[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) v[m] = m < M ? gRecv[((t * split + j) * M + m) * cnt_max + r] : 0.f;
                    for (int o = 1; o < split; o <<= 1) {
#pragma unroll
                        for (int m = 0; m < MT; ++m) v[m] += __shfl_xor_sync(0xffffffffu, v[m], o);
                    }
                    if (j == 0 && n < N) {
#pragma unroll
                        for (int m = 0; m < MT; ++m)
                            if (m < M) {
                                const float w = v[m] * kGuardUp + poison;
                                if (fa.keys) {
                                    if (w > bestv[m]) {
                                        bestv[m] = w;
                                        besti[m] = (uint32_t)n;
                                    }
                                } else {
                                    store_out(Y, y_dtype, (int64_t)m * N + n, w, (int64_t)M * N);
                                }
                            }
                    }
                }
            }
        }
        if (fa.keys) {
#pragma unroll
            for (int m = 0; m < MT; ++m)
                if (m < M) {
                    const unsigned long long k = warp_max_key(besti[m] != 0xFFFFFFFFu ? argmax_key(bestv[m], besti[m]) : 0ull);
                    if (lane == 0 && k) atomicMax(s_keys + m, k);
                }
            fused_accept_finish(fa, s_keys, M, gridDim.x, ct);
        }
    }

    if (split > 1 && warp < 2) cluster_wait();   // pairs with the arrive in the prologue (the other warps waited before their push)
}

template <int NB, bool MULTI, bool BRING, int EPI>
cudaError_t launch_umma(const UmmaPlan &p, const CUtensorMap &map, const void *X, const uint8_t *codes,
                       const uint8_t *scales, void *Y, int y_dtype, const uint8_t *presplit, cudaStream_t stream, const FusedAccept &fa) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_umma_kernel<NB, MULTI, BRING, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kUmmaSmemLimit);
        if (e != cudaSuccess) return e;
        // all of the SM's L1/shared array as shared memory: how many CTAs (of this and of the next kernel) fit on an
        // SM is what decides how early the next kernel's weight stream can start
        e = cudaFuncSetAttribute(linear_umma_kernel<NB, MULTI, BRING, EPI>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(kUmmaThreads);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (p.split > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)p.split;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl_enabled()) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, linear_umma_kernel<NB, MULTI, BRING, EPI>, map, (const __nv_bfloat16 *)X, p.M, codes, scales, p.N, p.K,
                              Y, y_dtype, p.split, p.ring, p.ks, p.chunk_max, p.tmem_cols, p.groups, p.tiles, p.tiles_max, presplit, fa);
}

}  // namespace

// token rows from which the token operand is split ahead of the weight kernel when a workspace is there
static int presplit_min_m() {
    const int forced = layout_override().presplit_min_m;
    return forced > 0 ? forced : kUmmaPresplitMinM;
}
static bool presplit_wanted(int M, int64_t N, int64_t K) {
    const int min_m = presplit_min_m();
    return M >= min_m || (min_m == kUmmaPresplitMinM && M == 2 && N * K >= kUmmaPresplitTwoRowsMinWeights);
}

bool linear_umma_plan(int M, int64_t N, int64_t K, UmmaPlan &p, bool with_workspace, bool pow2_split, bool one_wave) {
    if (M < 1 || M > kUmmaMaxM || N < 1 || K < 128 || (K % 128) != 0) return false;
    if (K > 0x3FFFFFFF || N > 0x7FFFFFFF) return false;
    p.presplit = with_workspace && presplit_wanted(M, N, K) ? 1 : 0;
    p.pow2_split = pow2_split ? 1 : 0;
    p.layer_tiles = 0;
    p.one_wave = one_wave ? 1 : 0;
    p.M = M;
    p.N = N;
    p.K = K;
    p.nb = umma_nb(M);
    p.ks = (int)(K / kUmmaStageK);
    p.tiles = (int)((N + kUmmaTileRows - 1) / kUmmaTileRows);
    const LayoutOverride o = layout_override();
    return umma_layout(p, sm_count(), o.split, o.ring, o.tiles, o.operand_through_ring);
}

template <int NB>
static cudaError_t pick_umma(const UmmaPlan &p, bool bring, const CUtensorMap &map, const void *X, const uint8_t *codes,
                             const uint8_t *scales, void *Y, int y_dtype, const uint8_t *ws, cudaStream_t stream, const FusedAccept &fa) {
    const bool multi = p.tiles_max > 1;
#define MXQ_UMMA_PICK(EPI)                                                                                                    \
    return multi ? (bring ? launch_umma<NB, true, true, EPI>(p, map, X, codes, scales, Y, y_dtype, ws, stream, fa)           \
                          : launch_umma<NB, true, false, EPI>(p, map, X, codes, scales, Y, y_dtype, ws, stream, fa))         \
                 : (bring ? launch_umma<NB, false, true, EPI>(p, map, X, codes, scales, Y, y_dtype, ws, stream, fa)          \
                          : launch_umma<NB, false, false, EPI>(p, map, X, codes, scales, Y, y_dtype, ws, stream, fa))
    switch (epilogue_kind(fa)) {
        case kEpiAccept: MXQ_UMMA_PICK(kEpiAccept);
        case kEpiLayer: MXQ_UMMA_PICK(kEpiLayer);
        default: MXQ_UMMA_PICK(kEpiStore);
    }
#undef MXQ_UMMA_PICK
}

size_t linear_umma_workspace_bytes(int M, int64_t K) {
    // (two token rows: used on large matrices only, see presplit_wanted; the size does not depend on N)
    if ((M < presplit_min_m() && !(M == 2 && presplit_min_m() == kUmmaPresplitMinM)) || M > kUmmaMaxM || K < 128 || (K % 128) != 0 ||
        K > 0x3FFFFFFF)
        return 0;
    return umma_ws_bytes(umma_nb(M), (int)(K / kUmmaStageK));
}

cudaError_t linear_umma_launch(const UmmaPlan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                              int y_dtype, void *workspace, size_t workspace_bytes, cudaStream_t stream, const FusedAccept *fused) {
    if (fused && fused->swiglu && ((p.split & (p.split - 1)) != 0 || (p.N & 1))) return cudaErrorNotSupported;   // see linear_umma_plan's pow2_split
    CUtensorMap map;
    if (!codes_tensor_map(codes, p.N, p.K, /*expand_fp4=*/true, &map)) return cudaErrorNotSupported;
    // a workspace that is large enough (and aligned for bulk copies) lets the token operand be split once per call
    const size_t need = umma_ws_bytes(p.nb, p.ks);
    uint8_t *ws = nullptr;
    if (p.presplit && workspace && workspace_bytes >= need && (reinterpret_cast<uintptr_t>(workspace) & 15u) == 0)
        ws = static_cast<uint8_t *>(workspace);
    if (p.presplit && !ws) {   // planned for a workspace that is not there: plan again without
        UmmaPlan q;
        if (!linear_umma_plan(p.M, p.N, p.K, q, false, p.pow2_split != 0, p.one_wave != 0)) return cudaErrorNotSupported;
        return linear_umma_launch(q, X, codes, scales, Y, y_dtype, nullptr, 0, stream, fused);
    }
    if (ws) {
        const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(X);
        const cudaError_t e = p.nb == 16   ? launch_split<16>(x, p.M, p.K, p.ks, ws, stream)
                              : p.nb == 32 ? launch_split<32>(x, p.M, p.K, p.ks, ws, stream)
                                           : launch_split<48>(x, p.M, p.K, p.ks, ws, stream);
        if (e != cudaSuccess) return e;
    }
    const bool bring = ws && p.bring;
    const FusedAccept fa = fused ? *fused : FusedAccept{};
    switch (p.nb) {
        case 16:
            return pick_umma<16>(p, bring, map, X, codes, scales, Y, y_dtype, ws, stream, fa);
        case 32:
            return pick_umma<32>(p, bring, map, X, codes, scales, Y, y_dtype, ws, stream, fa);
        default:
            return pick_umma<48>(p, bring, map, X, codes, scales, Y, y_dtype, ws, stream, fa);
    }
}

bool linear_umma_available() { return tensor_map_available(); }

// returns and clears this kernel's sticky status word (see mxq_linear_device_status)
static int linear_umma_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_umma_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_umma_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

MXQ_BOUNDS_TU(bounds_take_linear_umma)

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)
int mxq_linear_device_status(uint32_t *status_host) {
    if (!status_host) return MXQ_ERR_NULL;
    uint32_t v = 0, v4 = 0, vb = 0, vp = 0, vm = 0;
    int rc = mxq::linear_umma_take_status(&v);
    if (rc != MXQ_OK) return rc;
    rc = mxq::linear_fp4_take_status(&v4);
    if (rc != MXQ_OK) return rc;
    rc = mxq::linear_bf16_take_status(&vb);
    if (rc != MXQ_OK) return rc;
    rc = mxq::linear_batch_take_status(&vp);
    if (rc != MXQ_OK) return rc;
    rc = mxq::linear_mma_take_status(&vm);
    if (rc != MXQ_OK) return rc;
    *status_host = v | (v4 << 8) | (vb << 16) | (vp << 24) | (vm << 28);
    return MXQ_OK;
}

int mxq_debug_bounds_report(uint64_t *report) {
    if (!report) return MXQ_ERR_NULL;
    for (int i = 0; i < 6; ++i) report[i] = 0;
#ifdef MXQ_DEBUG_BOUNDS
    report[0] = 1;
#endif
    int (*const take[6])(unsigned long long *) = {mxq::bounds_take_linear,     mxq::bounds_take_linear_umma,  mxq::bounds_take_linear_fp4,
                                                 mxq::bounds_take_linear_mma, mxq::bounds_take_linear_batch, mxq::bounds_take_linear_bf16};
    for (int u = 0; u < 6; ++u) {
        unsigned long long r[4] = {0, 0, 0, 0};
        const int rc = take[u](r);
        if (rc != MXQ_OK) return rc;
        if (r[0] != 0 && report[1] == 0) {
            report[2] = (uint64_t)u;
            report[3] = r[1];
            report[4] = r[2];
            report[5] = r[3];
        }
        report[1] += r[0];
    }
    return MXQ_OK;
}
#pragma GCC visibility pop
}
