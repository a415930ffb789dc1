// mxq_linear for 1..4 token rows on the 5th-generation tensor cores with BOTH operands in packed 4-bit form
// (tcgen05.mma kind::mxf4.block_scale, 64 k per instruction, one E8M0 scale per 32 k on each side).
//
// The layer (Sec. III-D-3, Eq. 2) is  Y[m][n] = sum_blocks 2^(b-127) * sum_{k in block} X[m][k] * value(code[n][k]).
//   A (128 weight rows x 64 k)  <- the canonical codes array [N][K/2] as it is: one TMA box of 128 rows x 128
//                                  bytes (256 k, 128-byte swizzle) per stage; shared memory holds the weights at
//                                  4 bits each, so a CTA can keep its whole K range in flight
//   SFA                         <- the canonical scale bytes, 4-byte cp.async per row into 512-byte scale atoms,
//                                  tcgen05.cp into tensor memory
//   B (16 columns per token)    <- a BF16 activation is not an E2M1 number, but within a 32-block it is an
//                                  integer multiple of a common power of two: relative to the block's largest
//                                  exponent every element is a 32-bit fixed-point number, i.e. 16 radix-4
//                                  digits.  Digit plane p (digits 0..3 are the E2M1 values 0, 1, 2, 3, with the
//                                  element's sign) is column p of the token, with block scale 2^(S - 2p).  The
//                                  tensor core multiplies every plane with the weights exactly; the epilogue
//                                  adds the 16 accumulator columns.  Elements more than 24 binades below their
//                                  block's maximum would lose bits (so would Inf/NaN): a CTA that meets one
//                                  computes its share with scalar FP32 code instead.
//   D (128 rows x 16 M columns, FP32) <- tensor memory; tcgen05.ld in the epilogue.
//
// Work decomposition, pipeline, programmatic dependent launch and bounded waits are those of the FP8-operand
// kernel (mxq_linear_umma.cu): one CTA per (128-row tile, K range), the CTAs of a tile form a cluster and add
// their partial results through distributed shared memory in rank order; warp 0 issues the MMAs, warp 1 the
// TMA copies, warps 2-3 the scale copies; the first `ring` stages are requested before griddepcontrol.wait.
#include <cstdlib>
#include <cstring>

#include "mxq_host.h"
#include "mxq_linear_fp4.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

namespace {

__device__ unsigned int g_fp4_status = 0;   // sticky: bit 0 full-wait, 1 empty-wait, 2 done-wait, 3 drain-wait gave up

constexpr uint32_t kFullArrivals = 1 + 64;   // TMA thread's expect_tx arrive + one cp.async arrive per scale thread

// Every partial sum is bounded by sum |x w^|, which cancellation can leave up to 1/2e-3 = 500 times larger than a
// result that still has to come out finite.  So the token operand's scales carry an extra 2^-kGuard, all sums are
// formed 2^kGuard too small, and the factor is restored once, at the final store.  (What this costs at the bottom of
// the FP32 range is far below the layer's absolute tolerance.)
constexpr int kGuard = 10;
constexpr float kGuardUp = 1024.f, kGuardDown = 1.f / 1024.f;

// 8 radix-4 digits (16 bits) -> 8 nibbles holding the digits' E2M1 codes (0, 1, 2, 3 -> 0000, 0010, 0100, 0101)
__device__ __forceinline__ uint32_t digit_codes(uint32_t v16, uint32_t sign_nibbles) {
    uint32_t w = (v16 | (v16 << 8)) & 0x00FF00FFu;
    w = (w | (w << 4)) & 0x0F0F0F0Fu;
    w = (w | (w << 2)) & 0x33333333u;
    const uint32_t d1 = (w >> 1) & 0x11111111u, d0 = w & 0x11111111u;
    return (d1 << 2) | ((d0 & ~d1) << 1) | (d0 & d1) | sign_nibbles;
}

// in place: x[j] nibble i  <-  x[i] nibble j
__device__ __forceinline__ void transpose_nibbles8(uint32_t (&x)[8]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = x[i], b = x[i + 4];
        x[i] = __byte_perm(a, b, 0x5410);
        x[i + 4] = __byte_perm(a, b, 0x7632);
    }
#pragma unroll
    for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const uint32_t a = x[4 * g + i], b = x[4 * g + i + 2];
            x[4 * g + i] = __byte_perm(a, b, 0x6240);
            x[4 * g + i + 2] = __byte_perm(a, b, 0x7351);
        }
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        const uint32_t a = x[i], b = x[i + 1];
        x[i] = (a & 0x0F0F0F0Fu) | ((b & 0x0F0F0F0Fu) << 4);
        x[i + 1] = ((a >> 4) & 0x0F0F0F0Fu) | (b & 0xF0F0F0F0u);
    }
}

// One 8-element unit of X (token m, k offset kk inside the CTA's range) -> 16 digit planes in B and, from one lane
// of the four that share a 32-block, the planes' 16 scale bytes.  All 32 lanes call it together.
template <int NB>
__device__ __forceinline__ bool split_unit(const uint4 raw, bool act, int m, int kk, int lane, uint8_t *gB, uint8_t *gSFB) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t emax = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        emax = max(emax, (w[i] >> 7) & 0xFFu);
        emax = max(emax, (w[i] >> 23) & 0xFFu);
    }
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 1));
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 2));
    bool inexact = emax == 255u;                        // Inf or NaN in the block
    const uint32_t top = max(emax, 31u + kGuard);       // plane p carries 2^(top - 128 - 2p); its scale byte is kGuard lower
    uint32_t hi[8], lo[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t bits = (i & 1) ? (w[i >> 1] >> 16) : (w[i >> 1] & 0xFFFFu);
        const uint32_t e = (bits >> 7) & 0xFFu;
        const uint32_t sig = (bits & 0x7Fu) | (e ? 0x80u : 0u);             // 8-bit significand
        const int sh = 24 - (int)(top - max(e, 1u));                         // position of its lowest bit in the 32-bit fixed point
        const uint32_t down = (uint32_t)min(max(-sh, 0), 8);
        const uint32_t f = sh >= 0 ? (sig << sh) : (sig >> down);
        if (sh < 0 && (f << down) != sig) inexact = true;                    // bits fell off the bottom
        const uint32_t sgn = (bits & 0x8000u) ? 0x88888888u : 0u;
        hi[i] = digit_codes(f >> 16, sgn);       // nibble j = plane 7 - j
        lo[i] = digit_codes(f & 0xFFFFu, sgn);   // nibble j = plane 15 - j
    }
    transpose_nibbles8(hi);   // now hi[j] = plane 7 - j, nibble i = element i
    transpose_nibbles8(lo);
    if (act) {
        const int j = kk >> 8, kin = kk & 255;
        uint8_t *dst = gB + (size_t)j * (NB * 128) + (size_t)(m * 2) * 1024 + (kin >> 5) * 128 + ((kin & 31) >> 1);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            *reinterpret_cast<uint32_t *>(dst + (7 - q) * 16) = hi[q];           // planes 0..7: row group 2m, row 7 - q
            *reinterpret_cast<uint32_t *>(dst + 1024 + (7 - q) * 16) = lo[q];    // planes 8..15: row group 2m + 1
        }
        if ((lane & 3) == 0) {
            const int kb = kin >> 5;
            uint8_t *sf = gSFB + (size_t)j * kFp4SfStageBytes + (kb >> 2) * 512 + (kb & 3);
#pragma unroll
            for (int p = 0; p < kFp4Planes; ++p) {
                const int row = kFp4Planes * m + p;
                sf[(row & 31) * 16 + (row >> 5) * 4] = (uint8_t)(top - 1 - kGuard - 2 * p);
            }
        }
    }
    return inexact && act;
}

// NB: columns of the B operand / accumulator = 16 planes x tokens (16, 32 or 64).
template <int NB>
__global__ void __launch_bounds__(kFp4Threads)
linear_fp4_kernel(const __grid_constant__ CUtensorMap tmap, const __nv_bfloat16 *__restrict__ X, int M,
                  const uint8_t *__restrict__ codes, const uint8_t *__restrict__ scales, int64_t N, int64_t K,
                  void *__restrict__ Y, int y_dtype, int split, int ring, int ks, int chunk_max, int tmem_cols) {
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = split > 1 ? cluster_rank() : 0u;
    const int tile = blockIdx.x / split;
    const int64_t n0 = (int64_t)tile * kFp4TileRows;
    const int s_begin = (int)(((int64_t)rank * ks) / split), s_end = (int)(((int64_t)(rank + 1) * ks) / split);
    const int nst = s_end - s_begin;   // stages of this CTA (>= 1 because split <= ks)
    const int kb_row = (int)(K / 32);
    const int k_begin = s_begin * kFp4StageK;
    const int k_len = (int)min((int64_t)nst * kFp4StageK, K - k_begin);   // the tile's last stage may be half full
    const bool half_tail = (k_len & (kFp4StageK - 1)) != 0;

    // carve shared memory (1024-byte aligned for the 128-byte swizzle)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base;
    const uint32_t sSFA = sA + (uint32_t)ring * kFp4StageBytes;
    const uint32_t sB = sSFA + (uint32_t)ring * kFp4SfStageBytes;
    const uint32_t sSFB = sB + (uint32_t)chunk_max * (NB * 128);
    const uint32_t sRecv = sSFB + (uint32_t)chunk_max * kFp4SfStageBytes;   // [split][M][rows of this rank] floats
    const uint32_t sBar = sRecv + (uint32_t)M * kFp4RecvRows * 4u;           // full[ring], empty[ring], done, holder, fail
    uint8_t *gB = gbase + (sB - base), *gSFB = gbase + (sSFB - base);
    const float *gRecv = reinterpret_cast<const float *>(gbase + (sRecv - base));
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(gbase + (sBar - base) + (2 * ring + 1) * 8);
    volatile int &s_fail = *reinterpret_cast<volatile int *>(gbase + (sBar - base) + (2 * ring + 1) * 8 + 4);
    const uint32_t full0 = sBar, empty0 = sBar + (uint32_t)ring * 8u, done_bar = sBar + (uint32_t)ring * 16u;

    // ---- prologue: request the first stages of weights (they do not depend on the previous kernel) --------
    const int pre = nst < ring ? nst : ring;
    if (tid == 32) {   // the TMA thread sets up the barriers and starts the weight stream at once
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");
        s_fail = 0;
        for (int i = 0; i < ring; ++i) {
            mbar_init(full0 + i * 8, kFullArrivals);
            mbar_init(empty0 + i * 8, 1);
        }
        mbar_init(done_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < pre; ++i) {
            mbar_expect_tx(full0 + i * 8, kFp4StageBytes);
            tma_load_codes(sA + (uint32_t)i * kFp4StageBytes, &tmap, (s_begin + i) * (kFp4StageK / 2), (int)n0, full0 + i * 8);
        }
    }
    __syncthreads();
    pdl_trigger();
    const int64_t row_a = n0 + (tid - 64), row_b = row_a + 64;   // rows of the scale threads (tid 64..127)
    const uint8_t *srow_a = scales + row_a * kb_row + (int64_t)s_begin * 8;
    const uint8_t *srow_b = scales + row_b * kb_row + (int64_t)s_begin * 8;
    const bool has_a = row_a < N, has_b = row_b < N;
    const uint32_t sf_a = sSFA + (uint32_t)(((tid - 64) & 31) * 16 + ((tid - 64) >> 5) * 4), sf_b = sf_a + 8;
    auto copy_scales = [&](int i, uint32_t slot) {   // stage i of this CTA into ring slot `slot`
        const bool second = !(half_tail && i == nst - 1);
        const uint32_t dst = slot * kFp4SfStageBytes;
        if (has_a) {
            cp_async4(sf_a + dst, srow_a + i * 8);
            if (second) cp_async4(sf_a + dst + 512, srow_a + i * 8 + 4);
        }
        if (has_b) {
            cp_async4(sf_b + dst, srow_b + i * 8);
            if (second) cp_async4(sf_b + dst + 512, srow_b + i * 8 + 4);
        }
        cp_async_arrive(full0 + slot * 8);
    };
    if (warp >= 2) {
        for (int i = 0; i < pre; ++i) copy_scales(i, (uint32_t)i);
    } else if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         sBar + (uint32_t)(2 * ring + 1) * 8),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // ---- X of this CTA's K range -> 16 digit planes per token + their block scales ---------------------------
    pdl_wait();
    bool inexact = false;
    {
        const int upr = k_len / 8;                 // 8-element units per token row
        const int total = M * upr;
        const __nv_bfloat16 *xbase = X + k_begin;
        for (int u0 = 0; u0 < total; u0 += 2 * kFp4Threads) {
            uint4 raw[2];
            int mm[2], kk[2];
#pragma unroll
            for (int b = 0; b < 2; ++b) {   // both loads of the batch first
                const int u = u0 + b * kFp4Threads + tid;
                const bool act = u < total;
                mm[b] = act ? u / upr : -1;
                kk[b] = act ? (u - mm[b] * upr) * 8 : 0;
                raw[b] = make_uint4(0, 0, 0, 0);
                if (act) raw[b] = *reinterpret_cast<const uint4 *>(xbase + (int64_t)mm[b] * K + kk[b]);
            }
#pragma unroll
            for (int b = 0; b < 2; ++b)
                if (u0 + b * kFp4Threads < total)   // uniform across the CTA
                    inexact |= split_unit<NB>(raw[b], mm[b] >= 0, mm[b], kk[b], lane, gB, gSFB);
        }
    }
    fence_async_proxy();   // B and its scales were written with ordinary stores; the tensor core reads them
    tc_fence_before();
    const int bad = __syncthreads_or(inexact ? 1 : 0);
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;

    float y[kFp4MaxM];
#pragma unroll
    for (int m = 0; m < kFp4MaxM; ++m) y[m] = 0.f;

    if (!bad) {
        if (warp == 0) {
            // ---- MMA warp: the loop is warp-uniform, one elected lane issues ----------------------------------
            // descriptors as 32-bit halves: only the start-address field changes from MMA to MMA
            const uint32_t idesc = (1u << 7) | (1u << 10) | (((uint32_t)NB >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
            const uint32_t a_hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32), b_hi = (uint32_t)(smem_desc(0, 128, 1024, 0) >> 32);
            const uint32_t s_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);
            const uint32_t a_lo0 = (uint32_t)smem_desc(sA, 16, 1024, 2), s_lo0 = (uint32_t)smem_desc(sSFA, 0, 128, 0);
            uint32_t b_lo = (uint32_t)smem_desc(sB, 128, 1024, 0), sb_lo = (uint32_t)smem_desc(sSFB, 0, 128, 0);
            uint32_t slot = 0, phase = 0, accumulate = 0;
            for (int i = 0; i < nst; ++i) {
                if (!mbar_wait(full0 + slot * 8, phase)) {
                    if (lane == 0) {
                        atomicOr(&g_fp4_status, 1u);
                        s_fail = 1;
                    }
                    break;
                }
                tc_fence_after();
                const uint32_t a_lo = a_lo0 + slot * (kFp4StageBytes >> 4);
                const uint32_t sa_lo = s_lo0 + slot * (kFp4SfStageBytes >> 4);
                const int nmma = (half_tail && i == nst - 1) ? 2 : 4;
                const uint32_t t_sf = tmem + NB + (uint32_t)(i & 1) * 16u;   // two slots of 8 + 8 scale columns, alternating
                if (elect_one()) {
                    fence_async_proxy();   // the scale atoms were written by cp.async
                    tc_copy_sf_lohi(t_sf, sa_lo, s_hi);
                    tc_copy_sf_lohi(t_sf + 4, sa_lo + 32, s_hi);
                    tc_copy_sf_lohi(t_sf + 8, sb_lo, s_hi);
                    tc_copy_sf_lohi(t_sf + 12, sb_lo + 32, s_hi);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j < nmma) {
                            const uint32_t sfid = (uint32_t)(j & 1) * 2u;   // scales 2 (j & 1), 2 (j & 1) + 1 of atom j >> 1
                            asm volatile(
                                "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                                "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
                                "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %5, [%7], [%8], p;\n\t}"
                                ::"r"(tmem), "r"(a_lo + j * 2), "r"(a_hi), "r"(b_lo + j * 16), "r"(b_hi),
                                "r"(idesc | (sfid << 4) | (sfid << 29)), "r"(j == 0 ? accumulate : 1u),
                                "r"(t_sf + 4u * (j >> 1)), "r"(t_sf + 8u + 4u * (j >> 1))
                                : "memory");
                        }
                    tc_commit(empty0 + slot * 8);
                }
                __syncwarp();
                accumulate = 1;
                b_lo += (NB * 128) >> 4;
                sb_lo += kFp4SfStageBytes >> 4;
                if (++slot == (uint32_t)ring) {
                    slot = 0;
                    phase ^= 1u;
                }
            }
            if (elect_one()) tc_commit(done_bar);
            __syncwarp();
        } else if (warp == 1) {
            // ---- TMA warp ------------------------------------------------------------------------------------
            uint32_t slot = 0, phase = 0;   // stage `pre` reuses slot 0 (pre == ring whenever the loop runs)
            for (int i = pre; i < nst; ++i) {
                if (!mbar_wait(empty0 + slot * 8, phase)) {
                    if (lane == 0) {
                        atomicOr(&g_fp4_status, 2u);
                        s_fail = 1;
                    }
                    break;
                }
                if (elect_one()) {
                    mbar_expect_tx(full0 + slot * 8, kFp4StageBytes);
                    tma_load_codes(sA + slot * kFp4StageBytes, &tmap, (s_begin + i) * (kFp4StageK / 2), (int)n0, full0 + slot * 8);
                }
                __syncwarp();
                if (++slot == (uint32_t)ring) {
                    slot = 0;
                    phase ^= 1u;
                }
            }
        } else {
            uint32_t slot = 0, phase = 0;
            for (int i = pre; i < nst; ++i) {
                if (!mbar_wait(empty0 + slot * 8, phase)) {
                    atomicOr(&g_fp4_status, 2u);
                    s_fail = 1;
                    break;
                }
                copy_scales(i, slot);
                if (++slot == (uint32_t)ring) {
                    slot = 0;
                    phase ^= 1u;
                }
            }
        }
        // ---- epilogue: accumulator row -> registers; a token's 16 planes are 16 columns, smallest first -----
        if (!mbar_wait(done_bar, 0)) {
            atomicOr(&g_fp4_status, 4u);
            s_fail = 1;
        }
        tc_fence_after();
        const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll
        for (int m = 0; m < NB / kFp4Planes; ++m) {
            float d[16];
            tc_load16(t_row + m * 16, d);
            float acc = d[15];
#pragma unroll
            for (int p = 14; p >= 0; --p) acc += d[p];
            y[m] = acc;
        }
    } else {
        // ---- scalar path for a K range whose X cannot be written as digit planes exactly --------------------
        // first let the copies requested in the prologue land (nothing may be in flight when the CTA ends)
        for (int i = 0; i < pre; ++i)
            if (!mbar_wait(full0 + i * 8, 0)) {
                atomicOr(&g_fp4_status, 8u);
                s_fail = 1;
                break;
            }
        const int64_t n = n0 + tid;
        if (n < N) {
            const uint4 *crow = reinterpret_cast<const uint4 *>(codes + n * (K / 2));
            const uint8_t *srow = scales + n * kb_row;
            for (int blk = k_begin / 32; blk < (k_begin + k_len) / 32; ++blk) {
                const uint4 c = ld_stream_u4(crow + blk);
                const float sc = e8m0_to_float(srow[blk]) * kGuardDown;
                const uint32_t w[4] = {c.x, c.y, c.z, c.w};
                float part[kFp4MaxM];
#pragma unroll
                for (int m = 0; m < kFp4MaxM; ++m) part[m] = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 wv = __half22float2(e2m1x2_to_half2((w[q] >> (8 * i)) & 0xFFu));
                        const int64_t k = (int64_t)blk * 32 + q * 8 + i * 2;
#pragma unroll
                        for (int m = 0; m < kFp4MaxM; ++m)
                            if (m < M) {
                                const uint32_t xb = *reinterpret_cast<const uint32_t *>(X + (int64_t)m * K + k);
                                part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                                part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                            }
                    }
#pragma unroll
                for (int m = 0; m < kFp4MaxM; ++m) y[m] = fmaf(part[m], sc, y[m]);
            }
        }
    }
    // ---- result: direct store, or rank-ordered sum across the cluster --------------------------------------
    __syncthreads();   // s_fail is final
    if (s_fail) {
#pragma unroll
        for (int m = 0; m < kFp4MaxM; ++m) y[m] = __uint_as_float(0x7FC00000u);
    }
    if (split == 1) {
        const int64_t n = n0 + tid;
        if (n < N)
#pragma unroll
            for (int m = 0; m < kFp4MaxM; ++m)
                if (m < M) store_out(Y, y_dtype, (int64_t)m * N + n, y[m] * kGuardUp);
    } else {
        // rank q owns rows [q*128/split, (q+1)*128/split) of the tile: every CTA pushes its partial results
        // for those rows into q's shared memory (slot = sender's rank), one cluster barrier, q adds in rank order
        const int cnt_max = (kFp4TileRows + split - 1) / split;
        const uint32_t owner = (uint32_t)(((tid + 1) * split - 1) / kFp4TileRows);
        const int rr = tid - (int)(owner * kFp4TileRows) / split;
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(sRecv), "r"(owner));
#pragma unroll
        for (int m = 0; m < kFp4MaxM; ++m)
            if (m < M)
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote + (uint32_t)(((int)rank * M + m) * cnt_max + rr) * 4u),
                             "f"(y[m])
                             : "memory");
        cluster_sync_all();
        const int rb = (int)(rank * kFp4TileRows) / split, cnt = (int)((rank + 1) * kFp4TileRows) / split - rb;
        for (int idx = tid; idx < M * cnt; idx += kFp4Threads) {
            const int m = idx / cnt, r = idx - m * cnt;
            float acc = 0.f;
            for (int j = 0; j < split; ++j) acc += gRecv[(j * M + m) * cnt_max + r];
            const int64_t n = n0 + rb + r;
            if (n < N) store_out(Y, y_dtype, (int64_t)m * N + n, acc * kGuardUp);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

int env_int(const char *name) {
    const char *e = std::getenv(name);
    return e ? std::atoi(e) : 0;
}

template <int NB>
cudaError_t launch_fp4(const Fp4Plan &p, const CUtensorMap &map, const void *X, const uint8_t *codes,
                       const uint8_t *scales, void *Y, int y_dtype, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_fp4_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kFp4SmemLimit);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(kFp4Threads);
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
    return cudaLaunchKernelEx(&cfg, linear_fp4_kernel<NB>, map, (const __nv_bfloat16 *)X, p.M, codes, scales, p.N, p.K,
                              Y, y_dtype, p.split, p.ring, p.ks, p.chunk_max, p.tmem_cols);
}

}  // namespace

bool linear_fp4_plan(int M, int64_t N, int64_t K, Fp4Plan &p) {
    if (M < 1 || M > kFp4MaxM || N < 1 || K < 128 || (K % 128) != 0) return false;
    if (K > 0x3FFFFFFF || N > 0x7FFFFFFF) return false;
    p.M = M;
    p.N = N;
    p.K = K;
    p.nb = M == 1 ? 16 : (M == 2 ? 32 : 64);
    p.ks = (int)((K + kFp4StageK - 1) / kFp4StageK);
    p.tiles = (int)((N + kFp4TileRows - 1) / kFp4TileRows);
    return fp4_layout(p, sm_count(), env_int("MXQ_FP4_SPLIT"), env_int("MXQ_FP4_RING"));
}

cudaError_t linear_fp4_launch(const Fp4Plan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                              int y_dtype, cudaStream_t stream) {
    CUtensorMap map;
    if (!codes_tensor_map(codes, p.N, p.K, /*expand_fp4=*/false, &map)) return cudaErrorNotSupported;
    switch (p.nb) {
        case 16: return launch_fp4<16>(p, map, X, codes, scales, Y, y_dtype, stream);
        case 32: return launch_fp4<32>(p, map, X, codes, scales, Y, y_dtype, stream);
        default: return launch_fp4<64>(p, map, X, codes, scales, Y, y_dtype, stream);
    }
}

// returns and clears this kernel's sticky status word (see mxq_linear_device_status)
int linear_fp4_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_fp4_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_fp4_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

}  // namespace mxq
