// mxq_linear on the 5th-generation tensor cores (tcgen05) with the MXFP4 weights as a NATIVE operand.
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
// Work decomposition: one CTA per (128-row tile, K chunk); the `split` CTAs of a tile form a thread-block
// cluster and add their partial results through distributed shared memory in rank order, so the result is
// bit-reproducible and no global workspace or atomics are needed.  Inside a CTA: warp 0 issues the MMAs,
// warp 1 the TMA copies, warps 2-3 the scale copies, over a ring of `ring` stages (128 k each) guarded by
// full/empty mbarriers; all four warps run the X split before and the epilogue after.
//
// Programmatic dependent launch: weights are constants, so the first `ring` stages are requested before
// griddepcontrol.wait; X is read and Y written only after it.
//
// Every mbarrier wait is bounded (about a second); a wait that gives up sets a sticky device word that
// mxq_linear_device_status() returns, the tile is written as NaN, and the kernel still ends cleanly.
#include <cuda.h>   // CUtensorMap and its enums only; the encoder is looked up at run time (no libcuda link)

#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxq_device.cuh"
#include "mxq_host.h"
#include "mxq_linear_umma.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

__device__ unsigned int g_umma_status = 0;   // sticky: bit 0 full-wait, 1 empty-wait, 2 done-wait, 3 drain-wait gave up

namespace {

constexpr uint32_t kFullArrivals = 1 + 64;   // TMA thread's expect_tx arrive + one cp.async arrive per scale thread

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

// ---- the kernel ----------------------------------------------------------------------------------------
// One 8-element unit of X (token m, k offset kk inside the CTA's range): split into parts, store into B and SFB.
// All 32 lanes call it together (the block maximum crosses the four lanes of a 32-block by shuffle).
template <int NB>
__device__ __forceinline__ bool split_unit(const uint4 raw, bool act, int m, int kk, int lane, uint8_t *gB, uint8_t *gSFB) {
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
            *reinterpret_cast<uint2 *>(dst) = make_uint2(part[p][0], part[p][1]);
            if ((lane & 3) == 0)
                gSFB[(size_t)j * kUmmaSfAtomBytes + (row & 31) * 16 + (row >> 5) * 4 + ((kk >> 5) & 3)] = (uint8_t)(sb1 - kGuard - 3 * p);
        }
    }
    return inexact && act;
}

// NB: columns of the B operand / accumulator (16, 32 or 48 >= 3 * M).
template <int NB>
__global__ void __launch_bounds__(kUmmaThreads)
linear_umma_kernel(const __grid_constant__ CUtensorMap tmap, const __nv_bfloat16 *__restrict__ X, int M,
                   const uint8_t *__restrict__ codes, const uint8_t *__restrict__ scales, int64_t N, int64_t K,
                   void *__restrict__ Y, int y_dtype, int split, int ring, int ks, int chunk_max, int tmem_cols) {
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = split > 1 ? cluster_rank() : 0u;
    const int tile = blockIdx.x / split;
    const int64_t n0 = (int64_t)tile * kUmmaTileRows;
    const int s_begin = (int)(((int64_t)rank * ks) / split), s_end = (int)(((int64_t)(rank + 1) * ks) / split);
    const int nst = s_end - s_begin;   // stages of this CTA (>= 1 because split <= ks)
    const int kb_row = (int)(K / 32);

    // carve shared memory (1024-byte aligned for the 128-byte swizzle)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base;
    const uint32_t sSFA = sA + (uint32_t)ring * kUmmaStageSmemBytes;
    const uint32_t sB = sSFA + (uint32_t)ring * kUmmaSfAtomBytes;
    const uint32_t sSFB = sB + (uint32_t)chunk_max * (NB * 128);
    const uint32_t sRecv = sSFB + (uint32_t)chunk_max * kUmmaSfAtomBytes;   // [split][M][rows of this rank] floats
    const uint32_t sBar = sRecv + (uint32_t)M * kUmmaRecvRows * 4u;    // full[ring], empty[ring], done, holder, fail
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
            mbar_expect_tx(full0 + i * 8, kUmmaStageTxBytes);
            tma_load_codes(sA + (uint32_t)i * kUmmaStageSmemBytes, &tmap, (s_begin + i) * kUmmaStageK, (int)n0, full0 + i * 8);
        }
    }
    __syncthreads();
    pdl_trigger();
    const int64_t row_a = n0 + (tid - 64), row_b = row_a + 64;   // rows of the scale threads (tid 64..127)
    const uint8_t *srow_a = scales + row_a * kb_row + (int64_t)s_begin * 4;
    const uint8_t *srow_b = scales + row_b * kb_row + (int64_t)s_begin * 4;
    const bool has_a = row_a < N, has_b = row_b < N;
    const uint32_t sf_a = sSFA + (uint32_t)(((tid - 64) & 31) * 16 + ((tid - 64) >> 5) * 4), sf_b = sf_a + 8;
    if (warp >= 2) {
        for (int i = 0; i < pre; ++i) {
            if (has_a) cp_async4(sf_a + (uint32_t)i * kUmmaSfAtomBytes, srow_a + i * 4);
            if (has_b) cp_async4(sf_b + (uint32_t)i * kUmmaSfAtomBytes, srow_b + i * 4);
            cp_async_arrive(full0 + i * 8);
        }
    } else if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         sBar + (uint32_t)(2 * ring + 1) * 8),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // ---- X of this CTA's K range -> three E5M2 parts + block scales (after the previous kernel finished) ---
    pdl_wait();
    bool inexact = false;
    {
        const int upr = nst * (kUmmaStageK / 8);        // 8-element units per token row
        const int total = M * upr;
        const __nv_bfloat16 *xbase = X + (int64_t)s_begin * kUmmaStageK;
        for (int u0 = 0; u0 < total; u0 += 4 * kUmmaThreads) {
            uint4 raw[4];
            int mm[4], kk[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) {   // all loads of the batch first
                const int u = u0 + b * kUmmaThreads + tid;
                const bool act = u < total;
                mm[b] = act ? u / upr : -1;
                kk[b] = act ? (u - mm[b] * upr) * 8 : 0;
                raw[b] = make_uint4(0, 0, 0, 0);
                if (act) raw[b] = *reinterpret_cast<const uint4 *>(xbase + (int64_t)mm[b] * K + kk[b]);
            }
#pragma unroll
            for (int b = 0; b < 4; ++b)
                if (u0 + b * kUmmaThreads < total)   // uniform across the CTA
                    inexact |= split_unit<NB>(raw[b], mm[b] >= 0, mm[b], kk[b], lane, gB, gSFB);
        }
    }
    fence_async_proxy();   // B and its scales were written with ordinary stores; the tensor core reads them
    tc_fence_before();
    const int bad = __syncthreads_or(inexact ? 1 : 0);
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;

    float y[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) y[m] = 0.f;

    if (!bad) {
        if (warp == 0) {
            // ---- MMA warp: the loop is warp-uniform, one elected lane issues ----------------------------------
            // descriptors as 32-bit halves: only the start-address field changes from MMA to MMA
            const uint32_t idesc = (5u << 7) | (1u << 10) | (((uint32_t)NB >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
            const uint32_t a_hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32), b_hi = (uint32_t)(smem_desc(0, 128, 1024, 0) >> 32);
            const uint32_t s_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);
            const uint32_t a_lo0 = (uint32_t)smem_desc(sA, 16, 1024, 2), s_lo0 = (uint32_t)smem_desc(sSFA, 0, 128, 0);
            uint32_t b_lo = (uint32_t)smem_desc(sB, 128, 1024, 0), sb_lo = (uint32_t)smem_desc(sSFB, 0, 128, 0);
            const uint32_t t_sfa0 = tmem + NB, t_sfb0 = t_sfa0 + 4u * (uint32_t)ring;
            uint32_t slot = 0, phase = 0, accumulate = 0;
            for (int i = 0; i < nst; ++i) {
                if (!mbar_wait(full0 + slot * 8, phase)) {
                    if (lane == 0) {
                        atomicOr(&g_umma_status, 1u);
                        s_fail = 1;
                    }
                    break;
                }
                tc_fence_after();
                const uint32_t t_sfa = t_sfa0 + 4u * slot, t_sfb = t_sfb0 + 4u * slot;
                const uint32_t a_lo = a_lo0 + slot * (kUmmaStageSmemBytes >> 4);
                if (elect_one()) {
                    fence_async_proxy();   // the scale atom was written by cp.async
                    asm volatile(
                        "{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\ttcgen05.cp.cta_group::1.32x128b.warpx4 [%0], d;\n\t}"
                        ::"r"(t_sfa), "r"(s_lo0 + slot * (kUmmaSfAtomBytes >> 4)), "r"(s_hi) : "memory");
                    asm volatile(
                        "{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\ttcgen05.cp.cta_group::1.32x128b.warpx4 [%0], d;\n\t}"
                        ::"r"(t_sfb), "r"(sb_lo), "r"(s_hi) : "memory");
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb)
                        asm volatile(
                            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                            "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
                            "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], da, db, %5, [%7], [%8], p;\n\t}"
                            ::"r"(tmem), "r"(a_lo + kb * 2), "r"(a_hi), "r"(b_lo + kb * 16), "r"(b_hi),
                            "r"(idesc | ((uint32_t)kb << 4) | ((uint32_t)kb << 29)), "r"(kb == 0 ? accumulate : 1u), "r"(t_sfa),
                            "r"(t_sfb)
                            : "memory");
                    tc_commit(empty0 + slot * 8);
                }
                __syncwarp();
                accumulate = 1;
                b_lo += (NB * 128) >> 4;
                sb_lo += kUmmaSfAtomBytes >> 4;
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
                        atomicOr(&g_umma_status, 2u);
                        s_fail = 1;
                    }
                    break;
                }
                if (elect_one()) {
                    mbar_expect_tx(full0 + slot * 8, kUmmaStageTxBytes);
                    tma_load_codes(sA + slot * kUmmaStageSmemBytes, &tmap, (s_begin + i) * kUmmaStageK, (int)n0, full0 + slot * 8);
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
                    atomicOr(&g_umma_status, 2u);
                    s_fail = 1;
                    break;
                }
                if (has_a) cp_async4(sf_a + slot * kUmmaSfAtomBytes, srow_a + i * 4);
                if (has_b) cp_async4(sf_b + slot * kUmmaSfAtomBytes, srow_b + i * 4);
                cp_async_arrive(full0 + slot * 8);
                if (++slot == (uint32_t)ring) {
                    slot = 0;
                    phase ^= 1u;
                }
            }
        }
        // ---- epilogue: accumulator row -> registers; the three parts of a token are three columns ----------
        if (!mbar_wait(done_bar, 0)) {
            atomicOr(&g_umma_status, 4u);
            s_fail = 1;
        }
        tc_fence_after();
        const uint32_t t_row = tmem + ((uint32_t)(warp * 32) << 16);
#pragma unroll
        for (int c = 0; c < NB / 16; ++c) {
            float d[16];
            tc_load16(t_row + c * 16, d);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int col = c * 16 + j;
                if (col < 48) y[col / 3] += d[j];   // fixed order: parts 0, 1, 2 of token col / 3
            }
        }
    } else {
        // ---- scalar path for a K range whose X cannot be split exactly ------------------------------------
        // first let the copies requested in the prologue land (nothing may be in flight when the CTA ends)
        for (int i = 0; i < pre; ++i)
            if (!mbar_wait(full0 + i * 8, 0)) {
                atomicOr(&g_umma_status, 8u);
                s_fail = 1;
                break;
            }
        const int64_t n = n0 + tid;
        if (n < N) {
            const uint4 *crow = reinterpret_cast<const uint4 *>(codes + n * (K / 2));
            const uint8_t *srow = scales + n * kb_row;
            for (int blk = s_begin * 4; blk < s_end * 4; ++blk) {
                const uint4 c = ld_stream_u4(crow + blk);
                const float sc = e8m0_to_float(srow[blk]) * kGuardDown;
                const uint32_t w[4] = {c.x, c.y, c.z, c.w};
                float part[16];
#pragma unroll
                for (int m = 0; m < 16; ++m) part[m] = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 wv = __half22float2(e2m1x2_to_half2((w[q] >> (8 * i)) & 0xFFu));
                        const int64_t k = (int64_t)blk * 32 + q * 8 + i * 2;
#pragma unroll
                        for (int m = 0; m < 16; ++m)
                            if (m < M) {
                                const uint32_t xb = *reinterpret_cast<const uint32_t *>(X + (int64_t)m * K + k);
                                part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                                part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                            }
                    }
#pragma unroll
                for (int m = 0; m < 16; ++m) y[m] = fmaf(part[m], sc, y[m]);
            }
        }
    }

    // ---- result: direct store, or rank-ordered sum across the cluster --------------------------------------
    __syncthreads();   // s_fail is final
    if (s_fail) {
#pragma unroll
        for (int m = 0; m < 16; ++m) y[m] = __uint_as_float(0x7FC00000u);
    }
    if (split == 1) {
        const int64_t n = n0 + tid;
        if (n < N)
#pragma unroll
            for (int m = 0; m < 16; ++m)
                if (m < M) store_out(Y, y_dtype, (int64_t)m * N + n, y[m] * kGuardUp);
    } else {
        // rank q owns rows [q*128/split, (q+1)*128/split) of the tile: every CTA pushes its partial results
        // for those rows into q's shared memory (slot = sender's rank), one cluster barrier, q adds in rank order
        const int cnt_max = (kUmmaTileRows + split - 1) / split;
        const uint32_t owner = (uint32_t)(((tid + 1) * split - 1) / kUmmaTileRows);
        const int rr = tid - (int)(owner * kUmmaTileRows) / split;
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(sRecv), "r"(owner));
#pragma unroll
        for (int m = 0; m < 16; ++m)
            if (m < M)
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote + (uint32_t)(((int)rank * M + m) * cnt_max + rr) * 4u),
                             "f"(y[m])
                             : "memory");
        cluster_sync_all();
        const int rb = (int)(rank * kUmmaTileRows) / split, cnt = (int)((rank + 1) * kUmmaTileRows) / split - rb;
        for (int idx = tid; idx < M * cnt; idx += kUmmaThreads) {
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

// ---- host side -----------------------------------------------------------------------------------------
int env_int(const char *name) {
    const char *e = std::getenv(name);
    return e ? std::atoi(e) : 0;
}

template <int NB>
cudaError_t launch_umma(const UmmaPlan &p, const CUtensorMap &map, const void *X, const uint8_t *codes,
                        const uint8_t *scales, void *Y, int y_dtype, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_umma_kernel<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kUmmaSmemLimit);
        if (e != cudaSuccess) return e;
        // all of the SM's L1/shared array as shared memory: how many CTAs (of this and of the next kernel) fit on an
        // SM is what decides how early the next kernel's weight stream can start
        e = cudaFuncSetAttribute(linear_umma_kernel<NB>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
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
    return cudaLaunchKernelEx(&cfg, linear_umma_kernel<NB>, map, (const __nv_bfloat16 *)X, p.M, codes, scales, p.N, p.K,
                              Y, y_dtype, p.split, p.ring, p.ks, p.chunk_max, p.tmem_cols);
}

}  // namespace

bool linear_umma_plan(int M, int64_t N, int64_t K, UmmaPlan &p) {
    if (M < 1 || M > 16 || N < 1 || K < kUmmaStageK || (K % kUmmaStageK) != 0) return false;
    if (K / kUmmaStageK > 32767 || (N + kUmmaTileRows - 1) / kUmmaTileRows > (1 << 20)) return false;
    if (N > 0x7FFFFFFF || K > 0x7FFFFFFF) return false;
    p.M = M;
    p.N = N;
    p.K = K;
    p.nb = 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : 48);
    p.ks = (int)(K / kUmmaStageK);
    p.tiles = (int)((N + kUmmaTileRows - 1) / kUmmaTileRows);
    return umma_layout(p, sm_count(), env_int("MXQ_UMMA_SPLIT"), env_int("MXQ_UMMA_RING"));
}

cudaError_t linear_umma_launch(const UmmaPlan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                               int y_dtype, cudaStream_t stream) {
    CUtensorMap map;
    if (!codes_tensor_map(codes, p.N, p.K, /*expand_fp4=*/true, &map)) return cudaErrorNotSupported;
    switch (p.nb) {
        case 16: return launch_umma<16>(p, map, X, codes, scales, Y, y_dtype, stream);
        case 32: return launch_umma<32>(p, map, X, codes, scales, Y, y_dtype, stream);
        default: return launch_umma<48>(p, map, X, codes, scales, Y, y_dtype, stream);
    }
}

bool linear_umma_available() { return tensor_map_available(); }

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)
int mxq_linear_device_status(uint32_t *status_host) {
    if (!status_host) return MXQ_ERR_NULL;
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, mxq::g_umma_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(mxq::g_umma_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    uint32_t v4 = 0;
    const int rc = mxq::linear_fp4_take_status(&v4);
    if (rc != MXQ_OK) return rc;
    *status_host = v | (v4 << 8);
    return MXQ_OK;
}
#pragma GCC visibility pop
}
