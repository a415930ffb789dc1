// Tensor-core mxq_linear for sm_100a: Y[M,N] = X[M,K] . dequant(codes, scales)^T, M <= 16
// (the MXFP4 GEMM of Sec. III-D-3 with the late scaling of Eq. 2).
//
// Why tensor cores for a mat-vec: the weight stream delivers ~42 weights per clock per SM at
// HBM speed, and every way of turning a 4-bit code into an FP32 operand on the CUDA cores
// costs 2.5+ issue slots per weight (measured: conversion and logic pipes run at 64 lanes/clk).
// cvt.rn.f16x2.e2m1x2 decodes two weights per instruction, exactly, and mma.sync takes the
// FP16 pairs as they come; the multiply-accumulate then costs almost nothing for any M <= 8.
//
// Exactness: every E2M1 value is an FP16 number.  X is BF16; each CTA rescales its slice of X
// by one power of two so that the largest magnitude sits just below 2^15 and converts it to
// FP16, checking that every element converts exactly (true whenever an element is within 2^32
// of the largest).  Products FP16 x FP16 are exact in the FP32 accumulator.  If any element
// does not convert exactly the CTA takes a scalar FP32 path instead, so the result never
// depends on the shortcut.
//
// Decomposition: CTA c owns the weight rows [c*N/G, (c+1)*N/G) for the whole of K, so every
// CTA streams the same number of bytes to within one row, no output is shared between CTAs,
// and there is no workspace.  The rows are processed as 16-row tiles (the last one ragged:
// missing rows are neither fetched nor stored).  Within a CTA the 8 warps split each stage's
// 64 MX blocks; every warp leaves its FP32 partial tile in shared memory and the warp that
// arrives last (a counter, not a barrier) sums the 8 in warp order, so results are
// bit-reproducible.  When M*K is too large for X to fit in shared memory, K is cut into
// windows; the CTA walks its tiles once per window and keeps per-tile sums in shared memory.
//
// Pipeline: every warp runs its own ring of 16-byte cp.async copies for exactly the bytes it
// will consume (16 rows x 128 code bytes + 16 x 8 scale bytes per stage), so the main loop has
// no CTA-wide barrier and no spin-wait.  Weights never depend on the previous kernel, so the
// ring is filled before griddepcontrol.wait (programmatic dependent launch); X and Y are
// touched only after it.  A CTA is small enough that two kernels, two CTAs per SM each, can be
// resident: the next kernel prefetches while this one computes.
#include <cstdlib>

#include "mxq_device.cuh"
#include "mxq_host.h"
#include "mxq_linear_plan.h"

namespace mxq {

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ unsigned int g_mma_status = 0;   // sticky: bit 0 the wait for a reduction slot gave up

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// low byte of v (two E2M1 codes) -> FP16 pair, low nibble in the low half; the upper bits of v are ignored
__device__ __forceinline__ uint32_t e2m1x2_lowbyte_to_half2(uint32_t v) {
    uint32_t out;
    asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(out) : "r"(v));
    return out;
}
// four code bytes -> four FP16 pairs: one shift per byte beyond the first, one conversion per byte
__device__ __forceinline__ void e2m1x8_to_half2x4(uint32_t word, uint32_t &p0, uint32_t &p1, uint32_t &p2, uint32_t &p3) {
    p0 = e2m1x2_lowbyte_to_half2(word);
    p1 = e2m1x2_lowbyte_to_half2(word >> 8);
    p2 = e2m1x2_lowbyte_to_half2(word >> 16);
    p3 = e2m1x2_lowbyte_to_half2(word >> 24);
}
// two E8M0 bytes (low 16 bits of v) -> BF16 pair; 0 -> 2^-127 (a BF16 subnormal), 0xFF -> NaN
__device__ __forceinline__ uint32_t e8m0x2_to_bf16x2(uint32_t v) {
    uint32_t out;
    asm("{\n\t.reg .b16 h;\n\tcvt.u16.u32 h, %1;\n\tcvt.rn.bf16x2.ue8m0x2 %0, h;\n\t}" : "=r"(out) : "r"(v));
    return out;
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1, const float (&c)[4]) {
    asm(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// ---------------------------------------------------------------------------------------------
// stage table entry (uint4), built once per CTA from stage_lookup():
//   x  byte offset into codes of (first row of the tile, first block of the stage)
//   y  byte offset into scales of the same position
//   z  b (16 bits: first block within the window) | nblk << 16 | flags << 24 | (rows in tile - 1) << 28
//   w  tile (local to the CTA) | window << 20
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kFlagSegLast = 1, kFlagWinFirst = 2;

// (`count`: elements of Y, for the bounds-checked build)
__device__ __forceinline__ void store_out(void *Y, int y_dtype, int64_t idx, float v, int64_t count) {
    (void)count;
    if (y_dtype == MXQ_F32)
        *MXQ_AT(reinterpret_cast<float *>(Y) + idx, 4, Y, count * 4) = v;
    else
        *MXQ_AT(reinterpret_cast<__nv_bfloat16 *>(Y) + idx, 2, Y, count * 2) = __float2bfloat16_rn(v);
}

__device__ __forceinline__ uint32_t max_abs_bits(const uint4 &v) {  // largest BF16 magnitude pattern of 8 values
    return max(max(max(v.x & 0x7FFFu, (v.x >> 16) & 0x7FFFu), max(v.y & 0x7FFFu, (v.y >> 16) & 0x7FFFu)),
               max(max(v.z & 0x7FFFu, (v.z >> 16) & 0x7FFFu), max(v.w & 0x7FFFu, (v.w >> 16) & 0x7FFFu)));
}

// 8 BF16 -> 8 FP16 after scaling by `up`; returns non-zero if any conversion was inexact
__device__ __forceinline__ int bf16x8_to_f16x8(const uint4 &v, float up, uint4 &out) {
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
    int inexact = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float lo = __uint_as_float(in[j] << 16) * up;
        const float hi = __uint_as_float(in[j] & 0xFFFF0000u) * up;
        const __half2 h = __floats2half2_rn(lo, hi);
        const float2 back = __half22float2(h);
        inexact |= (back.x != lo) | (back.y != hi);
        o[j] = *reinterpret_cast<const uint32_t *>(&h);
    }
    out = make_uint4(o[0], o[1], o[2], o[3]);
    return inexact;
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
// NT8: 8-token column tiles (1 for M <= 8, 2 for M <= 16); NS: ring depth
template <int NT8, int NS>
__global__ void __launch_bounds__(kMmaThreads, 2)
linear_mma_kernel(const __grid_constant__ LinearPlan p, const uint16_t *__restrict__ X,
                  const uint8_t *__restrict__ codes, const uint8_t *__restrict__ scales, void *__restrict__ Y,
                  int y_dtype) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t sbase = smem_u32(smem);
    int *s_max = reinterpret_cast<int *>(smem + kOffMisc);            // [0]: largest |x| pattern of the window
    int *s_inexact = reinterpret_cast<int *>(smem + kOffMisc + 16);   // [0]
    int *s_cnt = reinterpret_cast<int *>(smem + kOffMisc + 32);       // [kRedSlots] warps arrived
    int *s_gen = reinterpret_cast<int *>(smem + kOffMisc + 64);       // [kRedSlots] tiles summed per slot
    const uint4 *s_table = reinterpret_cast<const uint4 *>(smem + kOffTable);
    float *s_red = reinterpret_cast<float *>(smem + kOffRed);         // [kRedSlots][warps][NT8*8][16]
    float *s_acc = reinterpret_cast<float *>(smem + p.off_acc);       // [tiles][NT8*8][16], only if nwin > 1
    constexpr int kOut = NT8 * 8 * kTileRows;                         // values of one tile
    constexpr int kPerLane = kOut / 32;

    pdl_trigger();  // let the next kernel in the stream start prefetching its weights

    // ---- this CTA's rows and its stage table (one thread per stage, closed form) ---------------------
    const int64_t r0 = row_begin(p, blockIdx.x), r1 = row_begin(p, blockIdx.x + 1);
    const int tiles = (int)((r1 - r0 + kTileRows - 1) / kTileRows);
    StageInfo si;
    const int nstages = stage_lookup(p, tiles, -1, si);
    for (int q = tid; q < nstages; q += kMmaThreads) {
        stage_lookup(p, tiles, q, si);
        const uint32_t j = (uint32_t)si.w * (uint32_t)p.bw + (uint32_t)si.b;   // block index within the row
        const int64_t row = r0 + (int64_t)si.tile * kTileRows;
        const int64_t rows_left = r1 - row;
        const uint32_t rows_m1 = (uint32_t)(rows_left < kTileRows ? rows_left : kTileRows) - 1u;
        uint4 e;
        e.x = (uint32_t)(row * (p.K / 2)) + j * 16u;
        e.y = (uint32_t)(row * p.kb) + j;
        e.z = (uint32_t)si.b | ((uint32_t)si.nblk << 16) |
              ((si.seg_last ? kFlagSegLast : 0u) | (si.win_first ? kFlagWinFirst : 0u)) << 24 | rows_m1 << 28;
        e.w = (uint32_t)si.tile | ((uint32_t)si.w << 20);
        reinterpret_cast<uint4 *>(smem + kOffTable)[q] = e;
    }
    if (tid < kRedSlots) s_cnt[tid] = s_gen[tid] = 0;
    if (tid == 0) s_inexact[0] = 0;
    __syncthreads();

    // ---- per-lane constants ---------------------------------------------------------------------------
    const int blk0 = warp * kWarpBlocks;  // this warp's blocks within a stage
    const uint32_t ring = sbase + p.off_ring + (uint32_t)warp * (uint32_t)(NS * kWarpStageBytes);
    // Copy role of this lane.  Four consecutive lanes fetch 64 contiguous bytes of one row (lanes that split a
    // 32-byte sector between two quarter-warps halve the L2 -> SM rate: measured 4.1 vs 6.4 TB/s), so a
    // quarter-warp covers rows r and r + 4.  In shared memory row r keeps its 8 chunks at (chunk ^ (r & 7)),
    // which makes both these writes and the fragment reads (8 rows, one chunk) bank-conflict free.
    // lane -> rows cr and cr + 8 of the tile, chunks cc and cc + 4; lanes 0..15 also copy row `lane`'s 8 scale bytes
    const uint32_t cc = lane & 3, cr = ((lane >> 2) & 1) * 4 + (lane >> 3);
    const uint32_t row_bytes = (uint32_t)(p.K / 2);
    const uint32_t dst_a = cr * 128 + ((cc ^ cr) << 4), dst_b = cr * 128 + (((cc + 4) ^ cr) << 4);
    const uint32_t dst_sc = kWarpCodeBytes + (lane & 15) * 8 + (lane >> 4) * 4;
    const uint8_t *src_lo = codes + (blk0 + cc) * 16 + (size_t)cr * row_bytes;
    const uint8_t *src_hi = src_lo + (size_t)8 * row_bytes;
    const uint8_t *src_sc = scales + blk0 + (lane >> 4) * 4 + (size_t)(lane & 15) * (uint32_t)p.kb;
    const bool sc8 = (p.kb % 8) == 0;   // scale rows 8-byte aligned: one 8-byte copy per row instead of two 4-byte ones

    auto issue = [&](int q, int slot) {
        const uint4 e = s_table[q];
        const int left = (int)((e.z >> 16) & 0xFF) - blk0;   // blocks of this stage from this warp's first one on
        const uint32_t rows_m1 = e.z >> 28;
        if (left > 0) {
            const uint32_t dst = ring + (uint32_t)slot * kWarpStageBytes;
            const bool lo_ok = cr <= rows_m1, hi_ok = cr + 8 <= rows_m1, sc_ok = (uint32_t)(lane & 15) <= rows_m1;
            if (lo_ok) cp_async16(dst + dst_a, MXQ_AT(src_lo + e.x, 16, codes, (int64_t)p.N * (p.K / 2)));
            if (hi_ok) cp_async16(dst + dst_a + 1024, MXQ_AT(src_hi + e.x, 16, codes, (int64_t)p.N * (p.K / 2)));
            if (left > 4) {
                if (lo_ok) cp_async16(dst + dst_b, MXQ_AT(src_lo + e.x + 64, 16, codes, (int64_t)p.N * (p.K / 2)));
                if (hi_ok) cp_async16(dst + dst_b + 1024, MXQ_AT(src_hi + e.x + 64, 16, codes, (int64_t)p.N * (p.K / 2)));
                if (sc8) {
                    if (lane < 16 && sc_ok) cp_async8(dst + dst_sc, MXQ_AT(src_sc + e.y, 8, scales, (int64_t)p.N * p.kb));
                } else if (sc_ok) {
                    cp_async4(dst + dst_sc, MXQ_AT(src_sc + e.y, 4, scales, (int64_t)p.N * p.kb));
                }
            } else if (lane < 16 && sc_ok) {
                cp_async4(dst + dst_sc, MXQ_AT(src_sc + e.y, 4, scales, (int64_t)p.N * p.kb));
            }
        }
    };

#pragma unroll
    for (int s = 0; s < NS; ++s) {
        if (s < nstages) issue(s, s);
        cp_async_commit();
    }

    pdl_wait();  // from here on X and Y may be touched

    float acc[NT8][4];
#pragma unroll
    for (int n = 0; n < NT8; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[n][i] = 0.f;

    // per-thread constants of the fragment reads
    // row g's chunk jb sits at g*128 + ((jb ^ g) << 4): with the slot 128-byte aligned that is
    // (slot + a_off) ^ (jb << 4); row g + 8 is 1024 bytes further
    const uint32_t a_off = (uint32_t)(g * 128 + (g << 4) + 4 * t);
    // B fragment: token g (and g + 8).  Lanes whose token does not exist read the last real token instead:
    // a column of B only ever feeds the same column of the result, and those columns are never stored.
    const uint32_t x_thread0 = sbase + p.off_x + (uint32_t)blk0 * 64u + 16u * t + (uint32_t)min(g, p.M - 1) * p.x_stride;
    const uint32_t x_thread1 = sbase + p.off_x + (uint32_t)blk0 * 64u + 16u * t + (uint32_t)min(g + 8, p.M - 1) * p.x_stride;

    int seg_index = 0, slot = 0;
    bool exact_ok = true;
    float un = 1.f;
#pragma unroll 1
    for (int q = 0; q < nstages; ++q) {
        const uint4 e = s_table[q];
        const int b_now = e.z & 0xFFFF, nblk_now = (e.z >> 16) & 0xFF;
        const uint32_t flags = (e.z >> 24) & 0xF;

        // ---- (re)stage this window's slice of X as scaled FP16 (the only CTA-wide barriers) ----------
        if (flags & kFlagWinFirst) {
            const int w_now = e.w >> 20;
            const int bwid = (w_now == p.nwin - 1) ? p.bw_last : p.bw;
            const int64_t k0 = (int64_t)w_now * p.bw * kBlock;
            const int vec_per_row = bwid * kBlock / 8;   // 16-byte vectors per token row
            const int nvec = vec_per_row * p.M;
            __syncthreads();                              // everyone is done with the previous window
            if (tid == 0) {
                s_max[0] = 0;
                s_inexact[0] = 0;
            }
            __syncthreads();
            // one trip to L2: the first four vectors of every thread stay in registers for the second pass
            constexpr int kKeep = 4;
            uint4 keep[kKeep];
            uint32_t mx = 0;
#pragma unroll
            for (int i = 0; i < kKeep; ++i) {
                const int v = tid + i * kMmaThreads;
                keep[i] = make_uint4(0, 0, 0, 0);
                if (v < nvec) {
                    const int m = v / vec_per_row, c = v - m * vec_per_row;
                    keep[i] = __ldcg(MXQ_AT(reinterpret_cast<const uint4 *>(X + (int64_t)m * p.K + k0) + c, 16, X, (int64_t)p.M * p.K * 2));
                }
                mx = max(mx, max_abs_bits(keep[i]));
            }
            for (int v = tid + kKeep * kMmaThreads; v < nvec; v += kMmaThreads) {
                const int m = v / vec_per_row, c = v - m * vec_per_row;
                mx = max(mx, max_abs_bits(__ldcg(MXQ_AT(reinterpret_cast<const uint4 *>(X + (int64_t)m * p.K + k0) + c, 16, X, (int64_t)p.M * p.K * 2))));
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (lane == 0 && mx) atomicMax(&s_max[0], (int)mx);
            __syncthreads();
            // one power-of-two scale for the whole slice: the largest magnitude lands in [2^14, 2^15)
            int sh = 141 - min(s_max[0] >> 7, 254);
            sh = sh > 126 ? 126 : sh;
            const float up = __uint_as_float((uint32_t)(sh + 127) << 23);
            un = __uint_as_float((uint32_t)(127 - sh) << 23);
            int inexact = 0;
#pragma unroll
            for (int i = 0; i < kKeep; ++i) {
                const int v = tid + i * kMmaThreads;
                if (v < nvec) {
                    const int m = v / vec_per_row, c = v - m * vec_per_row;
                    uint4 out;
                    inexact |= bf16x8_to_f16x8(keep[i], up, out);
                    *reinterpret_cast<uint4 *>(smem + p.off_x + (size_t)m * p.x_stride + (size_t)c * 16) = out;
                }
            }
            for (int v = tid + kKeep * kMmaThreads; v < nvec; v += kMmaThreads) {
                const int m = v / vec_per_row, c = v - m * vec_per_row;
                uint4 out;
                inexact |= bf16x8_to_f16x8(__ldcg(MXQ_AT(reinterpret_cast<const uint4 *>(X + (int64_t)m * p.K + k0) + c, 16, X, (int64_t)p.M * p.K * 2)), up, out);
                *reinterpret_cast<uint4 *>(smem + p.off_x + (size_t)m * p.x_stride + (size_t)c * 16) = out;
            }
            if (inexact) atomicOr(&s_inexact[0], 1);
            __syncthreads();
            exact_ok = s_inexact[0] == 0;
        }

        // ---- consume this warp's slice of the stage ------------------------------------------------
        cp_async_wait<NS - 1>();  // all but the newest NS-1 groups have landed: this stage is in
        __syncwarp();
        const int left = nblk_now - blk0;  // blocks of this stage that are this warp's: 8, 4 or none
        if (exact_ok && left > 0) {
            const uint32_t cbase = ring + (uint32_t)slot * kWarpStageBytes;
            const uint32_t abase = cbase + a_off;
            const uint32_t xbase0 = x_thread0 + (uint32_t)b_now * 64u, xbase1 = x_thread1 + (uint32_t)b_now * 64u;
            const uint2 sw_lo = lds64(cbase + kWarpCodeBytes + g * 8), sw_hi = lds64(cbase + kWarpCodeBytes + g * 8 + 64);
            auto four_blocks = [&](uint32_t s_lo, uint32_t s_hi, int jb0) {
                // all shared-memory reads of the four blocks first, so that their latencies overlap
                uint32_t a_lo[4], a_hi[4];
                uint4 xb[4][NT8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // A: this lane's 8 weights of rows g and g+8 of block jb (k = 8t .. 8t+7 of the block)
                    a_lo[i] = lds32(abase ^ (uint32_t)((jb0 + i) << 4));
                    a_hi[i] = lds32((abase ^ (uint32_t)((jb0 + i) << 4)) + 1024);
                    // B: the same 8 k of token g (+8 for the second column tile)
#pragma unroll
                    for (int n = 0; n < NT8; ++n) xb[i][n] = lds128((n == 0 ? xbase0 : xbase1) + (jb0 + i) * 64);
                }
                // the four blocks' scales of rows g and g+8; 2^-shift of X is folded in here
                const uint32_t sl01 = e8m0x2_to_bf16x2(s_lo), sl23 = e8m0x2_to_bf16x2(s_lo >> 16);
                const uint32_t sh01 = e8m0x2_to_bf16x2(s_hi), sh23 = e8m0x2_to_bf16x2(s_hi >> 16);
                const float sc_lo[4] = {__uint_as_float(sl01 << 16) * un, __uint_as_float(sl01 & 0xFFFF0000u) * un,
                                        __uint_as_float(sl23 << 16) * un, __uint_as_float(sl23 & 0xFFFF0000u) * un};
                const float sc_hi[4] = {__uint_as_float(sh01 << 16) * un, __uint_as_float(sh01 & 0xFFFF0000u) * un,
                                        __uint_as_float(sh23 << 16) * un, __uint_as_float(sh23 & 0xFFFF0000u) * un};
                const float zero[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t l[4][4], h[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    e2m1x8_to_half2x4(a_lo[i], l[i][0], l[i][1], l[i][2], l[i][3]);
                    e2m1x8_to_half2x4(a_hi[i], h[i][0], h[i][1], h[i][2], h[i][3]);
                }
#pragma unroll
                for (int n = 0; n < NT8; ++n) {
                    float part[4][4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_f16(part[i], l[i][0], h[i][0], l[i][1], h[i][1], xb[i][n].x, xb[i][n].y, zero);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_f16(part[i], l[i][2], h[i][2], l[i][3], h[i][3], xb[i][n].z, xb[i][n].w, part[i]);
                    // late scaling (Eq. 2): one multiply per 32-long partial sum
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        acc[n][0] = fmaf(part[i][0], sc_lo[i], acc[n][0]);
                        acc[n][1] = fmaf(part[i][1], sc_lo[i], acc[n][1]);
                        acc[n][2] = fmaf(part[i][2], sc_hi[i], acc[n][2]);
                        acc[n][3] = fmaf(part[i][3], sc_hi[i], acc[n][3]);
                    }
                }
            };
            four_blocks(sw_lo.x, sw_hi.x, 0);
            if (left > 4) four_blocks(sw_lo.y, sw_hi.y, 4);
        }
        __syncwarp();  // every lane is done reading the slot
        if (q + NS < nstages) issue(q + NS, slot);
        cp_async_commit();
        slot = (slot + 1 == NS) ? 0 : slot + 1;

        if (!(flags & kFlagSegLast)) continue;

        // ---- end of a (window, tile) pair -----------------------------------------------------------------
        // Each warp leaves its partial tile in red[rslot][warp]; the last warp to arrive sums them in warp
        // order and finishes the pair.  No CTA-wide barrier: the other warps move on to the next tile.
        const int tile_now = e.w & 0xFFFFF, w_now = e.w >> 20;
        const int rslot = seg_index % kRedSlots;
        float poison = 0.f;
        {   // the slot's previous pair (kRedSlots pairs ago) must have been summed.  The wait is bounded; if it
            // gives up, a sticky status bit is set (mxq_linear_device_status, bit 28) and this warp's share of the
            // tile goes out as NaN, so that the tile cannot pass for a result
            const int need = seg_index / kRedSlots;
            int spins = 0;
            while (*reinterpret_cast<volatile int *>(&s_gen[rslot]) < need && ++spins < (1 << 22)) __nanosleep(40);
            if (spins >= (1 << 22)) {
                poison = __uint_as_float(0x7FC00000u);
                if (lane == 0) atomicOr(&g_mma_status, 1u);
            }
        }
        float *mine = s_red + (rslot * kMmaWarps + warp) * kOut;
        if (exact_ok) {
#pragma unroll
            for (int n = 0; n < NT8; ++n) {
                mine[(8 * n + 2 * t) * kTileRows + g] = acc[n][0] + poison;
                mine[(8 * n + 2 * t + 1) * kTileRows + g] = acc[n][1] + poison;
                mine[(8 * n + 2 * t) * kTileRows + g + 8] = acc[n][2] + poison;
                mine[(8 * n + 2 * t + 1) * kTileRows + g + 8] = acc[n][3] + poison;
                acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            }
        } else {
            // scalar FP32 path for X that does not fit FP16 exactly: warp r computes tile rows r and r + 8
            // directly from global memory (same late scaling, FP32 accumulation), for every token; its partial
            // tile is zero everywhere else, so the common sum below still applies
            const int bwid = (w_now == p.nwin - 1) ? p.bw_last : p.bw;
            const int64_t j0 = (int64_t)w_now * p.bw;
            for (int i = lane; i < kOut; i += 32) mine[i] = poison;
            __syncwarp();
            for (int half = 0; half < 2; ++half) {
                const int64_t row = r0 + (int64_t)tile_now * kTileRows + warp + 8 * half;
                if (row >= r1) continue;
                for (int m = 0; m < p.M; ++m) {
                    float a = 0.f;
                    for (int j = lane; j < bwid; j += 32) {
                        const uint4 c = ld_stream_u4(MXQ_AT(codes + row * (p.K / 2) + (j0 + j) * 16, 16, codes, (int64_t)p.N * (p.K / 2)));
                        const float s = e8m0_to_float(*MXQ_AT(scales + row * p.kb + j0 + j, 1, scales, (int64_t)p.N * p.kb));
                        const uint32_t w4[4] = {c.x, c.y, c.z, c.w};
                        const uint16_t *xr = X + (int64_t)m * p.K + (j0 + j) * kBlock;
                        float part = 0.f;
#pragma unroll
                        for (int qd = 0; qd < 4; ++qd)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 wv = __half22float2(e2m1x2_to_half2((w4[qd] >> (8 * i)) & 0xFFu));
                                const uint32_t xb = __ldcg(MXQ_AT(reinterpret_cast<const uint32_t *>(xr + qd * 8 + i * 2), 4, X, (int64_t)p.M * p.K * 2));
                                part = fmaf(wv.x, __uint_as_float(xb << 16), part);
                                part = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part);
                            }
                        a = fmaf(part, s, a);
                    }
                    a = warp_sum(a);
                    if (lane == 0) mine[m * kTileRows + warp + 8 * half] = a;  // [token][row]
                }
            }
        }
        __threadfence_block();
        __syncwarp();
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(&s_cnt[rslot], 1);
        arrived = __shfl_sync(0xffffffffu, arrived, 0);
        if (arrived == kMmaWarps - 1) {
            // last warp in: sum the partial tiles in warp order
            __threadfence_block();
            float val[kPerLane];
            const float *all = s_red + rslot * kMmaWarps * kOut;
#pragma unroll
            for (int i = 0; i < kPerLane; ++i) {
                float v = 0.f;
#pragma unroll
                for (int w = 0; w < kMmaWarps; ++w) v += all[w * kOut + lane + 32 * i];
                val[i] = v;
            }
            __syncwarp();
            if (lane == 0) {
                s_cnt[rslot] = 0;
                __threadfence_block();
                *reinterpret_cast<volatile int *>(&s_gen[rslot]) = seg_index / kRedSlots + 1;  // slot free again
            }
            if (p.nwin > 1) {
                // windows are walked in order and each pair has exactly one summing warp, so the order of
                // these additions is fixed
                float *ta = s_acc + tile_now * kOut;
#pragma unroll
                for (int i = 0; i < kPerLane; ++i) {
                    if (w_now > 0) val[i] += ta[lane + 32 * i];
                    if (w_now < p.nwin - 1) ta[lane + 32 * i] = val[i];
                }
            }
            if (w_now == p.nwin - 1) {
#pragma unroll
                for (int i = 0; i < kPerLane; ++i) {
                    const int idx = lane + 32 * i, m_out = idx / kTileRows;
                    const int64_t n_out = r0 + (int64_t)tile_now * kTileRows + idx % kTileRows;
                    if (m_out < p.M && n_out < r1) store_out(Y, y_dtype, (int64_t)m_out * p.N + n_out, val[i], (int64_t)p.M * p.N);
                }
            }
        }
        ++seg_index;
    }
    cp_async_wait<0>();
}

// ---------------------------------------------------------------------------------------------
// host side: plan + launch
// ---------------------------------------------------------------------------------------------
bool linear_mma_plan(int M, int64_t N, int64_t K, LinearPlan &p) {
    if (M < 1 || M > 16 || (K % 128) != 0 || N < 1) return false;
    const int64_t kb = K / 32;
    if (kb > 65535 || N * (K / 2) >= (int64_t)1 << 32) return false;
    p.M = M;
    p.nt8 = M <= 8 ? 1 : 2;
    p.kb = (int)kb;
    p.N = N;
    p.K = K;
    const int sms = sm_count();
    const uint32_t kout_bytes = (uint32_t)p.nt8 * 8 * kTileRows * 4;
    const uint32_t red_bytes = (uint32_t)kRedSlots * kMmaWarps * kout_bytes;

    // grid: two CTAs per SM, more only if a CTA's stage table would overflow; never more CTAs than rows
    for (int mult = 2; mult <= 4096; mult *= 2) {
        int64_t grid = (int64_t)sms * mult;
        if (grid > N) grid = N;
        p.grid = (int)grid;
        const int64_t max_rows = (N + grid - 1) / grid;
        p.max_tiles = (int)((max_rows + kTileRows - 1) / kTileRows);

        // ring depth and K windows: prefer a quarter of an SM, 4 stages, one window
        auto layout = [&](int nstage, int64_t bw, int nwin) {
            p.off_acc = kOffRed + red_bytes;
            p.off_x = p.off_acc + (nwin > 1 ? (uint32_t)p.max_tiles * kout_bytes : 0u);
            p.x_stride = (uint32_t)(2 * bw * 32 + 64);
            p.off_ring = (p.off_x + (uint32_t)M * p.x_stride + 127) / 128 * 128;
            p.smem_bytes = p.off_ring + (uint32_t)(kMmaWarps * nstage * kWarpStageBytes);
            return p.smem_bytes;
        };
        int nstage = kMaxStages, nwin = 1;
        int64_t bw = kb;
        if (layout(nstage, bw, nwin) > kSmemThirdSm) {
            while (nstage > 2 && layout(nstage, bw, nwin) > kSmemHalfSm) --nstage;
            while (layout(nstage, bw, nwin) > kSmemHalfSm) {
                if (++nwin > 64) return false;
                bw = ((kb + nwin - 1) / nwin + 7) / 8 * 8;
            }
            while ((int64_t)(nwin - 1) * bw >= kb) --nwin;  // rounding up may have left the last window empty
            layout(nstage, bw, nwin);
        }
        p.nstage = nstage;
        p.nwin = nwin;
        p.bw = (int)bw;
        p.bw_last = (int)(kb - (int64_t)(nwin - 1) * bw);
        StageInfo si;
        if (stage_lookup(p, p.max_tiles, -1, si) <= kMaxCtaStages && p.smem_bytes <= kSmemHalfSm) return true;
        if (grid == N) return false;
    }
    return false;
}

size_t linear_mma_workspace_bytes(const LinearPlan &) { return 0; }

template <int NT8, int NS>
static cudaError_t launch_mma(const LinearPlan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                              int y_dtype, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_mma_kernel<NT8, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemHalfSm);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, linear_mma_kernel<NT8, NS>, p, (const uint16_t *)X, codes, scales, Y, y_dtype);
}

cudaError_t linear_mma_launch(const LinearPlan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                              int y_dtype, void *, cudaStream_t stream) {
#define MXQ_LAUNCH(NT, NSTG) launch_mma<NT, NSTG>(p, X, codes, scales, Y, y_dtype, stream)
    if (p.nt8 == 1) return p.nstage == 3 ? MXQ_LAUNCH(1, 3) : MXQ_LAUNCH(1, 2);
    return p.nstage == 3 ? MXQ_LAUNCH(2, 3) : MXQ_LAUNCH(2, 2);
#undef MXQ_LAUNCH
}

// returns and clears this kernel's sticky status word (see mxq_linear_device_status)
int linear_mma_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_mma_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_mma_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

MXQ_BOUNDS_TU(bounds_take_linear_mma)

}  // namespace mxq
