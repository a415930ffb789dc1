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
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxq_host.h"
#include "mxq_fp4_split.cuh"
#include "mxq_linear_fp4.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

namespace {

__device__ unsigned int g_fp4_status = 0;   // sticky: bit 0 full-wait, 1 empty-wait, 2 done-wait, 3 drain-wait gave up

constexpr uint32_t kFullArrivals = 1 + 32;   // the expect_tx arrive of the TMA lane + one cp.async arrive per producer lane

// Half of one 8-element unit of X (token m, k offset kk inside the CTA's range) into this CTA's operand buffers
// (sB_ / sSFB_ are shared-window addresses): see split_half_unit_to.
template <int NB>
__device__ __forceinline__ bool split_half_unit(const uint4 raw, int m, int kk, int half, int lane, uint32_t sB_, uint32_t sSFB_) {
    const uint32_t j = (uint32_t)kk >> 8, kin = (uint32_t)kk & 255u;
    return split_half_unit_to(raw, m, kin, half, lane, SplitToShared{sB_ + j * (NB * 128)}, SplitToShared{sSFB_ + j * kFp4SfStageBytes});
}

// NB: columns of the B operand / accumulator = 16 planes x tokens (16, 32 or 64).
// Warp roles (192 threads): warp 0 issues the MMAs and owns tensor memory; warp 1 is the producer (TMA copies of
// the codes, cp.async of the scale bytes, barrier set-up); warps 2..5 split the activations stage by stage and,
// at the end, read the accumulator (one row per thread), exchange partial results and store.
// MULTI: whether a CTA may own more than one tile (false: exactly one, and the per-tile loops fold away).
template <int NB, bool MULTI, int EPI>
__global__ void __launch_bounds__(kFp4Threads)
linear_fp4_kernel(const __grid_constant__ CUtensorMap tmap, const __nv_bfloat16 *__restrict__ X, int M,
                  const uint8_t *__restrict__ codes, const uint8_t *__restrict__ scales, int64_t N, int64_t K,
                  void *__restrict__ Y, int y_dtype, int split, int ring, int ks, int chunk_max, int tmem_cols, int groups,
                  int tiles, int tiles_max, const FusedAccept fa_arg) {
    extern __shared__ uint8_t smem_raw[];
    // EPI: what happens to a finished sum: stored (kEpiStore), competing for the verifier's argmax (kEpiAccept, fa.keys
    // set) or stored after a residual add or the gate / up pairing (kEpiLayer); a template parameter so that the plain
    // layer's epilogue carries none of the others
    FusedAccept fa = fa_arg;
    if (EPI != kEpiAccept) fa.keys = nullptr;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");   // needed by the first copy, 1 us from now
    const uint32_t rank = split > 1 ? cluster_rank() : 0u;
    const uint32_t group = blockIdx.x / (uint32_t)split;
    // this CTA's tiles [tile_lo, tile_lo + ntile) and, for all of them, its K range
    const int tile_lo = (int)((group * (uint32_t)tiles) / (uint32_t)groups);
    const int ntile = MULTI ? (int)(((group + 1u) * (uint32_t)tiles) / (uint32_t)groups) - tile_lo : 1;
    const int64_t n0 = (int64_t)tile_lo * kFp4TileRows;   // first weight row of the first tile
    // everything below fits in 32 bits (the plan refuses K >= 2^30 and more than 2^20 tiles)
    const int s_begin = (int)((rank * (uint32_t)ks) / (uint32_t)split), s_end = (int)(((rank + 1u) * (uint32_t)ks) / (uint32_t)split);
    const int nst = s_end - s_begin;   // stages of this CTA (>= 1 because split <= ks)
    const int kb_row = (int)((uint32_t)K >> 5);
    const int k_begin = s_begin * kFp4StageK;
    const int k_len = min(nst * kFp4StageK, (int)(uint32_t)K - k_begin);   // the tile's last stage may be half full
    const bool half_tail = (k_len & (kFp4StageK - 1)) != 0;

    // carve shared memory (1024-byte aligned for the 128-byte swizzle)
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base;
    const uint32_t sSFA = sA + (uint32_t)ring * kFp4StageBytes;
    const uint32_t sB = sSFA + (uint32_t)ring * kFp4SfStageBytes;
    const uint32_t sSFB = sB + (uint32_t)chunk_max * (NB * 128);
    const uint32_t sRecv = sSFB + (uint32_t)chunk_max * kFp4SfStageBytes;   // [tile][split][M][rows of this rank] floats
    const uint32_t sBar = sRecv + (split > 1 ? (uint32_t)(tiles_max * M) * kFp4RecvRows * 4u : 0u);   // no exchange, no buffer
    // barriers: full[ring], empty[ring], done, recv, ready[chunk_max]; then the tensor-memory address and two flags
    const uint32_t full0 = sBar, empty0 = sBar + (uint32_t)ring * 8u, done_bar = sBar + (uint32_t)ring * 16u;
    const uint32_t recv_bar = done_bar + 8u, ready0 = done_bar + 16u;
    const uint32_t sMisc = ready0 + (uint32_t)chunk_max * 8u;
    const float *gRecv = reinterpret_cast<const float *>(gbase + (sRecv - base));
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(gbase + (sMisc - base));
    volatile int &s_fail = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 4);
    const int row_lo = (int)(rank * kFp4TileRows) / split, row_cnt = (int)((rank + 1) * kFp4TileRows) / split - row_lo;
    const int groups_per_stage = 2 * M;   // a group = one warp's 32 tasks = 128 k of one token; a task = 8 elements x 8 planes

    // ---- prologue: barriers, tensor memory, and the first stages of weights (they do not depend on the previous
    //      kernel, so all of this runs before griddepcontrol.wait) -----------------------------------------------
    // The CTA's work is a sequence of units (tile, stage), tile-major; unit u goes through ring slot u % ring.
    const int nunit = ntile * nst;
    const int pre = nunit < ring ? nunit : ring;
    // The SM's requests are served roughly in order, so activations asked for behind a ring full of weight copies
    // arrive late, and everything after the split waits with them.  Only the first two units are requested up
    // front (1, 3 and 4 measured slower); the rest of the ring follows once the activations have been asked for, or
    // else at a trickle.
    const int pre0 = pre < 2 ? pre : 2;
    volatile int &s_xin = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 12);   // the activations have arrived
    // producer lane l owns rows l, l + 32, l + 64, l + 96 of a tile's scale bytes
    const uint8_t *srow0 = scales + (n0 + lane) * kb_row + s_begin * 8;
    const int64_t srow_step = (int64_t)32 * kb_row;
    const uint32_t sf_lane = sSFA + (uint32_t)lane * 16u;
    auto copy_scales = [&](int t, int i, uint32_t slot) {   // unit (t, i) into ring slot `slot` (all lanes of the producer warp)
        const bool second = !(half_tail && i == nst - 1);
        const uint32_t dst = sf_lane + slot * kFp4SfStageBytes;
        const uint8_t *src = srow0 + (int64_t)t * (4 * srow_step) + i * 8;
        const int rows_here = (int)min((int64_t)kFp4TileRows, N - n0 - (int64_t)t * kFp4TileRows);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (lane + 32 * q < rows_here) {
                cp_async4(dst + 4 * q, MXQ_AT(src, 4, scales, N * kb_row));
                if (second) cp_async4(dst + 4 * q + 512, MXQ_AT(src + 4, 4, scales, N * kb_row));
            }
            src += srow_step;
        }
        cp_async_arrive(full0 + slot * 8);
    };
    auto copy_codes = [&](int t, int i, uint32_t slot) {    // one lane
        mbar_expect_tx(full0 + slot * 8, kFp4StageBytes);
        tma_load_codes(sA + slot * kFp4StageBytes, &tmap, (s_begin + i) * (kFp4StageK / 2), (int)n0 + t * kFp4TileRows, full0 + slot * 8);
    };
    if (warp == 1) {
        for (int b = lane; b < 2 * ring + 2 + nst; b += 32) {
            const int st = b - (2 * ring + 2);   // >= 0: the barrier of stage st's share of the activations
            const uint32_t count = b < ring ? kFullArrivals
                                   : (st < 0 ? 1u : (uint32_t)((half_tail && st == nst - 1) ? M : groups_per_stage));
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
    // Only the activation warps read what the previous kernel wrote (X) and write what the next one reads (Y).  One of
    // them waits for it, at once (the wait makes the previous grid's writes visible to this whole grid, and a chain of
    // dependent launches runs 0.2 us per launch faster with one waiting warp than with four); the others meet it at the
    // CTA-wide barrier below (initialised mbarriers, tensor-memory address).
    if (warp >= 2) {
        if (warp == 2) pdl_wait();
    }
    if (split > 1) cluster_arrive();   // "my barriers exist"; the matching wait is just before the first push to a peer
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;
    if (warp == 1) {
        for (int u = 0, t = 0, i = 0; u < pre; ++u) {
            if (u >= pre0) {
                for (int spin = 0; spin < 3 && !s_xin; ++spin) __nanosleep(100);
                if (lane == 0) copy_codes(t, i, (uint32_t)u);
            }
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
        const uint32_t idesc = (1u << 7) | (1u << 10) | (((uint32_t)NB >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
        const uint32_t a_hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32), b_hi = (uint32_t)(smem_desc(0, 128, 1024, 0) >> 32);
        const uint32_t s_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);
        const uint32_t a_lo0 = (uint32_t)smem_desc(sA, 16, 1024, 2), s_lo0 = (uint32_t)smem_desc(sSFA, 0, 128, 0);
        const uint32_t b_lo0 = (uint32_t)smem_desc(sB, 128, 1024, 0), sb_lo0 = (uint32_t)smem_desc(sSFB, 0, 128, 0);
        const uint32_t t_sf0 = tmem + (uint32_t)(NB * tiles_max);   // after the accumulators: two slots of 8 + 8 scale columns
        uint32_t slot = 0, phase = 0, par = 0;
        bool ok = true;
        for (int t = 0; t < ntile && ok; ++t) {
          const uint32_t t_acc = tmem + (uint32_t)(t * NB);   // this tile's accumulator columns
          uint32_t b_lo = b_lo0, sb_lo = sb_lo0, accumulate = 0;
          for (int i = 0; i < nst; ++i) {
            // the unit's weights and scales have landed and (first tile only; the others find it done) the stage's
            // share of the activations has been split
            if ((t == 0 && !mbar_wait_relaxed(ready0 + (uint32_t)i * 8u, 0)) || !mbar_wait_relaxed(full0 + slot * 8, phase)) {
                if (lane == 0) {
                    atomicOr(&g_fp4_status, 1u);
                    s_fail = 1;
                }
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + slot * (kFp4StageBytes >> 4);
            const uint32_t sa_lo = s_lo0 + slot * (kFp4SfStageBytes >> 4);
            const int nmma = (half_tail && i == nst - 1) ? 2 : 4;
            const uint32_t t_sf = t_sf0 + par * 16u;   // alternating between consecutive units
            par ^= 1u;
            if (elect_one()) {
                fence_async_proxy();   // the weight scale atoms were written by cp.async
                tc_copy_sf_lohi(t_sf, sa_lo, s_hi);
                tc_copy_sf_lohi(t_sf + 4, sa_lo + 32, s_hi);
                tc_copy_sf_lohi(t_sf + 8, sb_lo, s_hi);
                tc_copy_sf_lohi(t_sf + 12, sb_lo + 32, s_hi);
                auto mma = [&](int j, uint32_t acc) {   // k [64 j, 64 j + 64) of the stage: scales 2 (j & 1), + 1 of atom j >> 1
                    const uint32_t sfid = (uint32_t)(j & 1) * 2u;
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
                        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %5, [%7], [%8], p;\n\t}"
                        ::"r"(t_acc), "r"(a_lo + j * 2), "r"(a_hi), "r"(b_lo + j * 16), "r"(b_hi),
                        "r"(idesc | (sfid << 4) | (sfid << 29)), "r"(acc), "r"(t_sf + 4u * (j >> 1)), "r"(t_sf + 8u + 4u * (j >> 1))
                        : "memory");
                };
                mma(0, accumulate);
                mma(1, 1u);
                if (nmma == 4) {
                    mma(2, 1u);
                    mma(3, 1u);
                }
                tc_commit(empty0 + slot * 8);
            }
            accumulate = 1;
            b_lo += (NB * 128) >> 4;
            sb_lo += kFp4SfStageBytes >> 4;
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
                    atomicOr(&g_fp4_status, 2u);
                    s_fail = 1;
                }
                break;
            }
            // (requests from a second warp are served beside this lane's, but measured no gain here: 128256 x 4096 got slower)
            if (lane == 0) copy_codes(t, i, slot);
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
        {
            // Groups of 32 tasks (128 k of one token, one warp) in stage-major order, so that the MMA warp can start on
            // stage 0 while later stages are being split.  Group G: stage G / (2M), then token and 128-k half; in a half
            // tail stage every group is a different token.  All of this is uniform across a warp.
            const int ngroups = (k_len >> 7) * M;
            const __nv_bfloat16 *xbase = X + k_begin;
            const int cw = ct >> 5;
            constexpr int kBatch = 4;   // loads in flight per thread
            for (int G0 = 0; G0 < ngroups; G0 += 4 * kBatch) {
                uint4 raw[kBatch];
                int mm[kBatch], kk[kBatch], stage[kBatch];
#pragma unroll
                for (int b = 0; b < kBatch; ++b) {   // all loads of the batch first
                    const int G = G0 + 4 * b + cw;
                    mm[b] = -1;
                    kk[b] = stage[b] = 0;
                    raw[b] = make_uint4(0, 0, 0, 0);
                    if (G < ngroups) {
                        const int st = M == 1 ? (G >> 1) : (M == 2 ? (G >> 2) : (M == 3 ? G / 6 : (G >> 3)));
                        const int rem = G - st * groups_per_stage;
                        const bool tail = half_tail && st == nst - 1;
                        stage[b] = st;
                        mm[b] = tail ? rem : (rem >> 1);
                        kk[b] = st * kFp4StageK + (tail ? 0 : (rem & 1) * 128) + (lane >> 1) * 8;
                        raw[b] = ld_ordered_u4(MXQ_AT(xbase + (int64_t)mm[b] * K + kk[b], 16, X, (int64_t)M * K * 2));
                    }
                }
                // The activations have been asked for: weight copies requested from here on queue up behind them, so
                // the producer may request the rest of the ring (asm volatile keeps this store after the loads).
                if (G0 == 0 && ct == 0) st_shared_flag(sMisc + 12, 1);
#pragma unroll
                for (int b = 0; b < kBatch; ++b)
                    if (G0 + 4 * b + cw < ngroups) {   // uniform across the warp
                        inexact |= split_half_unit<NB>(raw[b], mm[b], kk[b], lane & 1, lane, sB, sSFB);
                        fence_async_proxy();   // ordinary stores, read by the tensor core
                        __syncwarp();
                        if (lane == 0) mbar_arrive(ready0 + (uint32_t)stage[b] * 8u);
                    }
            }
        }
        if (inexact) s_bad = 1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const int bad = s_bad;

        // ---- epilogue: accumulator row -> registers; a token's 16 planes are 16 columns, smallest first ------------
        constexpr int MT = NB / kFp4Planes;   // token slots per tile (1, 2 or 4)
        // layer epilogues: the residual values this thread will add to its first tile's sums, requested before the wait
        float res[MT];   // (unused, and optimised away, in the other epilogues)
        if (EPI == kEpiLayer && split == 1) {
            const int64_t n_first = (int64_t)tile_lo * kFp4TileRows + row;
            layer_prefetch<MT>(fa, y_dtype, M, n_first, N, n_first < N, res);
        }
        if (!mbar_wait_relaxed(done_bar, 0)) {
            atomicOr(&g_fp4_status, 4u);
            s_fail = 1;
        }
        tc_fence_after();
        // Tile by tile: this thread's row of the accumulator -> registers -> direct store (split == 1) or, for the sum over
        // the cluster in a fixed order, a push to the row's owner.  Rank q owns rows [q*128/split, (q+1)*128/split) of every
        // tile of the group: every CTA pushes its partial results for those rows into q's shared memory (slot = tile,
        // sender's rank) with stores that count on q's mbarrier; q waits for all of them and adds them in a fixed
        // order.  No CTA reads a peer's memory, and a CTA leaves only after everything addressed to it has arrived.
        const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int cnt_max = (kFp4TileRows + split - 1) / split;
        const uint32_t owner = (uint32_t)(((row + 1) * split - 1) / kFp4TileRows);
        const int rr = row - (int)(owner * kFp4TileRows) / split;
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
                for (int m = 0; m < MT; ++m) {
                    float d[16];
                    tc_load16(t_row + t * NB + m * 16, d);
                    float acc = d[15];
#pragma unroll
                    for (int p = 14; p >= 0; --p) acc += d[p];
                    yt[m] = acc;
                }
            } else {
                // Scalar path for a K range whose X cannot be rewritten exactly (the MMA results are ignored).
                const int64_t n = n0 + (int64_t)t * kFp4TileRows + row;
                float acc[kFp4MaxM];
#pragma unroll
                for (int m = 0; m < kFp4MaxM; ++m) acc[m] = 0.f;
                if (n < N) {
                    const uint4 *crow = reinterpret_cast<const uint4 *>(codes + n * (K / 2));
                    const uint8_t *srw = scales + n * kb_row;
                    for (int blk = k_begin / 32; blk < (k_begin + k_len) / 32; ++blk) {
                        const uint4 c = ld_stream_u4(MXQ_AT(crow + blk, 16, codes, N * (K / 2)));
                        const float sc = e8m0_to_float(*MXQ_AT(srw + blk, 1, scales, N * kb_row)) * kGuardDown;
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
                                        const uint32_t xb = ld_dep_u32(MXQ_AT(X + (int64_t)m * K + k, 4, X, (int64_t)M * K * 2));
                                        part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                                        part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                                    }
                            }
#pragma unroll
                        for (int m = 0; m < kFp4MaxM; ++m) acc[m] = fmaf(part[m], sc, acc[m]);
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
                const int64_t n = n0 + (int64_t)t * kFp4TileRows + row;
                if (EPI == kEpiLayer) {
                    // (gate / up pairing: the partner row's sum sits in the neighbouring lane)
#pragma unroll
                    for (int m = 0; m < MT; ++m) yt[m] *= kGuardUp;
                    layer_emit<MT>(fa, Y, y_dtype, M, n, N, n < N, yt, res, 1);
                    if (t + 1 < ntile) layer_prefetch<MT>(fa, y_dtype, M, n + kFp4TileRows, N, n + kFp4TileRows < N, res);
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
                scatter_prefetch<MT>(fa, y_dtype, M, split, ct & (split - 1), (int64_t)tile_lo * kFp4TileRows + row_lo + ct / split, N, res_s);
            if (!mbar_wait_relaxed(recv_bar, 0)) {
                atomicOr(&g_fp4_status, 16u);
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
                    const int64_t n = n0 + (int64_t)t * kFp4TileRows + row_lo + r;
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
                    const int64_t n = n0 + (int64_t)t * kFp4TileRows + row_lo + r;
                    if (EPI != kEpiAccept) {
                        // plain store and layer epilogues: reduce-scatter over the token rows, every lane finishes its share
                        scatter_sum_store<MT, EPI>(gRecv + ((t * split + j) * M) * cnt_max + r, cnt_max, M, split, j, n, N, kGuardUp, poison,
                                                   fa, Y, y_dtype, res_s);
                        if (EPI == kEpiLayer && t + 1 < ntile) scatter_prefetch<MT>(fa, y_dtype, M, split, j, n + kFp4TileRows, N, res_s);
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

template <int NB, bool MULTI, int EPI>
cudaError_t launch_fp4(const Fp4Plan &p, const CUtensorMap &map, const void *X, const uint8_t *codes,
                       const uint8_t *scales, void *Y, int y_dtype, cudaStream_t stream, const FusedAccept &fa) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_fp4_kernel<NB, MULTI, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kFp4SmemLimit);
        if (e != cudaSuccess) return e;
        // all of the SM's L1/shared array as shared memory: how many CTAs (of this and of the next kernel) fit on an
        // SM is what decides how early the next kernel's weight stream can start
        e = cudaFuncSetAttribute(linear_fp4_kernel<NB, MULTI, EPI>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
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
    return cudaLaunchKernelEx(&cfg, linear_fp4_kernel<NB, MULTI, EPI>, map, (const __nv_bfloat16 *)X, p.M, codes, scales, p.N, p.K,
                              Y, y_dtype, p.split, p.ring, p.ks, p.chunk_max, p.tmem_cols, p.groups, p.tiles, p.tiles_max, fa);
}

}  // namespace

bool linear_fp4_plan(int M, int64_t N, int64_t K, Fp4Plan &p, bool pow2_split) {
    if (M < 1 || M > kFp4MaxM || N < 1 || K < 128 || (K % 128) != 0) return false;
    if (K > 0x3FFFFFFF || N > 0x7FFFFFFF) return false;
    p.M = M;
    p.N = N;
    p.K = K;
    p.nb = M == 1 ? 16 : (M == 2 ? 32 : 64);
    p.ks = (int)((K + kFp4StageK - 1) / kFp4StageK);
    p.tiles = (int)((N + kFp4TileRows - 1) / kFp4TileRows);
    p.pow2_split = pow2_split ? 1 : 0;
    const LayoutOverride o = layout_override();
    return fp4_layout(p, sm_count(), o.split, o.ring, o.tiles);
}

cudaError_t linear_fp4_launch(const Fp4Plan &p, const void *X, const uint8_t *codes, const uint8_t *scales, void *Y,
                              int y_dtype, cudaStream_t stream, const FusedAccept *fused) {
    CUtensorMap map;
    if (!codes_tensor_map(codes, p.N, p.K, /*expand_fp4=*/false, &map)) return cudaErrorNotSupported;
    const bool multi = p.tiles_max > 1;
    const FusedAccept fa = fused ? *fused : FusedAccept{};
    if (fa.swiglu && ((p.split & (p.split - 1)) != 0 || (p.N & 1))) return cudaErrorNotSupported;   // see linear_fp4_plan's pow2_split
#define MXQ_FP4_PICK(NB, EPI)                                                                             \
    return multi ? launch_fp4<NB, true, EPI>(p, map, X, codes, scales, Y, y_dtype, stream, fa)             \
                 : launch_fp4<NB, false, EPI>(p, map, X, codes, scales, Y, y_dtype, stream, fa)
#define MXQ_FP4_PICK_EPI(NB)                                     \
    switch (epilogue_kind(fa)) {                                 \
        case kEpiAccept: MXQ_FP4_PICK(NB, kEpiAccept);           \
        case kEpiLayer: MXQ_FP4_PICK(NB, kEpiLayer);             \
        default: MXQ_FP4_PICK(NB, kEpiStore);                    \
    }
    switch (p.nb) {
        case 16: MXQ_FP4_PICK_EPI(16)
        case 32: MXQ_FP4_PICK_EPI(32)
        default: MXQ_FP4_PICK_EPI(64)
    }
#undef MXQ_FP4_PICK_EPI
#undef MXQ_FP4_PICK
}


// returns and clears this kernel's sticky status word (see mxq_linear_device_status)
int linear_fp4_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_fp4_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_fp4_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

MXQ_BOUNDS_TU(bounds_take_linear_fp4)

}  // namespace mxq
