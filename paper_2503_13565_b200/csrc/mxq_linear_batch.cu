// mxq_linear_batch: the MXFP4 layers of one decoding step (Sec. III-D-3, Eq. 2; Sec. III-B: a draft step is the stream
// of its weights) in ONE persistent launch, for 1..4 token rows.
//
// A decoder layer is seven small matrices; launched one by one, each call pays a dependent chain of several
// microseconds (launch, activations arrive, rewrite them as tensor-core operands, sum over the cluster, store) against
// 1.4-3.7 us of weight traffic.  Here one grid of one CTA per SM walks all the layers of the call:
//   - The call's work is the sequence of units (layer, 128-row tile, 256-k stage), tile-major, cut into as many
//     contiguous ranges as there are CTAs.  A CTA streams whole weight rows for most of its range, and its TMA ring
//     runs on across tile and layer boundaries, so the weight stream never drains inside a call.
//   - The token rows are rewritten ONCE per distinct X (16 radix-4 digit planes per row, see mxq_fp4_split.cuh) by
//     all CTAs together into an image in the workspace, at the start of the kernel and while the first weights are
//     already in flight; every unit then fetches its 256 k of the image with one bulk copy beside its weights.
//   - A tile whose stages fall into two or three CTAs' ranges is finished by whichever of them delivers last: each
//     writes its partial sums to the workspace and takes a ticket; the last one adds the parts in range order (so the
//     result does not depend on who was last) and stores.
//   - Accumulators alternate between several tensor-memory slots, so the MMAs of the next tile start while the
//     epilogue warps read the previous one.
// Warp roles (320 threads): warp 0 issues the MMAs and owns tensor memory; warp 1 is the producer (TMA copies of the
// codes, bulk copies of the token operand); warps 2..5 first rewrite their share of the token rows and then run the
// epilogues; warps 6..9 move the scale bytes into the slots' scale atoms (warp w those of every fourth unit).  Every wait is bounded; one that gives up sets a sticky status bit and the
// CTA's remaining tiles are written as NaN.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxq_fp4_split.cuh"
#include "mxq_host.h"
#include "mxq_linear_batch.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

namespace {

// sticky: bit 0 a stage's data never arrived, 1 a ring slot was never released, 2 an accumulator never completed or was
// never released, 3 the token operand never became ready
__device__ unsigned int g_batch_status = 0;

constexpr uint32_t kFullArrivals = 1 + 1;   // the producer's arrive (with the bytes it announces) + the arrive of the scale warp that serves the unit

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 ld_cg_u4(const void *p) {   // through L2 only: another SM may have written it during this kernel
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ld_cg_f32(const float *p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ float load_in_cg(const void *R, int dtype, int64_t idx, int64_t count) {
    (void)count;
    if (dtype == MXQ_F32) return ld_cg_f32(MXQ_AT(reinterpret_cast<const float *>(R) + idx, 4, R, count * 4));
    unsigned short h;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(h) : "l"(MXQ_AT(reinterpret_cast<const unsigned short *>(R) + idx, 2, R, count * 2)) : "memory");
    return __uint_as_float((uint32_t)h << 16);
}


// Bounded wait on an mbarrier that also ends when the CTA's failure flag is raised.  False: gave up.  The probes are
// back to back (the instruction itself suspends the warp for a while when the phase is not complete): a sleep between
// probes costs far more than its nominal duration and put a floor of most of a microsecond under every wait.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *fail, uint32_t limit_us) {
    for (int i = 0; i < 1024; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 1024; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*fail || global_ns() - t0 > (uint64_t)limit_us * 1000ull) return false;
    }
}
// The same for a whole (converged) warp with ONE lane probing: threads that probe an mbarrier occupy the SM's
// shared-memory pipeline while they wait, and with all the waiting warps of a CTA probing (some 160 threads) every
// barrier operation of the CTA queued behind them: a unit of work took 0.9 us whatever it contained.
__device__ __forceinline__ bool warp_wait_bar(uint32_t bar, uint32_t parity, volatile int *fail, uint32_t limit_us, int lane) {
    int ok = 1;
    if (lane == 0) ok = wait_bar(bar, parity, fail, limit_us) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
// Bounded wait until a counter in global memory reaches `want`.  (Probes back to back: spacing them out with nanosleep was
// measured and cost a microsecond per launch without relieving anything.)
__device__ __forceinline__ bool wait_counter(const uint32_t *ctr, uint32_t want, volatile int *fail, uint32_t limit_us) {
    for (int i = 0; i < 256; ++i)
        if (ld_acquire_u32(ctr) >= want) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (ld_acquire_u32(ctr) >= want) return true;
        if (*fail || global_ns() - t0 > (uint64_t)limit_us * 1000ull) return false;
    }
}

// position in the call's unit sequence
struct Cursor {
    int d, t, s, ks, tiles;
};
__device__ __forceinline__ void cursor_at(const BatchTable &tb, int u, Cursor &c) {
    int d = 0, hi = tb.ndesc;   // the last layer whose first unit is <= u (bisection: up to 64 layers, and the scale warps ask per unit)
    while (hi - d > 1) {
        const int mid = (d + hi) >> 1;
        if (u >= tb.desc[mid].unit_base) d = mid;
        else hi = mid;
    }
    c.d = d;
    c.ks = tb.desc[d].ks;
    c.tiles = tb.desc[d].tiles;
    const int r = u - tb.desc[d].unit_base;
    c.t = r / c.ks;
    c.s = r - c.t * c.ks;
}
__device__ __forceinline__ void cursor_next(const BatchTable &tb, Cursor &c) {
    if (++c.s == c.ks) {
        c.s = 0;
        if (++c.t == c.tiles) {
            c.t = 0;
            if (++c.d < tb.ndesc) {
                c.ks = tb.desc[c.d].ks;
                c.tiles = tb.desc[c.d].tiles;
            }
        }
    }
}

// The order in which a CTA walks its range [u0, u0 + nunit): if the range ends inside a tile, that last piece (`tail`
// units, shared with the next CTA's range) comes first, then the range from its start.  Both pieces of a shared tile
// are thus delivered early in their CTAs' runs, and the sum across CTAs is hidden behind the rest of the stream
// instead of trailing the kernel.
struct Walk {
    int u0, nunit, tail;
};
__device__ __forceinline__ int walk_unit(const Walk &w, int i) { return i < w.tail ? w.u0 + w.nunit - w.tail + i : w.u0 + i - w.tail; }
__device__ __forceinline__ void walk_begin(const BatchTable &tb, const Walk &w, Cursor &c) { cursor_at(tb, walk_unit(w, 0), c); }
// from element i - 1 to element i
__device__ __forceinline__ void walk_to(const BatchTable &tb, const Walk &w, int i, Cursor &c) {
    if (w.tail != 0 && i == w.tail) cursor_at(tb, w.u0, c);
    else cursor_next(tb, c);
}
// element i opens / closes a piece of a tile (a run of stages that share an accumulator)
__device__ __forceinline__ bool walk_opens(const Walk &w, int i, const Cursor &c) { return i == 0 || i == w.tail || c.s == 0; }
__device__ __forceinline__ bool walk_closes(const Walk &w, int i, const Cursor &c) { return i == w.nunit - 1 || i == w.tail - 1 || c.s == c.ks - 1; }

// NB: columns of the token operand / accumulator = 16 planes x token slots (16, 32 or 64).
template <int NB, bool GROUPS>
__global__ void __launch_bounds__(kBatchThreads, 2) linear_batch_kernel(const __grid_constant__ BatchTable tb) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int MT = NB / 16;   // token slots
    constexpr uint32_t kXBytes = (uint32_t)NB * 128u + kBatchSfBytes;
    constexpr uint32_t kSlot = kBatchCodesBytes + kBatchSfBytes + kXBytes;
    const int A = tb.acc_slots;   // accumulator slots (1..4)
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = (int)gridDim.x, cta = (int)blockIdx.x;
    const int M = tb.M, ring = tb.ring;
    // The layers of a call form groups (a layer flagged as depending on earlier ones opens a new group); every group's
    // units are cut into ranges of their own, and all CTAs go through the groups in order.
    const int ngroups = GROUPS ? tb.ngroups : 1;
    // (64-bit divisions and a search: tens of thousands of cycles for one thread if every role did this for every
    // group after the wait below.  One lane per group does it before the wait and leaves the result in shared memory.)
    auto compute_walk = [&](int g, Walk &w) {   // this CTA's range of group g (nunit = 0: none)
        const int gu = tb.group_unit[g], ug = tb.group_unit[g + 1] - gu, gg = ug < G ? ug : G;
        w.u0 = gu;
        w.nunit = w.tail = 0;
        if (cta < gg) {
            w.u0 = gu + (int)((int64_t)cta * ug / gg);
            w.nunit = gu + (int)((int64_t)(cta + 1) * ug / gg) - w.u0;
            Cursor last;
            cursor_at(tb, w.u0 + w.nunit - 1, last);
            w.tail = (last.s != last.ks - 1 && last.s + 1 < w.nunit) ? last.s + 1 : 0;
        }
    };
    const uint32_t limit_us = tb.wait_us;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sBar = base + (uint32_t)ring * kSlot;
    const uint32_t full0 = sBar, empty0 = sBar + (uint32_t)ring * 8u;
    const uint32_t accf0 = sBar + (uint32_t)ring * 16u, acce0 = accf0 + 4u * 8u;
    const uint32_t sMisc = acce0 + 4u * 8u;
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(gbase + (sMisc - base));
    volatile int *s_fail = reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 4);
    volatile int *s_flag = reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 8);
    volatile int *s_zero = reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 12);   // always 0
    int *s_walk = reinterpret_cast<int *>(gbase + (sMisc - base) + 16);                      // [kBatchMaxGroups][3]
    auto group_walk = [&](int g, Walk &w) {   // (valid after the block-wide barrier of the set-up)
        w.u0 = s_walk[3 * g];
        w.nunit = s_walk[3 * g + 1];
        w.tail = s_walk[3 * g + 2];
    };

    uint32_t *hdr = reinterpret_cast<uint32_t *>(tb.ws);
    // (counter i of a kind lives kBatchCounterStride words after counter i - 1: a 128-byte line each)
    uint32_t *g_ready = hdr + kBatchWordReady, *g_bad = hdr + kBatchWordBad;

    // ---- set-up -------------------------------------------------------------------------------------------------------
    if (warp == 1) {
        for (int b = lane; b < 2 * ring + 8; b += 32) {
            const uint32_t count = b < ring ? kFullArrivals : (b < 2 * ring ? 1u : (b < 2 * ring + 4 ? 1u : 4u));
            mbar_init(sBar + (uint32_t)b * 8u, count);
        }
        if (lane == 0) {
            *s_fail = 0;
            *s_flag = 0;
            *s_zero = 0;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
    } else if (warp == 0) {
        pdl_trigger();   // the next kernel in the stream may start its own set-up
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sMisc), "r"(tb.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // One thread walks a CTA's units, and a lone thread issues an instruction every few cycles at best: what a role
    // does per unit has to stay at a few dozen instructions (no divisions, nothing re-read from the parameter table
    // that only changes with the layer).  Slot addresses, parities and descriptors are carried along incrementally.

    // The first ring of weights does not depend on the previous kernel in the stream: requested before the wait.
    // producer state: the ring position of the next unit whose codes are requested (carried across groups)
    uint32_t c_slot = base, c_fb = full0, c_eb = empty0, c_phase = 0;
    int c_count = 0;   // units whose codes have been requested so far
    const uint32_t ring_end = base + (uint32_t)ring * kSlot;
    // codes of the first `n` units of walk `w` (announced without an arrival: the arrival comes with the operand)
    auto request_codes_only = [&](const Walk &w, int n) -> bool {
        Cursor c;
        for (int i = 0; i < n; ++i) {
            if (i) walk_to(tb, w, i, c);
            else walk_begin(tb, w, c);
            if (c_count >= ring && !wait_bar(c_eb, c_phase, s_fail, limit_us)) return false;
            // (test hook: the bytes of unit tb.fault_unit are announced but never requested)
            asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(c_fb), "r"(kBatchCodesBytes) : "memory");
            if (walk_unit(w, i) != tb.fault_unit) tma_load_codes(c_slot, &tb.maps[c.d], c.s * (kBatchStageK / 2), c.t * kBatchTileRows, c_fb);
            c_slot += kSlot;
            c_fb += 8u;
            c_eb += 8u;
            if (c_slot == ring_end) {
                c_slot = base;
                c_fb = full0;
                c_eb = empty0;
                if (c_count >= ring) c_phase ^= 1u;
            }
            ++c_count;
        }
        return true;
    };
    int units_left = 0;   // (epilogue warps) of this CTA, over all groups: the last piece lets tensor memory go back
    if (warp >= 2 && warp < 6) {
        if (warp == 3 && lane < ngroups) {
            Walk w;
            compute_walk(lane, w);
            s_walk[3 * lane] = w.u0;
            s_walk[3 * lane + 1] = w.nunit;
            s_walk[3 * lane + 2] = w.tail;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        for (int g = 0; g < ngroups; ++g) units_left += s_walk[3 * g + 1];
    }
    if (warp == 1) {
        for (int d = lane; d < tb.ndesc; d += 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&tb.maps[d]) : "memory");
        __syncwarp();
        if (lane == 0) {
            Walk wk0;
            compute_walk(0, wk0);
            (void)request_codes_only(wk0, wk0.nunit < ring ? wk0.nunit : ring);   // (nothing to wait for yet)
        }
        __syncwarp();
        pdl_wait();   // the counters in the workspace belong to the previous call until it has completed
    }
    if (warp == 2) pdl_wait();   // X, Y and the workspace
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;

    if (warp == 0) {
        // ---- MMA warp -------------------------------------------------------------------------------------------------
        const uint32_t idesc = (1u << 7) | (1u << 10) | (((uint32_t)NB >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24);
        const uint32_t a_hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32), b_hi = (uint32_t)(smem_desc(0, 128, 1024, 0) >> 32);
        const uint32_t s_hi = (uint32_t)(smem_desc(0, 0, 128, 0) >> 32);
        const uint32_t t_sf0 = tmem + (uint32_t)(A * NB);   // after the accumulators: two slots of 8 + 8 scale columns
        // descriptors of slot 0; a slot further on adds kSlot / 16 to each start-address field (the whole ring lies
        // below 256 KB, so the 14-bit field never carries)
        const uint32_t a_lo0 = (uint32_t)smem_desc(base, 16, 1024, 2);
        const uint32_t sa_lo0 = (uint32_t)smem_desc(base + kBatchCodesBytes, 0, 128, 0);
        const uint32_t b_lo0 = (uint32_t)smem_desc(base + kBatchCodesBytes + kBatchSfBytes, 128, 1024, 0);
        const uint32_t sb_lo0 = (uint32_t)smem_desc(base + kBatchCodesBytes + kBatchSfBytes + (uint32_t)NB * 128u, 0, 128, 0);
        int d_seen = -1;
        bool half_k = false;
        uint32_t slot = 0, phase = 0, par = 0, accumulate = 0, off16 = 0;
        int acc_slot = -1;
        uint32_t acc_round = 0;   // how often the accumulator slots have wrapped
        uint32_t t_acc = tmem;
        bool alive = true;
        for (int g = 0; g < ngroups && alive; ++g) {
        Walk wk;
        group_walk(g, wk);
        const int nunit = wk.nunit;
        Cursor c;
        if (nunit) walk_begin(tb, wk, c);
        for (int i = 0; i < nunit; ++i) {
            if (i) walk_to(tb, wk, i, c);
            if (c.d != d_seen) {
                d_seen = c.d;
                half_k = (tb.desc[c.d].K & (kBatchStageK - 1)) != 0;
            }
            if (walk_opens(wk, i, c)) {   // the next accumulator slot, once the epilogue has read what it held
                if (++acc_slot == A) {
                    acc_slot = 0;
                    ++acc_round;
                }
                if (acc_round != 0 && !warp_wait_bar(acce0 + (uint32_t)acc_slot * 8u, (acc_round - 1u) & 1u, s_fail, limit_us, lane)) {
                    if (lane == 0) {
                        atomicOr(&g_batch_status, 4u);
                        *s_fail = 1;
                    }
                    alive = false;
                    break;
                }
                tc_fence_after();
                t_acc = tmem + (uint32_t)(acc_slot * NB);
                accumulate = 0;
            }
            if (!warp_wait_bar(full0 + slot * 8u, phase, s_fail, limit_us, lane)) {
                if (lane == 0) {
                    atomicOr(&g_batch_status, 1u);
                    *s_fail = 1;
                }
                alive = false;
                break;
            }
            tc_fence_after();
            const bool half_tail = half_k && c.s == c.ks - 1;
            const bool closes = walk_closes(wk, i, c);
            const uint32_t t_sf = t_sf0 + par * 16u;
            par ^= 1u;
            if (elect_one()) {
                const uint32_t a_lo = a_lo0 + off16, sa_lo = sa_lo0 + off16, b_lo = b_lo0 + off16, sb_lo = sb_lo0 + off16;
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
                if (!half_tail) {
                    mma(2, 1u);
                    mma(3, 1u);
                }
                tc_commit(empty0 + slot * 8u);
                if (closes) tc_commit(accf0 + (uint32_t)acc_slot * 8u);
            }
            __syncwarp();
            accumulate = 1;
            off16 += kSlot >> 4;
            if (++slot == (uint32_t)ring) {
                slot = 0;
                off16 = 0;
                phase ^= 1u;
            }
        }
        }
        __syncwarp();
        // tensor memory goes back once the epilogue warps have read their last accumulator
        asm volatile("bar.sync 2, 160;" ::: "memory");
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tb.tmem_cols) : "memory");
    } else if (warp == 1) {
        // ---- producer warp (one lane works) ------------------------------------------------------------------------------
        // The codes of the first ring are on their way; their share of the token operand follows as soon as the image
        // it comes from is complete (all of a call's images are, a microsecond or two into the kernel).  After that a
        // unit's codes and operand are requested together, as soon as the MMAs have released the slot they go to.
        if (lane == 0) {
            uint64_t ready_mask = 0;
            int d_seen = -1, im = 0;
            const CUtensorMap *map = nullptr;
            const uint8_t *img = nullptr;
            bool ok = true;
            auto layer = [&](const Cursor &c) -> bool {   // the cursor has entered another layer
                d_seen = c.d;
                map = &tb.maps[c.d];
                im = tb.desc[c.d].img;
                img = tb.ws + tb.img[im].offset;
                if (!((ready_mask >> im) & 1ull)) {
                    if (!wait_counter(g_ready + im * kBatchCounterStride, (uint32_t)tb.img[im].ntasks, s_fail, limit_us)) {
                        atomicOr(&g_batch_status, 8u);
                        *s_fail = 1;
                        return false;
                    }
                    fence_proxy_async_all();   // the image was written with ordinary stores; the bulk copies read it through the async proxy
                    ready_mask |= 1ull << im;
                }
                return true;
            };
            // the ring position of the next unit whose operand is requested (behind the codes by at most a ring)
            uint32_t o_slot = base, o_fb = full0;
            int issued = 0;   // units whose data has been requested in full
            for (int g = 0; g < ngroups && ok; ++g) {
                Walk wk;
                group_walk(g, wk);
                const int nunit = wk.nunit;
                if (nunit == 0) continue;
                const int pre = nunit < ring ? nunit : ring;
                // A group's first ring of codes is requested before its token operand exists (group 0: before the previous
                // kernel has completed; later groups: while the layers they depend on are being finished), as the slots
                // come free.
                if (g > 0 && !request_codes_only(wk, pre)) {
                    atomicOr(&g_batch_status, 2u);
                    *s_fail = 1;
                    ok = false;
                    break;
                }
                Cursor c;
                walk_begin(tb, wk, c);
                for (int i = 0; i < pre && ok; ++i) {
                    if (i) walk_to(tb, wk, i, c);
                    if (c.d != d_seen) ok = layer(c);
                    if (!ok) break;
                    mbar_expect_tx(o_fb, kXBytes);
                    bulk_load(o_slot + kBatchCodesBytes + kBatchSfBytes, MXQ_AT(img + (uint32_t)c.s * kXBytes, kXBytes, tb.ws, tb.ws_bytes), kXBytes, o_fb);
                    o_slot += kSlot;
                    o_fb += 8u;
                    if (o_slot == ring_end) {
                        o_slot = base;
                        o_fb = full0;
                    }
                    ++issued;
                }
                // from here on codes and operand of a unit go out together (the two ring positions coincide again)
                for (int i = pre; i < nunit && ok; ++i) {
                    walk_to(tb, wk, i, c);
                    if (c.d != d_seen) ok = layer(c);
                    if (!ok) break;
                    if (c_count >= ring && !wait_bar(c_eb, c_phase, s_fail, limit_us)) {
                        atomicOr(&g_batch_status, 2u);
                        *s_fail = 1;
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(c_fb, kBatchCodesBytes + kXBytes);
                    if (walk_unit(wk, i) != tb.fault_unit) tma_load_codes(c_slot, map, c.s * (kBatchStageK / 2), c.t * kBatchTileRows, c_fb);
                    bulk_load(c_slot + kBatchCodesBytes + kBatchSfBytes, MXQ_AT(img + (uint32_t)c.s * kXBytes, kXBytes, tb.ws, tb.ws_bytes), kXBytes, c_fb);
                    ++issued;
                    c_slot += kSlot;
                    c_fb += 8u;
                    c_eb += 8u;
                    if (c_slot == ring_end) {
                        c_slot = base;
                        c_fb = full0;
                        c_eb = empty0;
                        if (c_count >= ring) c_phase ^= 1u;
                    }
                    ++c_count;
                    o_slot = c_slot;
                    o_fb = c_fb;
                }
            }
            if (!ok || *s_fail) {
                // Copies this lane requested may still be in flight, and the CTA must not end before they have landed:
                // the barriers of complete requests are waited for, the rest is given time.
                for (int i = max(0, issued - ring); i < issued; ++i)
                    (void)wait_bar(full0 + (uint32_t)(i % ring) * 8u, (uint32_t)((i / ring) & 1), s_zero, 1000u);
                (void)c_count;
                const uint64_t t0 = global_ns();
                while (global_ns() - t0 < 100000ull) __nanosleep(1000);
            }
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ---- scale warps: warp w brings the scale bytes of units w, w + 4, w + 8, ... of the walk into the slots' scale atoms
        // (8 bytes per weight row and unit, rows K / 32 bytes apart).  Lane l takes rows l, l + 32, l + 64, l + 96, whose
        // bytes are neighbours in an atom: two 16-byte shared stores per lane and unit.  The loads of a warp's next unit
        // are in flight in registers while it waits for the slot of the current one.
        // (At most `ring` warps take part: a warp's consecutive units must be no more than a ring apart, or its parity wait
        // for the slot's release could be answered by the release before that one.)
        const int sw = warp - 6;   // 0..3
        const int nsw = ring < 4 ? ring : 4;
        uint32_t rows_lo[4], rows_hi[4];
        Walk wk;
        // (the cursor is carried from one of this warp's units to the next: no search, no division per unit)
        Cursor c;
        int c_at = -1;   // element of the current group's walk the cursor stands at (-1: nowhere yet)
        auto load = [&](int i, uint32_t (&lo)[4], uint32_t (&hi)[4]) {   // element i of the current group's walk, i > c_at
            if (c_at < 0) {
                walk_begin(tb, wk, c);
                c_at = 0;
            }
            while (c_at < i) walk_to(tb, wk, ++c_at, c);
            const BatchDesc &ds = tb.desc[c.d];
            const int kb_row = ds.K >> 5;
            const bool wide = (ds.K & (kBatchStageK - 1)) == 0;   // a unit's 8 bytes are one aligned load
            const bool second = wide || c.s != c.ks - 1;
            const int n0 = c.t * kBatchTileRows + lane;
            const uint8_t *src = ds.scales + (int64_t)n0 * kb_row + c.s * 8;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                lo[q] = hi[q] = 0u;
                if (n0 + 32 * q < ds.N) {
                    if (wide) {
                        asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(lo[q]), "=r"(hi[q]) : "l"(MXQ_AT(src, 8, ds.scales, (int64_t)ds.N * kb_row)));
                    } else {
                        asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(lo[q]) : "l"(MXQ_AT(src, 4, ds.scales, (int64_t)ds.N * kb_row)));
                        if (second) asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(hi[q]) : "l"(MXQ_AT(src + 4, 4, ds.scales, (int64_t)ds.N * kb_row)));
                    }
                }
                src += (int64_t)32 * kb_row;
            }
        };
        // The CTA's units are numbered through all groups; unit e goes to slot e % ring, and this warp takes the units
        // e = sw (mod nsw): the slot index advances by nsw (mod ring) from one unit of this warp to the next.
        const uint32_t step = (uint32_t)nsw % (uint32_t)ring, carry = (uint32_t)nsw / (uint32_t)ring;
        int ebase = 0;   // units of the groups before this one
        bool alive = sw < nsw;
        for (int g = 0; g < ngroups && alive; ++g) {
        group_walk(g, wk);
        c_at = -1;
        const int nunit = wk.nunit;
        // first unit of this group that is this warp's: the smallest i >= 0 with (ebase + i) % nsw == sw
        const int i0 = (sw - ebase % nsw + nsw) % nsw;
        uint32_t slot = (uint32_t)((ebase + i0) % ring), round = (uint32_t)((ebase + i0) / ring);
        ebase += nunit;
        if (i0 < nunit) load(i0, rows_lo, rows_hi);
        for (int i = i0; i < nunit; i += nsw) {
            uint32_t cur_lo[4], cur_hi[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                cur_lo[q] = rows_lo[q];
                cur_hi[q] = rows_hi[q];
            }
            if (i + nsw < nunit) load(i + nsw, rows_lo, rows_hi);
            if (round != 0 && !warp_wait_bar(empty0 + slot * 8u, (round - 1u) & 1u, s_fail, limit_us, lane)) {
                if (lane == 0) {
                    atomicOr(&g_batch_status, 2u);
                    *s_fail = 1;
                }
                alive = false;
                break;
            }
            const uint32_t sf = base + slot * kSlot + kBatchCodesBytes + (uint32_t)lane * 16u;
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(sf), "r"(cur_lo[0]), "r"(cur_lo[1]), "r"(cur_lo[2]), "r"(cur_lo[3]) : "memory");
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(sf + 512u), "r"(cur_hi[0]), "r"(cur_hi[1]), "r"(cur_hi[2]), "r"(cur_hi[3]) : "memory");
            fence_async_proxy();   // ordinary stores, read by tcgen05.cp
            __syncwarp();
            if (lane == 0) mbar_arrive(full0 + slot * 8u);
            slot += step;
            round += carry;
            if (slot >= (uint32_t)ring) {
                slot -= (uint32_t)ring;
                ++round;
            }
        }
        }
    } else {
        // ---- split / epilogue warps -----------------------------------------------------------------------------------
        const int ew = warp - 2;                          // 0..3
        const int et = tid - 64;                          // 0..127
        const int row = ((warp & 3) << 5) + lane;         // accumulator row this thread may read (its warp's quarter)

        // Everything between the wait above and the first MMA is paid by every launch in full, so the first task of the
        // rewriting is asked for before anything else.
        uint32_t first_task = 0;
        if (lane == 0) first_task = atomicAdd(hdr + kBatchWordTask, 1u);
        uint64_t seen_mask = 0, bad_mask = 0, fix_mask = 0;
        float *partials = reinterpret_cast<float *>(tb.ws + tb.partials_offset);
        uint32_t *g_ticket = hdr + kBatchWordTicket, *g_done = hdr + kBatchWordDone;
        const float nanv = __uint_as_float(0x7FC00000u);
        int seg = 0;
        if (units_left == 0) asm volatile("bar.arrive 2, 160;" ::: "memory");
        for (int g = 0; g < ngroups; ++g) {
        Walk wk;
        group_walk(g, wk);
        const int nunit = wk.nunit;
        const int gu = tb.group_unit[g], ug = tb.group_unit[g + 1] - gu, gg = ug < G ? ug : G;
        // 0. a later group reads what the groups before it wrote: all their tiles must have been stored
        if (g > 0) {
            if (et == 0 && !*s_fail && !wait_counter(g_done + (g - 1) * kBatchCounterStride, (uint32_t)tb.group_tiles[g - 1], s_fail, limit_us)) {
                atomicOr(&g_batch_status, 8u);
                *s_fail = 1;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        // 1. the rewriting of the group's token rows: task = 128 k of one token row of one image.  Tasks are handed out by a
        //    counter in the workspace, not by CTA index: every consumer waits for whole images, so a CTA that starts late
        //    (CTAs start over several microseconds as the previous kernel's leave) must not be holding tasks.
        for (bool first = g == 0;; first = false) {
            int task = 0;
            if (lane == 0) task = tb.group_task[g] + (int)(first ? first_task : atomicAdd(hdr + kBatchWordTask + g * kBatchCounterStride, 1u));
            task = __shfl_sync(0xffffffffu, task, 0);
            if (task >= tb.group_task[g + 1]) break;
            int im = 0;
            while (im + 1 < tb.nimg && task >= tb.img[im + 1].task_base) ++im;
            const BatchImg &gi = tb.img[im];
            const int local = task - gi.task_base;
            const int k128 = local / M, m = local - k128 * M;
            const int kk = k128 * 128 + (lane >> 1) * 8;
            const uint4 raw = ld_cg_u4(MXQ_AT(reinterpret_cast<const __nv_bfloat16 *>(gi.X) + (int64_t)m * gi.K + kk, 16, gi.X, (int64_t)M * gi.K * 2));
            uint8_t *stage = tb.ws + gi.offset + (size_t)(kk >> 8) * kXBytes;
            bool inexact = split_half_unit_to(raw, m, (uint32_t)kk & 255u, lane & 1, lane, SplitToGlobal{stage, tb.ws, tb.ws_bytes},
                                              SplitToGlobal{stage + (uint32_t)NB * 128u, tb.ws, tb.ws_bytes});
            if (__any_sync(0xffffffffu, inexact)) {
                // (rare, and kept off the common path, whose length every launch pays for: the rewriting is done again,
                // this time asking for what the planes cannot hold)
                float rem[8];
                inexact = split_half_unit_to(raw, m, (uint32_t)kk & 255u, lane & 1, lane, SplitToGlobal{stage, tb.ws, tb.ws_bytes},
                                             SplitToGlobal{stage + (uint32_t)NB * 128u, tb.ws, tb.ws_bytes}, rem);
                // Elements that do not fit the block's fixed point (more than 24 binades under the block's maximum; any
                // element of a block with an Inf or a NaN): the planes hold them truncated, and what is missing goes on the
                // image's list of corrections (token row, k, remainder), which the epilogues add as remainder * weight.  A
                // list that overflows flags the image; its layers are then computed by the scalar path.
                if (inexact && (lane & 1) == 0) {
                    BatchFix *fixes = reinterpret_cast<BatchFix *>(tb.ws + tb.fix_offset) + (size_t)im * kBatchMaxFixes;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (rem[e] != 0.f) {   // (NaN included)
                            const uint32_t at = atomicAdd(g_bad + im * kBatchCounterStride + 1, 1u);
                            if (at < (uint32_t)kBatchMaxFixes) {
                                BatchFix *fx = MXQ_AT(fixes + at, sizeof(BatchFix), tb.ws, tb.ws_bytes);
                                fx->m = m;
                                fx->k = kk + e;
                                fx->rem = rem[e];
                            } else {
                                atomicOr(g_bad + im * kBatchCounterStride, 1u);
                            }
                        }
                }
            }
            __syncwarp();   // (orders the lanes' stores before lane 0's release; the readers order them against their bulk copies)
            if (lane == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(g_ready + im * kBatchCounterStride) : "memory");
        }

        // 2. epilogues: one per piece of a tile in this CTA's walk of the group, in order
        for (int i = 0; i < nunit; ++seg) {
            Cursor c;
            const int u = walk_unit(wk, i);
            cursor_at(tb, u, c);
            const BatchDesc &ds = tb.desc[c.d];
            const int len = min(c.ks - c.s, (i < wk.tail ? wk.tail : nunit) - i);
            const int s_begin = c.s, s_end = c.s + len;
            const int a = seg % A;
            i += len;
            units_left -= len;
            const bool last_seg = units_left == 0;
            // has this layer's X been rewritten exactly?  (the counter is complete by now; waiting for it here makes the
            // flag's value certain)
            const int im = ds.img;
            if (!((seen_mask >> im) & 1ull)) {
                uint32_t b = 0;
                if (lane == 0) {
                    if (!wait_counter(g_ready + im * kBatchCounterStride, (uint32_t)tb.img[im].ntasks, s_fail, limit_us)) {
                        atomicOr(&g_batch_status, 8u);
                        *s_fail = 1;
                    }
                    b = *reinterpret_cast<volatile uint32_t *>(g_bad + im * kBatchCounterStride);
                    if (*reinterpret_cast<volatile uint32_t *>(g_bad + im * kBatchCounterStride + 1) != 0u) b |= 2u;
                }
                b = __shfl_sync(0xffffffffu, b, 0);
                seen_mask |= 1ull << im;
                if (b & 1u) bad_mask |= 1ull << im;
                if (b & 2u) fix_mask |= 1ull << im;
            }
            const bool bad = (bad_mask >> im) & 1ull;

            float yt[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) yt[m] = 0.f;
            // one thread probes for all four epilogue warps; barrier 1 passes the result on
            if (et == 0 && !*s_fail && !wait_bar(accf0 + (uint32_t)a * 8u, (uint32_t)((seg / A) & 1), s_fail, limit_us)) {
                atomicOr(&g_batch_status, 4u);
                *s_fail = 1;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            const bool got = !*s_fail;
            if (got) {
                tc_fence_after();
                const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(a * NB);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    float d[16];
                    tc_load16(t_row + m * 16, d);
                    float acc = d[15];
#pragma unroll
                    for (int p = 14; p >= 0; --p) acc += d[p];
                    yt[m] = acc;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acce0 + (uint32_t)a * 8u);
            }
            if (last_seg) asm volatile("bar.arrive 2, 160;" ::: "memory");   // tensor memory may go back
            const int n = c.t * kBatchTileRows + row;
            if (bad && got) {
                // Scalar path for a K range whose X cannot be rewritten exactly (the MMA results are ignored).
                float acc[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) acc[m] = 0.f;
                if (n < ds.N) {
                    const int kb_row = ds.K >> 5;
                    const uint4 *crow = reinterpret_cast<const uint4 *>(ds.codes + (int64_t)n * (ds.K / 2));
                    const uint8_t *srw = ds.scales + (int64_t)n * kb_row;
                    const __nv_bfloat16 *X = reinterpret_cast<const __nv_bfloat16 *>(ds.X);
                    const int blk_end = min(s_end * 8, kb_row);
                    for (int blk = s_begin * 8; blk < blk_end; ++blk) {
                        const uint4 cc = ld_stream_u4(MXQ_AT(crow + blk, 16, ds.codes, (int64_t)ds.N * (ds.K / 2)));
                        const float sc = e8m0_to_float(*MXQ_AT(srw + blk, 1, ds.scales, (int64_t)ds.N * kb_row)) * kGuardDown;
                        const uint32_t w[4] = {cc.x, cc.y, cc.z, cc.w};
                        float part[MT];
#pragma unroll
                        for (int m = 0; m < MT; ++m) part[m] = 0.f;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 wv = __half22float2(e2m1x2_to_half2((w[q] >> (8 * e)) & 0xFFu));
                                const int64_t k = (int64_t)blk * 32 + q * 8 + e * 2;
#pragma unroll
                                for (int m = 0; m < MT; ++m)
                                    if (m < M) {
                                        uint32_t xb;
                                        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(xb) : "l"(MXQ_AT(X + (int64_t)m * ds.K + k, 4, ds.X, (int64_t)M * ds.K * 2)) : "memory");
                                        part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                                        part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                                    }
                            }
#pragma unroll
                        for (int m = 0; m < MT; ++m) acc[m] = fmaf(part[m], sc, acc[m]);
                    }
                }
#pragma unroll
                for (int m = 0; m < MT; ++m) yt[m] = acc[m];
            }
            if (!got) {
#pragma unroll
                for (int m = 0; m < MT; ++m) yt[m] = nanv;
            }

            bool finish = true;   // whether this CTA stores the tile
            if (s_begin != 0 || s_end != c.ks) {
                // The tile is shared with the neighbouring ranges: deliver this part, and finish the tile if it was the last.
                const int64_t ta = (int64_t)ds.unit_base + (int64_t)c.t * c.ks, tz = ta + c.ks - 1;
                const int c_first = (int)batch_owner(ta - gu, ug, gg), c_last = (int)batch_owner(tz - gu, ug, gg);
                const int ncontrib = c_last - c_first + 1;
                const bool head = u == wk.u0;   // the piece that opens this CTA's range
                float *mine = partials + ((size_t)(cta * 2 + (head ? 0 : 1)) * MT) * 128u;
#pragma unroll
                for (int m = 0; m < MT; ++m)
                    if (m < M) *MXQ_AT(mine + m * 128 + row, 4, tb.ws, tb.ws_bytes) = yt[m];
                // The barrier orders the 128 threads' stores before thread 0's ticket, whose release (cumulative, GPU scope)
                // publishes them; its acquire, passed on through the next barrier, lets a finisher read the other parts.
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (et == 0) {
                    uint32_t old;
                    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(MXQ_AT(g_ticket + c_first, 4, tb.ws, kBatchHeaderBytes)) : "memory");
                    *s_flag = (int)old;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                finish = *s_flag == ncontrib - 1;
                asm volatile("bar.sync 1, 128;" ::: "memory");   // (s_flag may be rewritten by the next piece)
                if (finish) {
                    float sum[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) sum[m] = 0.f;
                    for (int j = 0; j < ncontrib; ++j) {   // range order, whoever finishes
                        const int cj = c_first + j;
                        const bool hj = j > 0 || gu + batch_range_lo(cj, ug, gg) == ta;
                        const float *part = partials + ((size_t)(cj * 2 + (hj ? 0 : 1)) * MT) * 128u;
#pragma unroll
                        for (int m = 0; m < MT; ++m)
                            if (m < M) sum[m] += ld_cg_f32(MXQ_AT(part + m * 128 + row, 4, tb.ws, tb.ws_bytes));
                    }
#pragma unroll
                    for (int m = 0; m < MT; ++m) yt[m] = sum[m];
                    if (et == 0) g_ticket[c_first] = 0u;   // every contributor has delivered: ready for the next call
                }
            }
            if (finish) {
                // finished sums of weight row n, one per token row: restore the guard factor, apply the layer's epilogue, store
#pragma unroll
                for (int m = 0; m < MT; ++m) yt[m] *= kGuardUp;
                if (((fix_mask >> im) & 1ull) && !bad && n < ds.N) {
                    // what the planes of this layer's X could not hold: remainder * weight, element by element
                    const BatchFix *fixes = reinterpret_cast<const BatchFix *>(tb.ws + tb.fix_offset) + (size_t)im * kBatchMaxFixes;
                    const uint32_t nfix = min(*reinterpret_cast<volatile uint32_t *>(g_bad + im * kBatchCounterStride + 1), (uint32_t)kBatchMaxFixes);
                    for (uint32_t e = 0; e < nfix; ++e) {
                        const uint4 fx = ld_cg_u4(MXQ_AT(fixes + e, 16, tb.ws, tb.ws_bytes));   // (written by another SM during this kernel: through L2)
                        const int fm = (int)fx.x, fk = (int)fx.y;
                        const uint32_t byte = *MXQ_AT(ds.codes + (int64_t)n * (ds.K / 2) + (fk >> 1), 1, ds.codes, (int64_t)ds.N * (ds.K / 2));
                        const float2 wv = __half22float2(e2m1x2_to_half2(byte));
                        const float wgt = ((fk & 1) ? wv.y : wv.x) * e8m0_to_float(*MXQ_AT(ds.scales + (int64_t)n * (ds.K >> 5) + (fk >> 5), 1, ds.scales, (int64_t)ds.N * (ds.K >> 5)));
                        const float add = __uint_as_float(fx.z) * wgt;
#pragma unroll
                        for (int m = 0; m < MT; ++m)
                            if (m == fm) yt[m] += add;
                    }
                }
                if (ds.epi == 2) {
                    // gate / up rows interleaved: the partner row's sums sit in the neighbouring lane
                    float y[MT];
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const float up = __shfl_xor_sync(0xffffffffu, yt[m], 1);
                        y[m] = yt[m] / (1.f + expf(-yt[m])) * up;
                    }
                    if (n < ds.N && (n & 1) == 0) {
#pragma unroll
                        for (int m = 0; m < MT; ++m)
                            if (m < M) store_out(ds.Y, ds.y_dtype, (int64_t)m * (ds.N >> 1) + (n >> 1), y[m], (int64_t)M * (ds.N >> 1));
                    }
                } else if (n < ds.N) {
#pragma unroll
                    for (int m = 0; m < MT; ++m)
                        if (m < M) {
                            const int64_t at = (int64_t)m * ds.N + n;
                            // (through L2: in a call of several groups another SM may have written the residual during this kernel)
                            const float r = ds.epi == 1 ? load_in_cg(ds.residual, ds.y_dtype, at, (int64_t)M * ds.N) : 0.f;
                            store_out(ds.Y, ds.y_dtype, at, yt[m] + r, (int64_t)M * ds.N);
                        }
                }
                if (ngroups > 1) {
                    // the tile is stored: one more of this group's tiles that the next group may read (barrier, then one
                    // thread's cumulative release)
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (et == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(g_done + g * kBatchCounterStride) : "memory");
                }
            }
        }
        }

        // 3. the last CTA to get here leaves the counters zero for the next call
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) {
            const uint32_t old = atomicAdd(hdr + kBatchWordExit, 1u);
            if (old == (uint32_t)G - 1u) {
                __threadfence();
                for (int i = 0; i < tb.nimg; ++i) {
                    g_ready[i * kBatchCounterStride] = 0u;
                    g_bad[i * kBatchCounterStride] = 0u;
                    g_bad[i * kBatchCounterStride + 1] = 0u;
                }
                for (int i = 0; i < ngroups; ++i) {
                    hdr[kBatchWordTask + i * kBatchCounterStride] = 0u;
                    g_done[i * kBatchCounterStride] = 0u;
                }
                hdr[kBatchWordExit] = 0u;
            }
        }
    }
}

template <int NB, bool GROUPS>
cudaError_t launch_batch(const BatchTable &tb, int grid, uint32_t smem, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_batch_kernel<NB, GROUPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBatchSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(linear_batch_kernel<NB, GROUPS>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kBatchThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, linear_batch_kernel<NB, GROUPS>, tb);
}

// test hook (mxq_debug_batch_fault): consumed by the next launch
std::atomic<int> g_fault_unit{-1};
std::atomic<unsigned> g_fault_wait_us{0};

struct BatchLayout {
    int nb, ring, grid, per_sm;
    uint32_t smem;
};

// ring slots and CTAs for `units` units of work
// `units`: units of work of the call's largest group
bool batch_layout(int M, int64_t units, BatchLayout &L) {
    const LayoutOverride o = layout_override();
    L.nb = batch_nb(M);
    // Two CTAs per SM by default: what a CTA's single MMA-issuing, single requesting and single probing threads do per
    // unit bounds one CTA at about two units per microsecond, and a second CTA's streams fill the gaps (7B layer sets at
    // M = 1, four per call: 25.5 us per layer set with one CTA per SM and a ring of 5, 21.1 us with two).
    const int per_sm = o.batch_ctas_per_sm >= 1 && o.batch_ctas_per_sm <= 2 ? o.batch_ctas_per_sm : 2;
    int ring = o.batch_ring > 0 ? o.batch_ring : 64;
    // the deepest ring that lets `per_sm` CTAs share an SM's shared memory (each CTA also takes 1 KB of system use)
    while (ring > 1 && (batch_smem_bytes(L.nb, ring) + 1024u) * (uint32_t)per_sm > 228u * 1024u) --ring;
    if (batch_smem_bytes(L.nb, ring) > kBatchSmemLimit) return false;
    if (batch_acc_slots(L.nb, per_sm) < 1) return false;
    L.per_sm = per_sm;
    L.ring = ring;
    int64_t grid = (int64_t)sm_count() * per_sm;
    if (grid > units) grid = units;
    if (grid > kBatchMaxGrid) grid = kBatchMaxGrid;
    L.grid = (int)grid;
    L.smem = batch_smem_bytes(L.nb, ring);
    return true;
}

}  // namespace

int linear_batch_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_batch_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_batch_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

// whether the persistent kernel covers the call
static bool batch_covered(const mxq_linear_desc *descs, int count, int M) {
    if (!linear_umma_available() || M > kBatchMaxM || count > kBatchMaxDescs) return false;
    int64_t units = 0;
    for (int i = 0; i < count; ++i) {
        const mxq_linear_desc &d = descs[i];
        if (d.K < 128 || (d.K % 128) != 0 || d.K > 0x3FFFFFFF || d.N > 0x7FFFFF00) return false;
        units += ((d.N + 127) / 128) * ((d.K + 255) / 256);
    }
    return units < 0x40000000;
}

// 9..16 token rows: the rows of a linear layer are independent of one another (row m of Y needs row m of X and of the
// residual only), so the call runs as two passes of the persistent kernel, rows [0, 8) and [8, M).  The weights are
// streamed twice, which still costs far less than a launch per layer.
static bool batch_two_passes(const mxq_linear_desc *descs, int count, int M) {
    return M > kBatchMaxM && M <= 2 * kBatchMaxM && batch_covered(descs, count, kBatchMaxM);
}

static size_t batch_workspace_bytes(const mxq_linear_desc *descs, int count, int M) {
    const int nb = batch_nb(M);
    size_t b = kBatchHeaderBytes + batch_partials_bytes(kBatchMaxGrid, nb);
    for (int i = 0; i < count; ++i) b += (size_t)((descs[i].K + 255) / 256) * batch_image_stage_bytes(nb);
    b = (b + 255u) & ~(size_t)255u;
    b += (size_t)count * kBatchMaxFixes * sizeof(BatchFix);   // corrections: one list per image, at most one image per layer
    return (b + 255u) & ~(size_t)255u;
}

MXQ_BOUNDS_TU(bounds_take_linear_batch)

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)

static int batch_validate(const mxq_linear_desc *descs, int count, int M) {
    if (!descs) return MXQ_ERR_NULL;
    if (count < 1 || count > MXQ_MAX_BATCH || M < 1 || M > MXQ_MAX_M) return MXQ_ERR_SHAPE;
    int groups = 1;
    for (int i = 0; i < count; ++i) {
        const mxq_linear_desc &d = descs[i];
        if (!d.X_bf16 || !d.codes || !d.scales || !d.Y) return MXQ_ERR_NULL;
        if ((d.flags & ~MXQ_BATCH_DEPENDS) != 0 || d.reserved != 0) return MXQ_ERR_SHAPE;
        if (i > 0 && (d.flags & MXQ_BATCH_DEPENDS) && ++groups > MXQ_MAX_BATCH_GROUPS) return MXQ_ERR_SHAPE;
        if (d.epilogue < MXQ_EPI_NONE || d.epilogue > MXQ_EPI_SWIGLU) return MXQ_ERR_SHAPE;
        if (d.epilogue == MXQ_EPI_RESIDUAL && !d.residual) return MXQ_ERR_NULL;
        if (!mxq::shape_ok(d.N, d.K) || (d.epilogue == MXQ_EPI_SWIGLU && (d.N & 1))) return MXQ_ERR_SHAPE;
        if (d.y_dtype != MXQ_F32 && d.y_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
        if (!mxq::aligned16(d.X_bf16) || !mxq::aligned16(d.codes) || !mxq::aligned16(d.scales) || !mxq::aligned16(d.Y) ||
            (d.residual && !mxq::aligned16(d.residual)))
            return MXQ_ERR_ALIGN;
    }
    return MXQ_OK;
}

size_t mxq_linear_batch_workspace_bytes(const mxq_linear_desc *descs, int count, int M) {
    if (batch_validate(descs, count, M) != MXQ_OK) return 0;
    size_t b = mxq::kBatchHeaderBytes;
    if (mxq::batch_covered(descs, count, M)) b = mxq::batch_workspace_bytes(descs, count, M);
    else if (mxq::batch_two_passes(descs, count, M)) {   // what the larger of the two passes asks for
        const size_t first = mxq_linear_batch_workspace_bytes(descs, count, mxq::kBatchMaxM);
        const size_t second = mxq_linear_batch_workspace_bytes(descs, count, M - mxq::kBatchMaxM);
        return first > second ? first : second;
    }
    // where the persistent kernel does not cover the call the layers run one by one and share this much scratch
    size_t one = 0;
    for (int i = 0; i < count; ++i) {
        const size_t w = mxq_linear_fused_workspace_bytes(M, descs[i].N, descs[i].K);
        if (w > one) one = w;
    }
    return b + ((one + 255u) & ~(size_t)255u);
}

int mxq_debug_batch_fault(int unit, unsigned wait_us) {
    mxq::g_fault_unit.store(unit, std::memory_order_relaxed);
    mxq::g_fault_wait_us.store(wait_us, std::memory_order_relaxed);
    return MXQ_OK;
}

int mxq_linear_batch_info(const mxq_linear_desc *descs, int count, int M, int32_t *info) {
    if (!info) return MXQ_ERR_NULL;
    const int rc = batch_validate(descs, count, M);
    if (rc != MXQ_OK) return rc;
    for (int i = 0; i < 8; ++i) info[i] = 0;
    if (mxq::batch_two_passes(descs, count, M)) {   // described by its first pass (8 token rows)
        const int rc2 = mxq_linear_batch_info(descs, count, mxq::kBatchMaxM, info);
        if (rc2 == MXQ_OK && info[0] == 1) info[0] = 2;
        return rc2;
    }
    if (!mxq::batch_covered(descs, count, M)) return MXQ_OK;
    int64_t units = 0, total = 0, cur = 0;
    for (int i = 0; i < count; ++i) {
        if (i > 0 && (descs[i].flags & MXQ_BATCH_DEPENDS)) cur = 0;
        const int64_t u = ((descs[i].N + 127) / 128) * ((descs[i].K + 255) / 256);
        cur += u;
        total += u;
        if (cur > units) units = cur;
    }
    mxq::BatchLayout L;
    if (!mxq::batch_layout(M, units, L)) return MXQ_OK;
    info[0] = 1;
    info[1] = L.grid;
    info[2] = L.ring;
    info[3] = (int32_t)L.smem;
    info[4] = L.nb;
    info[5] = (int32_t)total;
    info[6] = mxq::batch_tmem_cols(L.nb, L.per_sm);
    info[7] = mxq::batch_acc_slots(L.nb, L.per_sm);
    return MXQ_OK;
}

int mxq_linear_batch(const mxq_linear_desc *descs, int count, int M, void *workspace, size_t workspace_bytes, void *stream) {
    int rc = batch_validate(descs, count, M);
    if (rc != MXQ_OK) return rc;
    if (!workspace) return MXQ_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MXQ_ERR_ALIGN;
    const size_t ws_needed = mxq_linear_batch_workspace_bytes(descs, count, M);
    if (workspace_bytes < ws_needed) return MXQ_ERR_WORKSPACE;
    if (mxq::batch_two_passes(descs, count, M)) {
        mxq_linear_desc part[MXQ_MAX_BATCH];
        for (int row0 = 0; row0 < M; row0 += mxq::kBatchMaxM) {
            const int rows = M - row0 < mxq::kBatchMaxM ? M - row0 : mxq::kBatchMaxM;
            for (int i = 0; i < count; ++i) {
                part[i] = descs[i];
                const size_t ysz = descs[i].y_dtype == MXQ_F32 ? 4 : 2;
                const int64_t ncol = descs[i].epilogue == MXQ_EPI_SWIGLU ? descs[i].N / 2 : descs[i].N;
                part[i].X_bf16 = static_cast<const uint8_t *>(descs[i].X_bf16) + (size_t)row0 * descs[i].K * 2;
                part[i].Y = static_cast<uint8_t *>(descs[i].Y) + (size_t)row0 * ncol * ysz;
                if (descs[i].residual) part[i].residual = static_cast<const uint8_t *>(descs[i].residual) + (size_t)row0 * ncol * ysz;
            }
            rc = mxq_linear_batch(part, count, rows, workspace, workspace_bytes, stream);
            if (rc != MXQ_OK) return rc;
        }
        return MXQ_OK;
    }
    cudaStream_t st = (cudaStream_t)stream;
    mxq::BatchLayout L;
    int64_t units = 0, cur = 0;   // units of the largest group
    for (int i = 0; i < count; ++i) {
        if (i > 0 && (descs[i].flags & MXQ_BATCH_DEPENDS)) cur = 0;
        cur += ((descs[i].N + 127) / 128) * ((descs[i].K + 255) / 256);
        if (cur > units) units = cur;
    }
    if (!mxq::batch_covered(descs, count, M) || !mxq::batch_layout(M, units, L)) {
        // one layer after the other through the ordinary entry points, sharing the scratch behind the header
        uint8_t *ws = static_cast<uint8_t *>(workspace) + mxq::kBatchHeaderBytes;
        const size_t ws_bytes = workspace_bytes - mxq::kBatchHeaderBytes;
        for (int i = 0; i < count; ++i) {
            const mxq_linear_desc &d = descs[i];
            rc = d.epilogue == MXQ_EPI_RESIDUAL ? mxq_linear_residual(d.X_bf16, M, d.codes, d.scales, d.N, d.K, d.residual, d.Y, d.y_dtype, ws, ws_bytes, stream)
                 : d.epilogue == MXQ_EPI_SWIGLU ? mxq_linear_swiglu(d.X_bf16, M, d.codes, d.scales, d.N, d.K, d.Y, d.y_dtype, ws, ws_bytes, stream)
                                                : mxq_linear(d.X_bf16, M, d.codes, d.scales, d.N, d.K, d.Y, d.y_dtype, ws, ws_bytes, stream);
            if (rc != MXQ_OK) return rc;
        }
        return MXQ_OK;
    }
    mxq::BatchTable tb;
    std::memset(&tb, 0, sizeof tb);
    const int nb = L.nb;
    tb.ws = static_cast<uint8_t *>(workspace);
    tb.ws_bytes = ws_needed;   // (what this call may touch, however large the caller's buffer)
    tb.ndesc = count;
    tb.M = M;
    tb.ring = L.ring;
    tb.tmem_cols = mxq::batch_tmem_cols(nb, L.per_sm);
    tb.acc_slots = mxq::batch_acc_slots(nb, L.per_sm);
    tb.partials_offset = (uint32_t)mxq::kBatchHeaderBytes;
    size_t img_off = mxq::kBatchHeaderBytes + mxq::batch_partials_bytes(mxq::kBatchMaxGrid, nb);
    int unit_base = 0, task_base = 0, nimg = 0, ngroups = 0, group_img0 = 0;
    for (int i = 0; i < count; ++i) {
        const mxq_linear_desc &d = descs[i];
        mxq::BatchDesc &o = tb.desc[i];
        if (i == 0 || (d.flags & MXQ_BATCH_DEPENDS)) {   // a new group: its layers may read what the layers before wrote
            tb.group_unit[ngroups] = unit_base;
            tb.group_task[ngroups] = task_base;
            tb.group_tiles[ngroups] = 0;
            group_img0 = nimg;
            ++ngroups;
        }
        if (!mxq::codes_tensor_map(d.codes, d.N, d.K, /*expand_fp4=*/false, &tb.maps[i])) return MXQ_ERR_CUDA;
        o.codes = d.codes;
        o.scales = d.scales;
        o.X = d.X_bf16;
        o.Y = d.Y;
        o.residual = d.residual;
        o.N = (int32_t)d.N;
        o.K = (int32_t)d.K;
        o.ks = (int32_t)((d.K + 255) / 256);
        o.tiles = (int32_t)((d.N + 127) / 128);
        o.unit_base = unit_base;
        o.y_dtype = d.y_dtype;
        o.epi = d.epilogue;
        unit_base += o.ks * o.tiles;
        tb.group_tiles[ngroups - 1] += o.tiles;
        // layers of a group that read the same X share one image
        int im = -1;
        for (int j = group_img0; j < nimg; ++j)
            if (tb.img[j].X == d.X_bf16 && tb.img[j].K == o.K) im = j;
        if (im < 0) {
            im = nimg++;
            mxq::BatchImg &g = tb.img[im];
            g.X = d.X_bf16;
            g.K = o.K;
            g.ks = o.ks;
            g.task_base = task_base;
            g.ntasks = M * (o.K / 128);
            g.offset = (uint32_t)img_off;
            task_base += g.ntasks;
            img_off += (size_t)o.ks * mxq::batch_image_stage_bytes(nb);
        }
        o.img = im;
    }
    tb.fix_offset = (uint32_t)((img_off + 255u) & ~(size_t)255u);
    tb.nimg = nimg;
    tb.units = unit_base;
    tb.tasks = task_base;
    tb.ngroups = ngroups;
    tb.group_unit[ngroups] = unit_base;
    tb.group_task[ngroups] = task_base;
    tb.fault_unit = mxq::g_fault_unit.exchange(-1, std::memory_order_relaxed);
    const unsigned w = mxq::g_fault_wait_us.exchange(0, std::memory_order_relaxed);
    tb.wait_us = w ? w : 1000000u;
    // (a call of one group runs the kernel compiled without the loops over groups: measured 2 us per launch faster at
    // one 7B layer set per call, equal at four)
    const cudaError_t e = ngroups > 1 ? (nb == 16 ? mxq::launch_batch<16, true>(tb, L.grid, L.smem, st)
                                         : nb == 32 ? mxq::launch_batch<32, true>(tb, L.grid, L.smem, st)
                                         : nb == 64 ? mxq::launch_batch<64, true>(tb, L.grid, L.smem, st)
                                                    : mxq::launch_batch<128, true>(tb, L.grid, L.smem, st))
                                      : (nb == 16 ? mxq::launch_batch<16, false>(tb, L.grid, L.smem, st)
                                         : nb == 32 ? mxq::launch_batch<32, false>(tb, L.grid, L.smem, st)
                                         : nb == 64 ? mxq::launch_batch<64, false>(tb, L.grid, L.smem, st)
                                                    : mxq::launch_batch<128, false>(tb, L.grid, L.smem, st));
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return MXQ_ERR_CUDA;
    }
    return mxq::launch_status();
}

#pragma GCC visibility pop
}  // extern "C"
