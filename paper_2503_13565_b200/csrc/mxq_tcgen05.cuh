// Thin wrappers around the sm_100a instructions the tcgen05 mxq_linear kernels share: mbarriers with bounded
// waits, TMA tensor copies, tcgen05 (tensor memory, block-scaled MMA, commit), cluster barriers and
// distributed shared memory.  One instruction (or one short idiom) per function; no policy here.
#pragma once
#include "mxq_host.h"
#include <cuda.h>   // CUtensorMap only

#include "mxq_device.cuh"

namespace mxq {

// ---- small PTX wrappers ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// bounded wait: false after about a second
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) {
    const uint64_t t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > 1000000000ull) return false;
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < 64; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity);
}
// bounded wait for a barrier that is expected to take a while: sleeps between probes, so that a waiting warp does
// not take issue slots from the warps it is waiting for; false after about a second
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 1024; ++i) {
            __nanosleep(40);
            if (mbar_try_wait(bar, parity)) return true;
        }
        if (global_ns() - t0 > 1000000000ull) return false;
    }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_codes(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// a 16-byte global load and a 32-bit shared store that the compiler keeps in program order with each other
__device__ __forceinline__ uint4 ld_ordered_u4(const void *p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_flag(uint32_t saddr, int v) {
    asm volatile("st.volatile.shared::cta.u32 [%0], %1;" ::"r"(saddr), "r"(v) : "memory");
}
// untiled bulk copy global -> shared memory (both 16-byte aligned, size a multiple of 16), counted on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared-memory matrix descriptor: start address, leading / stride byte offsets (all >> 4), version 1, layout
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (uint64_t)((lbo >> 4) & 0x3FFF) << 16 |
           (uint64_t)((sbo >> 4) & 0x3FFF) << 32 | (uint64_t)1 << 46 | (uint64_t)layout << 61;
}
__device__ __forceinline__ void tc_copy_sf(uint32_t tmem, uint32_t atom_saddr) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem), "l"(smem_desc(atom_saddr, 0, 128, 0))
                 : "memory");
}
// the same with the descriptor given as two 32-bit halves (only the low half changes between copies)
__device__ __forceinline__ void tc_copy_sf_lohi(uint32_t tmem, uint32_t desc_lo, uint32_t desc_hi) {
    asm volatile("{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\ttcgen05.cp.cta_group::1.32x128b.warpx4 [%0], d;\n\t}"
                 ::"r"(tmem), "r"(desc_lo), "r"(desc_hi)
                 : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t sfa, uint32_t sfb,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
}
__device__ __forceinline__ void tc_load16(uint32_t taddr, float *v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}
// one lane of a converged warp; the surrounding control flow stays warp-uniform, which lets the compiler keep
// descriptors and barrier addresses in uniform registers (the tcgen05 and TMA instructions take those)
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// split cluster barrier: arrive early, wait late (acquire).  The relaxed arrive orders nothing by itself: what peers
// must see (initialised mbarriers) is published by fence.mbarrier_init.release.cluster before it.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// address of the same shared-memory location in the CTA of rank `rank` of this cluster
__device__ __forceinline__ uint32_t peer_saddr(uint32_t local_saddr, uint32_t rank) {
    uint32_t raddr;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_saddr), "r"(rank));
    return raddr;
}
// 4-byte store into a peer's shared memory that also counts 4 bytes on the peer's mbarrier when it lands
__device__ __forceinline__ void st_async_f32(uint32_t peer_addr, float v, uint32_t peer_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(peer_addr),
                 "r"(__float_as_uint(v)), "r"(peer_bar)
                 : "memory");
}
__device__ __forceinline__ float ld_peer_f32(uint32_t local_saddr, uint32_t rank) {
    uint32_t raddr;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_saddr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(raddr) : "memory");
    return v;
}

// ---- vocabulary projection fused with the greedy verification (Sec. III-A, III-B) ----------------------------------
// With `keys` set a tcgen05 kernel does not store Y: every finished logit (token row m, vocabulary index n) competes
// for keys[m], the last CTA to deliver turns the keys into the verifier's tokens, walks the draft and leaves keys and
// ticket zero for the next call.
constexpr int kFusedKeyStride = 16;   // keys[m] lives at 64-bit word 16 m of the workspace header
constexpr uint32_t kFusedSmemBytes = 16 * 8 + 16 * 4 + 16;   // keys, tokens, "last CTA" flag
// Larger value wins, then the lower index; NaN and -inf never compete (a row of nothing else yields token 0).
__device__ __forceinline__ unsigned long long argmax_key(float v, uint32_t index) {
    if (!(v > -INFINITY)) return 0ull;
    const uint32_t b = __float_as_uint(v + 0.f);   // -0 -> +0: equal values must tie
    const uint32_t u = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    return ((unsigned long long)u << 32) | (uint32_t)~index;
}
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, k, o);
        k = other > k ? other : k;
    }
    return k;
}
// All 128 epilogue threads (named barrier 1), after their candidates are in s_keys (shared memory, [16]).
// R = token rows, grid = CTAs of the launch.
__device__ __forceinline__ void fused_accept_finish(const FusedAccept &fa, unsigned long long *s_keys, int R, uint32_t grid, int ct) {
    int32_t *s_tok = reinterpret_cast<int32_t *>(s_keys + 16);
    volatile int *s_last = reinterpret_cast<volatile int *>(s_tok + 16);
    asm volatile("bar.sync 1, 128;" ::: "memory");
    // (a token row's key has a 128-byte line to itself, and a CTA that cannot raise it does not try: same-address atomics
    // from every SM at once are served one after the other)
    if (ct < R && s_keys[ct] > *reinterpret_cast<volatile unsigned long long *>(fa.keys + ct * kFusedKeyStride))
        atomicMax(fa.keys + ct * kFusedKeyStride, s_keys[ct]);
    __threadfence();
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ct == 0) *s_last = atomicAdd(fa.ticket, 1u) == grid - 1u;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (!*s_last) return;
    __threadfence();
    if (ct < R) {
        const unsigned long long key = atomicExch(fa.keys + ct * kFusedKeyStride, 0ull);   // read and leave zero for the next call
        const int32_t tok = key ? (int32_t)~(uint32_t)key : 0;
        s_tok[ct] = tok;
        if (fa.verifier) fa.verifier[ct] = tok;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ct == 0) {
        int G = 0;
        while (G < fa.T && fa.draft[G] == s_tok[G]) ++G;   // tokens after the first mismatch are dropped (R >= T)
        *fa.accept_len = G;
        *fa.next_token = G < R ? s_tok[G] : -1;
        *fa.ticket = 0u;
    }
}

// (`count`: elements of the array, for the bounds-checked build)
__device__ __forceinline__ void store_out(void *Y, int y_dtype, int64_t idx, float v, int64_t count) {
    (void)count;
    if (y_dtype == MXQ_F32)
        *MXQ_AT(reinterpret_cast<float *>(Y) + idx, 4, Y, count * 4) = v;
    else
        *MXQ_AT(reinterpret_cast<__nv_bfloat16 *>(Y) + idx, 2, Y, count * 2) = __float2bfloat16_rn(v);
}

__device__ __forceinline__ float load_in(const void *R, int dtype, int64_t idx, int64_t count) {
    (void)count;
    // (the residual may be the previous kernel's output)
    return dtype == MXQ_F32 ? ld_dep_f32(MXQ_AT(reinterpret_cast<const float *>(R) + idx, 4, R, count * 4))
                            : ld_dep_bf16(MXQ_AT(reinterpret_cast<const __nv_bfloat16 *>(R) + idx, 2, R, count * 2));
}

// Layer epilogues of the tcgen05 kernels (kEpiLayer): what happens to the finished sums w[m] of weight row n, one per
// token row.  Everything is done for all token rows at once -- all loads, then all arithmetic, then all stores -- so
// that the latencies overlap (one row at a time cost 0.25 us per token row).
// layer_prefetch: the residual values this thread will add (zeros if there is no residual or the thread is inactive).
template <int MT>
__device__ __forceinline__ void layer_prefetch(const FusedAccept &fa, int y_dtype, int M, int64_t n, int64_t N, bool active, float (&r)[MT]) {
#pragma unroll
    for (int m = 0; m < MT; ++m) r[m] = (fa.residual != nullptr && active && m < M) ? load_in(fa.residual, y_dtype, (int64_t)m * N + n, (int64_t)M * N) : 0.f;
}
// layer_emit: called by all 32 lanes of a warp together.  Gate / up pairing: the holder of weight row n ^ 1 is
// `pair_lanes` lanes away; the even row's holder stores silu(gate) * up with silu(g) = g / (1 + e^-g), which goes to -0
// for g -> -inf and to g for g -> +inf.  Residual: Y may be the residual itself (every element is read by the thread
// that writes it, before it writes).
template <int MT>
__device__ __forceinline__ void layer_emit(const FusedAccept &fa, void *Y, int y_dtype, int M, int64_t n, int64_t N, bool active,
                                           const float (&w)[MT], const float (&r)[MT], int pair_lanes) {
    if (fa.swiglu) {
        float y[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float up = __shfl_xor_sync(0xffffffffu, w[m], pair_lanes);
            y[m] = w[m] / (1.f + expf(-w[m])) * up;
        }
        if (active && (n & 1) == 0) {
#pragma unroll
            for (int m = 0; m < MT; ++m)
                if (m < M) store_out(Y, y_dtype, (int64_t)m * (N >> 1) + (n >> 1), y[m], (int64_t)M * (N >> 1));
        }
    } else if (active) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < M) store_out(Y, y_dtype, (int64_t)m * N + n, w[m] + r[m], (int64_t)M * N);
    }
}

// ---- sum over the senders of a power-of-two cluster, as a reduce-scatter over the token rows -------------------------------
// Thread (row r, sender j) of the owner CTA holds sender j's partial sums of all token rows of weight row n; the `split`
// senders of a row sit in neighbouring lanes.  Step s exchanges between lanes j and j ^ 2^s: the lane with bit s clear
// keeps the token rows with bit s clear and gets its partner's values for them, and vice versa.  After log2(split)
// steps lane j holds the finished sums of the token rows m = i * S + (j & (S - 1)), i = 0, 1, .. (S = min(split, P), P =
// token slots rounded up to a power of two): a third of the shuffles of an all-to-all butterfly, and the final stores
// (and the residual loads, and the activation) are spread over the lanes instead of falling to lane j = 0.  Every
// sum is formed by the same tree of additions as in the butterfly (first j ^ 1, then j ^ 2, then j ^ 4), so the
// result is bit-identical whatever the token count.  Where split > P the last steps add whole values and the lanes
// j >= P hold duplicates and stay silent.
template <int MT>
struct TokenScatter {
    static constexpr int P = MT <= 1 ? 1 : (MT <= 2 ? 2 : (MT <= 4 ? 4 : (MT <= 8 ? 8 : 16)));
    static constexpr int PH = P >= 2 ? P / 2 : 1;   // most positions a lane ends up with (split >= 2)
};

// residual values of the positions this lane will finish (zeros where there is nothing to add)
template <int MT>
__device__ __forceinline__ void scatter_prefetch(const FusedAccept &fa, int y_dtype, int M, int split, int j, int64_t n, int64_t N,
                                                 float (&res)[TokenScatter<MT>::PH]) {
    constexpr int P = TokenScatter<MT>::P, PH = TokenScatter<MT>::PH;
    const int S = split < P ? split : P, npos = P / S;
    const bool speaks = j < P && n < N && fa.residual != nullptr;
#pragma unroll
    for (int i = 0; i < PH; ++i) {
        const int m = i * S + (j & (S - 1));
        res[i] = (speaks && i < npos && m < M) ? load_in(fa.residual, y_dtype, (int64_t)m * N + n, (int64_t)M * N) : 0.f;
    }
}

// recv: sender j's partial sums for this thread's row, token row m at recv[m * stride].  All 32 lanes call together.
template <int MT, int EPI>
__device__ __forceinline__ void scatter_sum_store(const float *recv, int stride, int M, int split, int j, int64_t n, int64_t N, float scale,
                                                  float poison, const FusedAccept &fa, void *Y, int y_dtype,
                                                  const float (&res)[TokenScatter<MT>::PH]) {
    constexpr int P = TokenScatter<MT>::P, PH = TokenScatter<MT>::PH;
    float a[P];
#pragma unroll
    for (int i = 0; i < P; ++i) a[i] = (i < MT && i < M) ? recv[i * stride] : 0.f;
#pragma unroll
    for (int s = 0; s < 3; ++s) {   // clusters of up to 8
        const int o = 1 << s;
        if (o < split) {
            if ((P >> s) >= 2) {
                const bool up = ((j >> s) & 1) != 0;
#pragma unroll
                for (int i = 0; i < P / 2; ++i)
                    if (i < ((P >> s) >> 1)) {
                        const float lo = a[2 * i], hi = a[2 * i + 1];
                        const float keep = up ? hi : lo, send = up ? lo : hi;
                        a[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                    }
            } else {
                a[0] += __shfl_xor_sync(0xffffffffu, a[0], o);
            }
        }
    }
    const int S = split < P ? split : P, npos = P / S;
    const bool swiglu = EPI == kEpiLayer && fa.swiglu != 0;
#pragma unroll
    for (int i = 0; i < PH; ++i) {
        a[i] = a[i] * scale + poison;
        if (swiglu) {   // the partner row's sums sit `split` lanes away, at the same positions
            const float up = __shfl_xor_sync(0xffffffffu, a[i], split);
            a[i] = a[i] / (1.f + expf(-a[i])) * up;
        } else if (EPI == kEpiLayer) {
            a[i] += res[i];
        }
    }
    if (j < P && n < N && !(swiglu && (n & 1))) {
#pragma unroll
        for (int i = 0; i < PH; ++i) {
            const int m = i * S + (j & (S - 1));
            if (i < npos && m < M)
                store_out(Y, y_dtype, swiglu ? (int64_t)m * (N >> 1) + (n >> 1) : (int64_t)m * N + n, a[i], (int64_t)M * (swiglu ? N >> 1 : N));
        }
    }
}

}  // namespace mxq
