// mxq_linear_bf16: the same layer with the weights NOT quantised, Y[M,N] = X[M,K] . W[N,K]^T with W in BF16.
//
// This is the comparison point of Sec. III-D-3 and IV-D: MXFP4 streams 4.25 bits per weight where BF16 streams 16, so a
// bandwidth-bound decoding step can gain at most 3.76x from the cast.  The kernel has the structure of the MXFP4 tcgen05
// kernels (mxq_linear_fp4.cu) with everything specific to the cast removed: TMA copies 128 rows x 64 k boxes of W
// straight into the A operand (128-byte swizzle), X needs no rewriting (tcgen05.mma kind::f16 takes BF16 on both
// sides; a 16-row box of X per stage, rows beyond M filled with zeros by the copy engine), accumulation in FP32 in
// tensor memory, K split across a thread-block cluster whose CTAs push their partial rows to the owning rank.
// Products of two BF16 numbers are exact in FP32, so the result differs from the exact one by accumulation rounding only.
#include <cstdio>
#include <cstdlib>

#include "mxq_host.h"
#include "mxq_tcgen05.cuh"
#include "mxq_tensor_map.h"

namespace mxq {

namespace {

constexpr int kTileRows = 128, kStageK = 64, kThreads = 192, kMaxM = 16, kNB = 16, kMaxSplit = 8;
constexpr uint32_t kStageBytes = 16384;   // 128 rows x 64 k BF16
constexpr uint32_t kXStageBytes = 2048;   // 16 token rows x 64 k BF16
constexpr uint32_t kRecvRows = 136;       // >= split * ceil(128 / split) for every split <= 8
constexpr uint32_t kSmemLimit = 227 * 1024;

__device__ unsigned int g_bf16_status = 0;   // sticky: a bounded wait gave up

struct Bf16Plan {
    int M, ks, tiles, split, ring, chunk_max, grid;
    uint32_t smem_bytes;
    int64_t N, K;
};

uint32_t smem_bytes(int M, int chunk, int ring, int split) {
    const uint32_t recv = split > 1 ? (uint32_t)M * kRecvRows * 4u : 0u;
    return 1024u + (uint32_t)ring * kStageBytes + (uint32_t)chunk * kXStageBytes + recv + (uint32_t)(2 * ring + 3) * 8u + 16u;
}

// One tile per CTA, two CTAs per SM, ring of up to 6 stages.  Few tiles (layer-sized matrices): the split that brings the
// grid closest to two CTAs per SM (never 7).  Many tiles: several waves of CTAs; the smallest split whose K range of X
// (2 KB per stage: a 16-row box) still leaves three ring slots.
bool layout(Bf16Plan &p, int sms) {
    long best = -1;
    const int smax = p.ks < kMaxSplit ? p.ks : kMaxSplit;
    for (int s = 1; s <= smax; ++s) {
        if (s == 7) continue;
        const int chunk = (p.ks + s - 1) / s;
        int ring = chunk < 6 ? chunk : 6;
        while (ring > 1 && smem_bytes(p.M, chunk, ring, s) > 113u * 1024u) --ring;
        if (smem_bytes(p.M, chunk, ring, s) > kSmemLimit) continue;
        const long ctas = (long)p.tiles * s;
        const long shallow = (ring < 3 && ring < chunk) ? (long)(3 - ring) * 100000 : 0;   // a ring that cannot cover the latency
        const long off = ctas > 2L * sms ? (long)s * 1000 : 2L * sms - ctas;
        const long cost = shallow + off;
        if (best < 0 || cost < best || (cost == best && ctas <= 2L * sms)) {
            best = cost;
            p.split = s;
            p.ring = ring;
            p.chunk_max = chunk;
        }
    }
    if (best < 0) return false;
    p.grid = p.tiles * p.split;
    p.smem_bytes = smem_bytes(p.M, p.chunk_max, p.ring, p.split);
    return true;
}

__global__ void __launch_bounds__(kThreads)
linear_bf16_kernel(const __grid_constant__ CUtensorMap wmap, const __grid_constant__ CUtensorMap xmap, int M, int64_t N,
                   void *__restrict__ Y, int y_dtype, int split, int ring, int ks, int chunk_max) {
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&wmap) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&xmap) : "memory");
    }
    const uint32_t rank = split > 1 ? cluster_rank() : 0u;
    const int tile = (int)(blockIdx.x / (uint32_t)split);
    const int64_t n0 = (int64_t)tile * kTileRows;
    const int s_begin = (int)((rank * (uint32_t)ks) / (uint32_t)split), s_end = (int)(((rank + 1u) * (uint32_t)ks) / (uint32_t)split);
    const int nst = s_end - s_begin;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t sA = base;
    const uint32_t sX = sA + (uint32_t)ring * kStageBytes;
    const uint32_t sRecv = sX + (uint32_t)chunk_max * kXStageBytes;
    const uint32_t sBar = sRecv + (split > 1 ? (uint32_t)M * kRecvRows * 4u : 0u);
    const uint32_t full0 = sBar, empty0 = sBar + (uint32_t)ring * 8u, done_bar = sBar + (uint32_t)ring * 16u;
    const uint32_t recv_bar = done_bar + 8u, x_bar = done_bar + 16u, sMisc = done_bar + 24u;
    const float *gRecv = reinterpret_cast<const float *>(gbase + (sRecv - base));
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(gbase + (sMisc - base));
    volatile int &s_fail = *reinterpret_cast<volatile int *>(gbase + (sMisc - base) + 4);
    const int row_lo = (int)(rank * kTileRows) / split, row_cnt = (int)((rank + 1) * kTileRows) / split - row_lo;
    const int pre = nst < ring ? nst : ring;

    auto copy_w = [&](int i, uint32_t slot) {   // one lane: stage i of this CTA's K range into ring slot `slot`
        mbar_expect_tx(full0 + slot * 8, kStageBytes);
        tma_load_codes(sA + slot * kStageBytes, &wmap, (s_begin + i) * kStageK, (int)n0, full0 + slot * 8);
    };
    if (warp == 1) {
        for (int b = lane; b < 2 * ring + 3; b += 32) mbar_init(sBar + (uint32_t)b * 8u, 1u);
        if (lane == 31) s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
            if (split > 1) mbar_expect_tx(recv_bar, (uint32_t)(split * M * row_cnt) * 4u);
            for (int u = 0; u < pre; ++u) copy_w(u, (uint32_t)u);   // the weights do not depend on the previous kernel
        }
        pdl_wait();   // X may be the previous kernel's output
        if (lane == 0) {
            mbar_expect_tx(x_bar, (uint32_t)nst * kXStageBytes);
            for (int i = 0; i < nst; ++i) tma_load_codes(sX + (uint32_t)i * kXStageBytes, &xmap, (s_begin + i) * kStageK, 0, x_bar);
        }
    } else if (warp == 0) {
        pdl_trigger();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sMisc), "r"(32) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (split > 1) cluster_arrive();
    tc_fence_before();
    asm volatile("bar.sync 0;" ::: "memory");
    tc_fence_after();
    const uint32_t tmem = *tmem_holder;

    if (warp == 0) {
        // D = F32, A = B = BF16, both K-major, N = 16, M = 128
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)kNB >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t hi = (uint32_t)(smem_desc(0, 16, 1024, 2) >> 32);
        const uint32_t a_lo0 = (uint32_t)smem_desc(sA, 16, 1024, 2), b_lo0 = (uint32_t)smem_desc(sX, 16, 1024, 2);
        uint32_t slot = 0, phase = 0;
        bool ok = mbar_wait_relaxed(x_bar, 0);
        for (int i = 0; i < nst && ok; ++i) {
            if (!mbar_wait_relaxed(full0 + slot * 8, phase)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + slot * (kStageBytes >> 4), b_lo = b_lo0 + (uint32_t)i * (kXStageBytes >> 4);
            if (elect_one()) {
#pragma unroll
                for (int j = 0; j < 4; ++j)   // k [16 j, 16 j + 16) of the stage: 32 bytes further along both rows
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %6, 0;\n\t"
                        "mov.b64 da, {%1, %2};\n\tmov.b64 db, {%3, %4};\n\t"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
                        ::"r"(tmem), "r"(a_lo + j * 2), "r"(hi), "r"(b_lo + j * 2), "r"(hi), "r"(idesc), "r"((i | j) ? 1u : 0u)
                        : "memory");
                tc_commit(empty0 + slot * 8);
            }
            if (++slot == (uint32_t)ring) {
                slot = 0;
                phase ^= 1u;
            }
        }
        if (!ok && lane == 0) {
            atomicOr(&g_bf16_status, 1u);
            s_fail = 1;
        }
        __syncwarp();
        if (elect_one()) tc_commit(done_bar);
        __syncwarp();
        asm volatile("bar.sync 2, 160;" ::: "memory");   // the epilogue warps have read the accumulator
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(32) : "memory");
    } else if (warp == 1) {
        uint32_t slot = 0, phase = 0;
        for (int u = pre; u < nst; ++u) {
            if (!mbar_wait_relaxed(empty0 + slot * 8, phase)) {
                if (lane == 0) {
                    atomicOr(&g_bf16_status, 2u);
                    s_fail = 1;
                }
                break;
            }
            if (lane == 0) copy_w(u, slot);
            if (++slot == (uint32_t)ring) {
                slot = 0;
                phase ^= 1u;
            }
        }
    } else {
        const int ct = tid - 64, row = ((warp & 3) << 5) + lane;
        if (!mbar_wait_relaxed(done_bar, 0)) {
            atomicOr(&g_bf16_status, 4u);
            s_fail = 1;
        }
        tc_fence_after();
        float d[16];
        tc_load16(tmem + ((uint32_t)((warp & 3) * 32) << 16), d);   // this thread's row: one column per token
        tc_fence_before();
        asm volatile("bar.arrive 2, 160;" ::: "memory");
        if (s_fail) {
#pragma unroll
            for (int m = 0; m < 16; ++m) d[m] = __uint_as_float(0x7FC00000u);
        }
        if (split == 1) {
            const int64_t n = n0 + row;
            if (n < N)
#pragma unroll
                for (int m = 0; m < 16; ++m)
                    if (m < M) store_out(Y, y_dtype, (int64_t)m * N + n, d[m], (int64_t)M * N);
        } else {
            // as in the MXFP4 kernels: partial rows go to the rank that owns them, which adds them in a fixed order
            const int cnt_max = (kTileRows + split - 1) / split;
            const uint32_t owner = (uint32_t)(((row + 1) * split - 1) / kTileRows);
            const int rr = row - (int)(owner * kTileRows) / split;
            const uint32_t remote = peer_saddr(sRecv, owner), remote_bar = peer_saddr(recv_bar, owner);
            cluster_wait();
#pragma unroll
            for (int m = 0; m < 16; ++m)
                if (m < M) st_async_f32(remote + (uint32_t)(((int)rank * M + m) * cnt_max + rr) * 4u, d[m], remote_bar);
            if (!mbar_wait_relaxed(recv_bar, 0)) {
                atomicOr(&g_bf16_status, 16u);
                s_fail = 1;
            }
            const float poison = s_fail ? __uint_as_float(0x7FC00000u) : 0.f;
            for (int idx = ct; idx < M * row_cnt; idx += 128) {
                const int m = idx / row_cnt, r = idx - m * row_cnt;
                float acc = 0.f;
                for (int j = 0; j < split; ++j) acc += gRecv[(j * M + m) * cnt_max + r];
                const int64_t n = n0 + row_lo + r;
                if (n < N) store_out(Y, y_dtype, (int64_t)m * N + n, acc + poison, (int64_t)M * N);
            }
        }
    }
    if (split > 1 && warp < 2) cluster_wait();
}

// Fallback for K % 64 != 0 or where tensor maps are unavailable: one warp per output row, FP32 FMAs.
__global__ void __launch_bounds__(256)
linear_bf16_rowwarp_kernel(const __nv_bfloat16 *__restrict__ X, int M, const __nv_bfloat16 *__restrict__ W, int64_t N, int64_t K,
                           void *__restrict__ Y, int y_dtype) {
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (n >= N) return;
    float acc[kMaxM];
#pragma unroll
    for (int m = 0; m < kMaxM; ++m) acc[m] = 0.f;
    pdl_wait();
    for (int64_t k = lane * 2; k < K; k += 64) {
        const uint32_t wb = *reinterpret_cast<const uint32_t *>(MXQ_AT(W + n * K + k, 4, W, N * K * 2));
        const float w0 = __uint_as_float(wb << 16), w1 = __uint_as_float(wb & 0xFFFF0000u);
#pragma unroll
        for (int m = 0; m < kMaxM; ++m)
            if (m < M) {
                const uint32_t xb = ld_dep_u32(MXQ_AT(X + (int64_t)m * K + k, 4, X, (int64_t)M * K * 2));
                acc[m] = fmaf(w0, __uint_as_float(xb << 16), acc[m]);
                acc[m] = fmaf(w1, __uint_as_float(xb & 0xFFFF0000u), acc[m]);
            }
    }
#pragma unroll
    for (int m = 0; m < kMaxM; ++m) {
        float v = acc[m];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && m < M) store_out(Y, y_dtype, (int64_t)m * N + n, v, (int64_t)M * N);
    }
}

}  // namespace

int linear_bf16_take_status(uint32_t *out) {
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_bf16_status, sizeof v) != cudaSuccess) return MXQ_ERR_CUDA;
    if (v != 0 && cudaMemcpyToSymbol(g_bf16_status, &zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    *out = v;
    return MXQ_OK;
}

MXQ_BOUNDS_TU(bounds_take_linear_bf16)

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)

int mxq_linear_bf16(const void *X_bf16, int M, const void *W_bf16, int64_t N, int64_t K, void *Y, int y_dtype, void *stream) {
    using namespace mxq;
    if (!X_bf16 || !W_bf16 || !Y) return MXQ_ERR_NULL;
    if (M < 1 || M > kMaxM || N < 1 || K < 2 || (K % 2) != 0 || N > 0x7FFFFFFF || K > 0x3FFFFFFF) return MXQ_ERR_SHAPE;
    if (y_dtype != MXQ_F32 && y_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    if (!aligned16(X_bf16) || !aligned16(W_bf16) || !aligned16(Y)) return MXQ_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    cudaLaunchAttribute attr[2];
    CUtensorMap wmap, xmap;
    Bf16Plan p;
    p.M = M;
    p.N = N;
    p.K = K;
    p.ks = (int)(K / kStageK);
    p.tiles = (int)((N + kTileRows - 1) / kTileRows);
    if ((K % kStageK) == 0 && tensor_map_available() && layout(p, sm_count()) &&
        bf16_tensor_map(W_bf16, N, K, kTileRows, &wmap) && bf16_tensor_map(X_bf16, M, K, kNB, &xmap)) {
        static bool configured[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !configured[dev]) {
            if (cudaFuncSetAttribute(linear_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemLimit) != cudaSuccess ||
                cudaFuncSetAttribute(linear_bf16_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) !=
                    cudaSuccess) {
                (void)cudaGetLastError();
                return MXQ_ERR_CUDA;
            }
            configured[dev] = true;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p.grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = p.smem_bytes;
        cfg.stream = st;
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
        if (cudaLaunchKernelEx(&cfg, linear_bf16_kernel, wmap, xmap, M, N, Y, y_dtype, p.split, p.ring, p.ks, p.chunk_max) != cudaSuccess) {
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
        return launch_status();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + 7) / 8));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    cudaLaunchKernelEx(&cfg, linear_bf16_rowwarp_kernel, (const __nv_bfloat16 *)X_bf16, M, (const __nv_bfloat16 *)W_bf16, N, K, Y,
                       y_dtype);
    return launch_status();
}

#pragma GCC visibility pop
}
