// mxq_linear: Y[M,N] = X[M,K] . dequant(codes, scales)[N,K]^T  (Sec. III-D-3, Eq. 2).
//
// This file holds the entry points, the dispatch and the generic kernel.  Shapes with
// K % 128 == 0 go to a tcgen05 kernel (weights as a native tensor-core operand: mxq_linear_fp4.cu
// for up to 4 token rows, mxq_linear_umma.cu above that) or, where neither covers the call, to the
// mma.sync kernel in mxq_linear_mma.cu; everything else runs the generic kernel below.
// mxq_set_linear_kernel, or MXQ_LINEAR_VARIANT in the environment (umma | mma | generic), caps the choice.
//
// Generic kernel: the weight stream (4.25 bits per weight) is the cost; X and Y are negligible.  Each warp
// owns whole output rows, so no partial sums ever leave the warp and the summation order is
// fixed.  Lanes walk the row's MX blocks with 16-byte loads (one load = one block of 32
// weights = one scale byte), decode the E2M1 pairs in registers, accumulate the 32-long
// partial sum in FP32 and apply the block scale once per block (the late scaling of Eq. 2).
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "mxq_device.cuh"
#include "mxq_host.h"
#include "mxq_linear_plan.h"
#include "mxq_linear_fp4.h"
#include "mxq_linear_umma.h"

namespace mxq {

constexpr int kRowWarpThreads = 256;
constexpr int kRowWarpRows = kRowWarpThreads / 32;

// (`count`: elements of Y, for the bounds-checked build)
__device__ __forceinline__ void store_y(void *Y, int y_dtype, int64_t idx, float v, int64_t count) {
    (void)count;
    if (y_dtype == MXQ_F32)
        *MXQ_AT(reinterpret_cast<float *>(Y) + idx, 4, Y, count * 4) = v;
    else
        *MXQ_AT(reinterpret_cast<__nv_bfloat16 *>(Y) + idx, 2, Y, count * 2) = __float2bfloat16_rn(v);
}

// Generic kernel: any M <= MT, any N, any K % 32 == 0.  One warp per output row.
template <int MT>
__global__ void __launch_bounds__(kRowWarpThreads)
linear_rowwarp_kernel(const __nv_bfloat16 *__restrict__ X, int M, const uint4 *__restrict__ codes,
                      const uint8_t *__restrict__ scales, int64_t N, int64_t K, void *__restrict__ Y, int y_dtype) {
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * kRowWarpRows + (threadIdx.x >> 5);
    if (n >= N) return;
    const int64_t nblk = K / kBlock;
    const uint4 *crow = codes + n * nblk;
    const uint8_t *srow = scales + n * nblk;

    float acc[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[m] = 0.f;

    pdl_wait();  // X may be the previous kernel's output
    for (int64_t j = lane; j < nblk; j += 32) {
        const uint4 c = ld_stream_u4(MXQ_AT(crow + j, 16, codes, N * nblk * 16));
        const float s = e8m0_to_float(*MXQ_AT(srow + j, 1, scales, N * nblk));
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
        float part[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) part[m] = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 wv = __half22float2(e2m1x2_to_half2((w[q] >> (8 * i)) & 0xFFu));
                const int64_t k = j * kBlock + q * 8 + i * 2;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    if (m < M) {
                        const uint32_t xb = ld_dep_u32(MXQ_AT(X + (int64_t)m * K + k, 4, X, (int64_t)M * K * 2));
                        part[m] = fmaf(wv.x, __uint_as_float(xb << 16), part[m]);
                        part[m] = fmaf(wv.y, __uint_as_float(xb & 0xFFFF0000u), part[m]);
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = fmaf(part[m], s, acc[m]);
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        const float v = warp_sum(acc[m]);
        if (lane == 0 && m < M) store_y(Y, y_dtype, (int64_t)m * N + n, v, (int64_t)M * N);
    }
}

template <int MT>
static void launch_rowwarp(const void *X, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                           void *Y, int y_dtype, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + kRowWarpRows - 1) / kRowWarpRows));
    cfg.blockDim = dim3(kRowWarpThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    cudaLaunchKernelEx(&cfg, linear_rowwarp_kernel<MT>, (const __nv_bfloat16 *)X, M, (const uint4 *)codes, scales, N,
                       K, Y, y_dtype);
}

// The layer epilogues where no tcgen05 kernel covers the call: one thread per output over the plain layer's FP32 sums.
__global__ void __launch_bounds__(256)
layer_epilogue_kernel(const float *__restrict__ S, int M, int64_t N, const void *residual, int swiglu, void *Y, int y_dtype) {
    pdl_trigger();
    pdl_wait();   // S is the previous kernel's output
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (swiglu) {
        const int64_t F = N >> 1;
        if (i >= (int64_t)M * F) return;
        const int64_t m = i / F, f = i - m * F;
        const float g = ld_dep_f32(MXQ_AT(S + m * N + 2 * f, 4, S, (int64_t)M * N * 4)), u = ld_dep_f32(MXQ_AT(S + m * N + 2 * f + 1, 4, S, (int64_t)M * N * 4));
        store_y(Y, y_dtype, i, g / (1.f + expf(-g)) * u, (int64_t)M * F);
    } else {
        if (i >= (int64_t)M * N) return;
        const int64_t count = (int64_t)M * N;
        const float r = y_dtype == MXQ_F32 ? ld_dep_f32(MXQ_AT(reinterpret_cast<const float *>(residual) + i, 4, residual, count * 4))
                                           : ld_dep_bf16(MXQ_AT(reinterpret_cast<const __nv_bfloat16 *>(residual) + i, 2, residual, count * 2));
        store_y(Y, y_dtype, i, ld_dep_f32(MXQ_AT(S + i, 4, S, count * 4)) + r, count);
    }
}

// mxq_linear_host: X from page-locked host memory into the device staging buffer, 16 bytes per thread.  The loads do
// not depend on earlier kernels; the stores wait for them (the previous call may still be reading the staging buffer).
__global__ void __launch_bounds__(256) stage_from_host_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int64_t n16) {
    pdl_trigger();
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (i < n16) v = *MXQ_AT(src + i, 16, src, n16 * 16);
    pdl_wait();
    if (i < n16) *MXQ_AT(dst + i, 16, dst, n16 * 16) = v;
}

// mxq_set_linear_kernel / MXQ_LINEAR_VARIANT: MXQ_KERNEL_AUTO (-1), or the highest kernel mxq_linear may use
static std::atomic<int> g_ceiling{-2};
static int kernel_ceiling() {
    int v = g_ceiling.load(std::memory_order_relaxed);
    if (v < -1) {
        const char *e = std::getenv("MXQ_LINEAR_VARIANT");
        v = MXQ_KERNEL_AUTO;
        if (e && std::strcmp(e, "generic") == 0) v = MXQ_KERNEL_GENERIC;
        else if (e && std::strcmp(e, "mma") == 0) v = MXQ_KERNEL_MMA;
        else if (e && std::strcmp(e, "umma") == 0) v = MXQ_KERNEL_UMMA;
        else if (e && std::strcmp(e, "fp4") == 0) v = MXQ_KERNEL_FP4;
        g_ceiling.store(v, std::memory_order_relaxed);
    }
    return v;
}

// The kernel mxq_linear runs for this call.
//   ceiling >= 0: the first of FP4, UMMA, MMA, GENERIC that is not above the ceiling and covers the call.
//   MXQ_KERNEL_AUTO: the same order, except that measured speed decides among the kernels that cover the call
//   (B200, layer shapes and vocabulary projections, M = 1..16): the packed-FP4 kernel wins at M = 1 everywhere and
//   at M = 2 on matrices of more row tiles of 128 than SMs; otherwise, from M = 2, its activation split (16 planes
//   per token) costs more than the FP8-operand kernel's (3 parts per token), which wins everywhere except where it
//   cannot run as one CTA per SM (M = 16 on the largest vocabularies), where the mma.sync kernel does.
// The tcgen05 kernels read the codes through a tensor map (FP4: 16-byte aligned base, which every call has; UMMA:
// 32-byte aligned base); codes == nullptr means "suitably aligned".
struct Choice {
    int kernel;
    Fp4Plan fp4;
    UmmaPlan umma;
    LinearPlan mma;
};
static void choose(int ceiling, int M, int64_t N, int64_t K, const uint8_t *codes, bool with_workspace, Choice &c, bool pow2_split = false,
                   bool one_wave = false) {
    const bool tc = linear_umma_available();
    const bool aligned32 = !codes || (reinterpret_cast<uintptr_t>(codes) & 31u) == 0;
    bool try_fp4 = ceiling == MXQ_KERNEL_AUTO || ceiling >= MXQ_KERNEL_FP4;
    bool try_umma = ceiling == MXQ_KERNEL_AUTO || ceiling >= MXQ_KERNEL_UMMA;
    const bool try_mma = ceiling == MXQ_KERNEL_AUTO || ceiling >= MXQ_KERNEL_MMA;
    if (ceiling == MXQ_KERNEL_AUTO && M >= 2) {
        const int64_t tiles = (N + 127) / 128;
        if (tiles <= (int64_t)sm_count()) {
            try_fp4 = false;
        } else {
            // vocabulary-sized matrices, where a CTA per SM walks several tiles: the packed-FP4 kernel still wins at two
            // token rows; above, the FP8-operand kernel, unless its token operand leaves no room for one CTA per SM
            try_fp4 = M == 2;
            if (M > 2 && !(tc && aligned32 && linear_umma_plan(M, N, K, c.umma, with_workspace, pow2_split, one_wave) && (c.umma.grid <= sm_count() || c.umma.tiles_max == 1)) &&
                linear_mma_plan(M, N, K, c.mma))
                try_umma = false;
        }
    }
    if (try_fp4 && tc && linear_fp4_plan(M, N, K, c.fp4, pow2_split)) c.kernel = MXQ_KERNEL_FP4;
    else if (try_umma && tc && aligned32 && linear_umma_plan(M, N, K, c.umma, with_workspace, pow2_split, one_wave)) c.kernel = MXQ_KERNEL_UMMA;
    else if (try_mma && linear_mma_plan(M, N, K, c.mma)) c.kernel = MXQ_KERNEL_MMA;
    else c.kernel = MXQ_KERNEL_GENERIC;
}

#ifdef MXQ_DEBUG_BOUNDS
// mxq_debug_bounds_selftest: one store 100 bytes into a 64-byte buffer, through the checked address: it must be counted,
// recorded and redirected (the buffer's neighbours stay as they were)
__device__ uint32_t g_selftest_buf[16 + 64];
__global__ void bounds_selftest_kernel() {
    uint8_t *buf = reinterpret_cast<uint8_t *>(g_selftest_buf);
    *MXQ_AT(reinterpret_cast<uint32_t *>(buf + 100), 4, buf, 64) = 0xDEADBEEFu;
    *MXQ_AT(reinterpret_cast<uint32_t *>(buf + 60), 4, buf, 64) = 0x600DF00Du;   // the last word inside
}
#endif

MXQ_BOUNDS_TU(bounds_take_linear)

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)
int mxq_debug_bounds_selftest(void *stream) {
#ifdef MXQ_DEBUG_BOUNDS
    uint32_t zero[16 + 64] = {};
    if (cudaMemcpyToSymbol(mxq::g_selftest_buf, zero, sizeof zero) != cudaSuccess) return MXQ_ERR_CUDA;
    mxq::bounds_selftest_kernel<<<1, 1, 0, (cudaStream_t)stream>>>();
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return MXQ_ERR_CUDA;
    uint32_t got[16 + 64];
    if (cudaMemcpyFromSymbol(got, mxq::g_selftest_buf, sizeof got) != cudaSuccess) return MXQ_ERR_CUDA;
    for (int i = 0; i < 16 + 64; ++i)
        if (got[i] != (i == 15 ? 0x600DF00Du : 0u)) return MXQ_ERR_SHAPE;   // the refused store landed in the buffer's neighbourhood
    return MXQ_OK;
#else
    (void)stream;
    return MXQ_ERR_SHAPE;   // not the bounds-checked build
#endif
}

size_t mxq_linear_workspace_bytes(int M, int64_t N, int64_t K) {
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K)) return 0;
    // No kernel needs one (partial results are added inside a thread-block cluster or never leave a warp); the
    // FP8-operand tcgen05 kernel is faster with one: the token operand is then split once per call.
    if (M == 2 && N * K < mxq::kUmmaPresplitTwoRowsMinWeights) return 0;   // two rows: only large matrices use it
    return mxq::linear_umma_available() ? mxq::linear_umma_workspace_bytes(M, K) : 0;
}

int mxq_set_linear_kernel(int kernel) {
    const int prev = mxq::kernel_ceiling();
    mxq::g_ceiling.store(kernel < MXQ_KERNEL_GENERIC || kernel > MXQ_KERNEL_FP4 ? MXQ_KERNEL_AUTO : kernel,
                         std::memory_order_relaxed);
    return prev;
}

int mxq_linear_plan_info(int kernel, int M, int64_t N, int64_t K, int32_t *info) {
    if (!info) return MXQ_ERR_NULL;
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K)) return MXQ_ERR_SHAPE;
    if (kernel < MXQ_KERNEL_AUTO || kernel > MXQ_KERNEL_FP4) return MXQ_ERR_SHAPE;
    for (int i = 0; i < 12; ++i) info[i] = 0;
    mxq::Choice c;
    if (kernel == MXQ_KERNEL_AUTO) {
        mxq::choose(mxq::kernel_ceiling(), M, N, K, nullptr, true, c);
    } else {
        c.kernel = kernel;
        const bool ok = kernel == MXQ_KERNEL_FP4    ? mxq::linear_fp4_plan(M, N, K, c.fp4)
                        : kernel == MXQ_KERNEL_UMMA ? mxq::linear_umma_plan(M, N, K, c.umma, true)
                        : kernel == MXQ_KERNEL_MMA  ? mxq::linear_mma_plan(M, N, K, c.mma)
                                                    : true;
        if (!ok) {
            info[0] = -1;
            return MXQ_OK;
        }
    }
    info[0] = c.kernel;
    if (c.kernel == MXQ_KERNEL_FP4 || c.kernel == MXQ_KERNEL_UMMA) {
        const bool f = c.kernel == MXQ_KERNEL_FP4;
        info[1] = f ? c.fp4.grid : c.umma.grid;
        info[2] = f ? c.fp4.ring : c.umma.ring;
        info[3] = f ? c.fp4.split : c.umma.split;
        info[4] = f ? c.fp4.chunk_max : c.umma.chunk_max;
        info[5] = f ? c.fp4.tiles : c.umma.tiles;
        info[6] = f ? c.fp4.tmem_cols : c.umma.tmem_cols;
        info[7] = (int32_t)(f ? c.fp4.smem_bytes : c.umma.smem_bytes);
        info[8] = f ? c.fp4.nb : c.umma.nb;
        info[9] = (int32_t)(K / 32);
        info[10] = f ? c.fp4.groups : c.umma.groups;
        info[11] = f ? c.fp4.tiles_max : c.umma.tiles_max;
    } else if (c.kernel == MXQ_KERNEL_MMA) {
        const mxq::LinearPlan &p = c.mma;
        info[1] = p.grid;
        info[2] = p.nstage;
        info[3] = p.nwin;
        info[4] = p.bw;
        info[5] = p.bw_last;
        info[6] = p.max_tiles;
        info[7] = (int32_t)p.smem_bytes;
        info[8] = p.nt8;
        info[9] = p.kb;
    } else {
        info[1] = (int32_t)((N + mxq::kRowWarpRows - 1) / mxq::kRowWarpRows);
    }
    return MXQ_OK;
}

int mxq_linear(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
               void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
    if (!X_bf16 || !codes || !scales || !Y) return MXQ_ERR_NULL;
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K)) return MXQ_ERR_SHAPE;
    if (y_dtype != MXQ_F32 && y_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    if (!mxq::aligned16(X_bf16) || !mxq::aligned16(codes) || !mxq::aligned16(scales) || !mxq::aligned16(Y))
        return MXQ_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    mxq::Choice c;
    const bool with_workspace = workspace && workspace_bytes >= mxq::linear_umma_workspace_bytes(M, K) &&
                                (reinterpret_cast<uintptr_t>(workspace) & 15u) == 0;
    mxq::choose(mxq::kernel_ceiling(), M, N, K, codes, with_workspace, c);
    if (c.kernel != MXQ_KERNEL_GENERIC) {
        const cudaError_t e =
            c.kernel == MXQ_KERNEL_FP4    ? mxq::linear_fp4_launch(c.fp4, X_bf16, codes, scales, Y, y_dtype, st)
            : c.kernel == MXQ_KERNEL_UMMA ? mxq::linear_umma_launch(c.umma, X_bf16, codes, scales, Y, y_dtype, workspace, workspace_bytes, st)
                                          : mxq::linear_mma_launch(c.mma, X_bf16, codes, scales, Y, y_dtype, nullptr, st);
        if (e != cudaSuccess) {
            if (std::getenv("MXQ_DEBUG")) std::fprintf(stderr, "mxq_linear (kernel %d): %s\n", c.kernel, cudaGetErrorString(e));
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
        return mxq::launch_status();
    }
    if (M == 1) mxq::launch_rowwarp<1>(X_bf16, M, codes, scales, N, K, Y, y_dtype, st);
    else if (M == 2) mxq::launch_rowwarp<2>(X_bf16, M, codes, scales, N, K, Y, y_dtype, st);
    else if (M <= 4) mxq::launch_rowwarp<4>(X_bf16, M, codes, scales, N, K, Y, y_dtype, st);
    else if (M <= 8) mxq::launch_rowwarp<8>(X_bf16, M, codes, scales, N, K, Y, y_dtype, st);
    else mxq::launch_rowwarp<16>(X_bf16, M, codes, scales, N, K, Y, y_dtype, st);
    return mxq::launch_status();
}

// ---- vocabulary projection fused with the greedy verification ---------------------------------------------------------
// workspace: [4096-byte header: 16 keys 128 bytes apart, ticket, a constant -1][mxq_linear's own workspace][fallback only: logits, accept scratch]
static constexpr size_t kFusedHeader = 4096;
static size_t align256(size_t v) { return (v + 255u) & ~(size_t)255u; }

// Whether the call runs as the plain layer + mxq_greedy_accept, the logits passing through the workspace: where no
// tcgen05 kernel covers it, and for the widest token operand (11 or more rows) on matrices of more than two tiles per SM,
// where the plain layer's waves of small CTAs beat the fused kernel's one-wave layout by more than the second pass over
// the logits costs (128256 x 4096 at R = 16: 69 + 15 us against 92 us; 64000 x 4096: 38 + 12 against 60 us).
static bool lm_head_unfused(const mxq::Choice &c, int R, int64_t V) {
    if (c.kernel != MXQ_KERNEL_FP4 && c.kernel != MXQ_KERNEL_UMMA) return true;
    return c.kernel == MXQ_KERNEL_UMMA && R >= 11 && (V + 127) / 128 > 2 * (int64_t)mxq::sm_count();
}

size_t mxq_lm_head_accept_workspace_bytes(int R, int64_t V, int64_t K) {
    if (R < 1 || R > MXQ_MAX_M || !mxq::shape_ok(V, K)) return 0;
    // The query does not know `codes`: a base that is 16-byte but not 32-byte aligned rules out the FP8-operand kernel
    // and may send the call down the unfused path, which needs room for the logits.  The answer covers both.
    size_t need = 0;
    for (int variant = 0; variant < 2; ++variant) {
        mxq::Choice c;
        mxq::choose(mxq::kernel_ceiling(), R, V, K, variant ? reinterpret_cast<const uint8_t *>(uintptr_t(16)) : nullptr, true, c, false, true);
        size_t b = kFusedHeader + align256(mxq_linear_workspace_bytes(R, V, K));
        if (lm_head_unfused(c, R, V))
            b += align256((size_t)R * (size_t)V * 4u) + align256(mxq_accept_workspace_bytes(R, 1, V));
        if (b > need) need = b;
    }
    return need;
}

int mxq_lm_head_accept(const void *X_bf16, int R, const uint8_t *codes, const uint8_t *scales, int64_t V, int64_t K,
                       const int32_t *draft, int T, int32_t *verifier, int32_t *accept_len, int32_t *next_token,
                       void *workspace, size_t workspace_bytes, void *stream) {
    if (!X_bf16 || !codes || !scales || !accept_len || !next_token || !workspace || (T > 0 && !draft)) return MXQ_ERR_NULL;
    if (R < 1 || R > MXQ_MAX_M || T < 0 || (R != T && R != T + 1) || !mxq::shape_ok(V, K) || V > 0x7FFFFFFF) return MXQ_ERR_SHAPE;
    if (!mxq::aligned16(X_bf16) || !mxq::aligned16(codes) || !mxq::aligned16(scales) || !mxq::aligned16(workspace)) return MXQ_ERR_ALIGN;
    if (workspace_bytes < mxq_lm_head_accept_workspace_bytes(R, V, K)) return MXQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    void *lin_ws = ws + kFusedHeader;
    const size_t lin_ws_bytes = align256(mxq_linear_workspace_bytes(R, V, K));
    mxq::Choice c;
    mxq::choose(mxq::kernel_ceiling(), R, V, K, codes, true, c, false, true);
    if (!lm_head_unfused(c, R, V)) {
        mxq::FusedAccept fa{};
        fa.keys = reinterpret_cast<unsigned long long *>(ws);
        fa.ticket = reinterpret_cast<unsigned int *>(ws + 2048);
        fa.draft = draft;
        fa.verifier = verifier;
        fa.accept_len = accept_len;
        fa.next_token = next_token;
        fa.T = T;
        const cudaError_t e = c.kernel == MXQ_KERNEL_FP4
                                  ? mxq::linear_fp4_launch(c.fp4, X_bf16, codes, scales, nullptr, MXQ_F32, st, &fa)
                                  : mxq::linear_umma_launch(c.umma, X_bf16, codes, scales, nullptr, MXQ_F32, lin_ws, lin_ws_bytes, st, &fa);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
        return mxq::launch_status();
    }
    // The plain layer with the logits in the workspace, then the argmax of every row in ONE launch (R "sequences" of one
    // row each, whose draft token -1 never matches: G = 0 and the row's argmax comes back as the next token), then the
    // walk over the draft on the R tokens.
    float *logits = reinterpret_cast<float *>(ws + kFusedHeader + lin_ws_bytes);
    void *acc_ws = ws + kFusedHeader + lin_ws_bytes + align256((size_t)R * (size_t)V * 4u);
    const size_t acc_ws_bytes = align256(mxq_accept_workspace_bytes(R, 1, V));
    if (workspace_bytes < kFusedHeader + lin_ws_bytes + align256((size_t)R * (size_t)V * 4u) + acc_ws_bytes) return MXQ_ERR_WORKSPACE;
    int32_t *minus_one = reinterpret_cast<int32_t *>(ws + 2176);   // [16]; the header's keys and ticket end at 2052
    int32_t *zeros_out = reinterpret_cast<int32_t *>(ws + 2304);   // [16] accept lengths of the argmax pass (all 0)
    int32_t *tok = verifier ? verifier : reinterpret_cast<int32_t *>(ws + 2432);
    if (cudaMemsetAsync(minus_one, 0xFF, 64, st) != cudaSuccess || cudaMemsetAsync(acc_ws, 0, acc_ws_bytes, st) != cudaSuccess)
        return MXQ_ERR_CUDA;
    int rc = mxq_linear(X_bf16, R, codes, scales, V, K, logits, MXQ_F32, lin_ws, lin_ws_bytes, stream);
    if (rc != MXQ_OK) return rc;
    rc = mxq_greedy_accept(logits, MXQ_F32, R, 1, V, minus_one, 1, zeros_out, tok, acc_ws, acc_ws_bytes, stream);
    if (rc != MXQ_OK) return rc;
    if (T == 0) {   // the plain draft step: no token to verify, the argmax is the next token
        if (cudaMemsetAsync(accept_len, 0, 4, st) != cudaSuccess ||
            cudaMemcpyAsync(next_token, tok, 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return MXQ_ERR_CUDA;
        return MXQ_OK;
    }
    return mxq_greedy_accept_tokens(draft, tok, 1, T, R, accept_len, next_token, stream);
}

// ---- layer epilogues: residual add, gate / up pairing -------------------------------------------------------------------
// workspace: [mxq_linear's own workspace][FP32 sums of the plain layer, used where no tcgen05 kernel covers the call]
size_t mxq_linear_fused_workspace_bytes(int M, int64_t N, int64_t K) {
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K)) return 0;
    return align256(mxq_linear_workspace_bytes(M, N, K)) + align256((size_t)M * (size_t)N * 4u);
}

static int linear_with_epilogue(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                                const void *residual, int swiglu, void *Y, int y_dtype, void *workspace,
                                size_t workspace_bytes, void *stream) {
    if (!X_bf16 || !codes || !scales || !Y || !workspace || (!swiglu && !residual)) return MXQ_ERR_NULL;
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K) || (swiglu && (N & 1))) return MXQ_ERR_SHAPE;
    if (y_dtype != MXQ_F32 && y_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    if (!mxq::aligned16(X_bf16) || !mxq::aligned16(codes) || !mxq::aligned16(scales) || !mxq::aligned16(Y) ||
        !mxq::aligned16(workspace) || (residual && !mxq::aligned16(residual)))
        return MXQ_ERR_ALIGN;
    if (workspace_bytes < mxq_linear_fused_workspace_bytes(M, N, K)) return MXQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const size_t lin_ws_bytes = align256(mxq_linear_workspace_bytes(M, N, K));
    mxq::Choice c;
    mxq::choose(mxq::kernel_ceiling(), M, N, K, codes, true, c, swiglu != 0);
    if (c.kernel == MXQ_KERNEL_FP4 || c.kernel == MXQ_KERNEL_UMMA) {
        mxq::FusedAccept fa{};
        fa.residual = swiglu ? nullptr : residual;
        fa.swiglu = swiglu;
        const cudaError_t e = c.kernel == MXQ_KERNEL_FP4
                                  ? mxq::linear_fp4_launch(c.fp4, X_bf16, codes, scales, Y, y_dtype, st, &fa)
                                  : mxq::linear_umma_launch(c.umma, X_bf16, codes, scales, Y, y_dtype, ws, lin_ws_bytes, st, &fa);
        if (e != cudaSuccess) {
            if (std::getenv("MXQ_DEBUG")) std::fprintf(stderr, "mxq_linear epilogue (kernel %d): %s\n", c.kernel, cudaGetErrorString(e));
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
        return mxq::launch_status();
    }
    // no tcgen05 kernel covers the call: the plain layer's sums pass through the workspace
    float *sums = reinterpret_cast<float *>(ws + lin_ws_bytes);
    const int rc = mxq_linear(X_bf16, M, codes, scales, N, K, sums, MXQ_F32, ws, lin_ws_bytes, stream);
    if (rc != MXQ_OK) return rc;
    const int64_t outs = (int64_t)M * (swiglu ? N / 2 : N);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((outs + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = mxq::pdl_enabled() ? 1 : 0;
    cudaLaunchKernelEx(&cfg, mxq::layer_epilogue_kernel, (const float *)sums, M, N, residual, swiglu, Y, y_dtype);
    return mxq::launch_status();
}

int mxq_linear_residual(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                        const void *residual, void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
    return linear_with_epilogue(X_bf16, M, codes, scales, N, K, residual, 0, Y, y_dtype, workspace, workspace_bytes, stream);
}

int mxq_linear_swiglu(const void *X_bf16, int M, const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K,
                      void *Y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream) {
    return linear_with_epilogue(X_bf16, M, codes, scales, N, K, nullptr, 1, Y, y_dtype, workspace, workspace_bytes, stream);
}

// Device-side address of page-locked host memory that the GPU can reach, or nullptr (pageable memory, no mapping)
static void *device_view_of_host(const void *p) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

int mxq_linear_host(const void *X_host, int M, const uint8_t *codes, const uint8_t *scales, int64_t N,
                    int64_t K, void *Y_host, int y_dtype, void *X_stage_dev, void *Y_stage_dev,
                    void *workspace, size_t workspace_bytes, void *stream) {
    if (!X_host || !Y_host || !X_stage_dev || !Y_stage_dev || !codes || !scales) return MXQ_ERR_NULL;
    if (M < 1 || M > MXQ_MAX_M || !mxq::shape_ok(N, K)) return MXQ_ERR_SHAPE;
    if (y_dtype != MXQ_F32 && y_dtype != MXQ_BF16) return MXQ_ERR_DTYPE;
    // everything mxq_linear would refuse is refused here, before the staging copy of X is enqueued
    if (!mxq::aligned16(codes) || !mxq::aligned16(scales) || !mxq::aligned16(X_stage_dev) || !mxq::aligned16(Y_stage_dev))
        return MXQ_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    // Page-locked host buffers that the GPU can address are moved by the GPU itself: a one-wave kernel pulls X across
    // the bus into the staging buffer (the copy engine's start-up costs several times the transfer of 8-350 KB), and the
    // layer stores Y straight into host memory.  Anything else goes through cudaMemcpyAsync.
    void *x_view = device_view_of_host(X_host), *y_view = device_view_of_host(Y_host);
    if (x_view && mxq::aligned16(x_view) && mxq::aligned16(X_stage_dev)) {
        const int64_t n16 = (int64_t)M * K / 8;   // 16-byte pieces (K % 32 == 0)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((n16 + 255) / 256));
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = mxq::pdl_enabled() ? 1 : 0;
        if (cudaLaunchKernelEx(&cfg, mxq::stage_from_host_kernel, (const uint4 *)x_view, (uint4 *)X_stage_dev, n16) != cudaSuccess) {
            (void)cudaGetLastError();
            return MXQ_ERR_CUDA;
        }
    } else if (cudaMemcpyAsync(X_stage_dev, X_host, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return MXQ_ERR_CUDA;
    }
    const bool y_direct = y_view && mxq::aligned16(y_view);
    const int rc = mxq_linear(X_stage_dev, M, codes, scales, N, K, y_direct ? y_view : Y_stage_dev, y_dtype, workspace,
                              workspace_bytes, stream);
    if (rc != MXQ_OK || y_direct) return rc;
    const size_t ybytes = (size_t)M * N * (y_dtype == MXQ_F32 ? 4 : 2);
    if (cudaMemcpyAsync(Y_host, Y_stage_dev, ybytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return MXQ_ERR_CUDA;
    return MXQ_OK;
}

#pragma GCC visibility pop
}  // extern "C"
