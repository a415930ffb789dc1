// mxq_quantize / mxq_dequantize: the direct cast BF16 -> MXFP4 of Sec. III-D-3 and its
// exact inverse map.
//
// Data movement is the whole cost: 2 bytes read and 0.53125 bytes written per weight, so
// the kernel is a pure HBM stream.  Because K is a multiple of 32, MX blocks never straddle
// a row and the three tensors can be walked as flat arrays of blocks: block b is 64 bytes of
// W, 16 bytes of codes and one scale byte.  One lane per block: four 16-byte loads, the block
// maximum without any exchange between lanes, one 16-byte store of codes and one byte of scale.
// (The first version gave a lane one 16-byte chunk and let four lanes agree on the maximum with
// shuffles: 89 instructions per chunk, most of them index arithmetic, bounds checks and the
// exchange, kept the half-rate integer pipe 70 % busy and the kernel at 79 % of the copy rate.)
#include "mxq_device.cuh"
#include "mxq_host.h"

namespace mxq {

constexpr int kQuantThreads = 256;
constexpr int kQuantUnroll = 2;  // blocks (64 bytes each) in flight per lane

// Cast the 8 BF16 values of one chunk given the block's scale byte; returns 8 packed codes.
// The kernel is a stream of 2.5 bytes per weight, so the integer pipe must not spend more than a few instructions
// per weight: the conversion instruction takes the sign along (a negative value that rounds to zero gives the
// code of -0, as the cast requires).
__device__ __forceinline__ uint32_t cast_chunk(const uint4 &v, float inv_x) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float lo[4], hi[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        lo[j] = __uint_as_float(w[j] << 16) * inv_x;            // element 2j
        hi[j] = __uint_as_float(w[j] & 0xFFFF0000u) * inv_x;    // element 2j+1
    }
    // round-to-nearest-even, clamp, sign kept; the bytes are packed with multiply-adds, which run on the other pipe
    uint32_t c[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) c[j] = float2_to_e2m1x2(lo[j], hi[j]);
    uint32_t out;
    asm("{\n\t.reg .u32 t;\n\tmad.lo.u32 t, %2, 256, %1;\n\tmad.lo.u32 t, %3, 65536, t;\n\tmad.lo.u32 %0, %4, 16777216, t;\n\t}"
        : "=r"(out)
        : "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]));
    return out;
}

// largest magnitude pattern (15 bits, in both halves of the result's halves) among the 8 BF16 values of a chunk: for
// finite BF16 the magnitude bits order like the values; two values per instruction
__device__ __forceinline__ uint32_t chunk_max2(const uint4 &v) {
    const uint32_t m = 0x7FFF7FFFu;
    return __vmaxu2(__vmaxu2(v.x & m, v.y & m), __vmaxu2(v.z & m, v.w & m));
}

__device__ __forceinline__ uint4 ld_nc_u4(const uint4 *p) {   // (cached in L1: the four loads of a lane share sectors with its neighbours')
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// IDX: 32-bit block indices where the tensor allows it (half the index arithmetic)
template <typename IDX>
__global__ void __launch_bounds__(kQuantThreads)
quantize_kernel(const uint4 *__restrict__ W, uint4 *__restrict__ codes, uint8_t *__restrict__ scales,
                uint32_t *__restrict__ nonfinite_blocks, IDX nblocks, IDX iters) {
    const IDX stride = (IDX)gridDim.x * kQuantThreads;
    const IDX tid = (IDX)blockIdx.x * kQuantThreads + threadIdx.x;
    for (IDX it = 0; it < iters; ++it) {
        uint4 v[kQuantUnroll][4];
        IDX idx[kQuantUnroll];
#pragma unroll
        for (int u = 0; u < kQuantUnroll; ++u) {
            idx[u] = (it * kQuantUnroll + u) * stride + tid;
            if (idx[u] < nblocks) {
                const uint4 *src = W + (size_t)idx[u] * 4;
#pragma unroll
                for (int q = 0; q < 4; ++q) v[u][q] = ld_nc_u4(src + q);
            }
        }
#pragma unroll
        for (int u = 0; u < kQuantUnroll; ++u)
            if (idx[u] < nblocks) {
                const uint32_t a2 = __vmaxu2(__vmaxu2(chunk_max2(v[u][0]), chunk_max2(v[u][1])), __vmaxu2(chunk_max2(v[u][2]), chunk_max2(v[u][3])));
                const uint32_t a = max(a2 & 0xFFFFu, a2 >> 16);
                const uint32_t efield = a >> 7;               // biased exponent of the block maximum
                const bool nonfinite = efield == 0xFFu;       // Inf/NaN sort above every finite pattern
                // floor(log2 max) - 2 + 127 = efield - 2; clamped at 0 (also covers subnormal and zero maxima)
                const uint32_t byte = nonfinite ? 0xFFu : (efield > 2u ? efield - 2u : 0u);
                // v / X with X = 2^(byte-127): multiply by 2^(127-byte), exact (a power of two; results stay below 8 in
                // magnitude, and anything that underflows is far below the first rounding boundary)
                const float inv_x = __uint_as_float((254u - byte) << 23);
                uint4 c = make_uint4(0u, 0u, 0u, 0u);
                if (!nonfinite) c = make_uint4(cast_chunk(v[u][0], inv_x), cast_chunk(v[u][1], inv_x), cast_chunk(v[u][2], inv_x), cast_chunk(v[u][3], inv_x));
                codes[idx[u]] = c;
                scales[idx[u]] = (uint8_t)byte;
                if (nonfinite && nonfinite_blocks != nullptr) atomicAdd(nonfinite_blocks, 1u);
            }
    }
}

// One lane per MX block: 16 code bytes + 1 scale byte -> 32 BF16 values.
__global__ void __launch_bounds__(256)
dequantize_kernel(const uint4 *__restrict__ codes, const uint8_t *__restrict__ scales, uint4 *__restrict__ W,
                  int64_t nblocks) {
    const int64_t b = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (b >= nblocks) return;
    const uint4 c = codes[b];
    const float s = e8m0_to_float(scales[b]);
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(e2m1x2_to_half2((w[j] >> (8 * i)) & 0xFFu));
            // value * 2^(b-127) has at most two significant bits: the FP32 product is exact and its
            // upper 16 bits are the BF16 number (subnormal results included)
            o[i] = (__float_as_uint(f.x * s) >> 16) | (__float_as_uint(f.y * s) & 0xFFFF0000u);
        }
        W[b * 4 + j] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)

int mxq_quantize(const void *W_bf16, int64_t N, int64_t K, uint8_t *codes, uint8_t *scales,
                 uint32_t *nonfinite_blocks, void *stream) {
    if (!W_bf16 || !codes || !scales) return MXQ_ERR_NULL;
    if (!mxq::shape_ok(N, K)) return MXQ_ERR_SHAPE;
    if (!mxq::aligned16(W_bf16) || !mxq::aligned16(codes) || !mxq::aligned16(scales)) return MXQ_ERR_ALIGN;
    if (nonfinite_blocks && (reinterpret_cast<uintptr_t>(nonfinite_blocks) & 3u)) return MXQ_ERR_ALIGN;
    const int64_t nblocks = N * K / 32;
    const int64_t per_pass = (int64_t)mxq::kQuantThreads * mxq::kQuantUnroll;
    int64_t grid = (nblocks + per_pass - 1) / per_pass;
    const int64_t cap = (int64_t)mxq::sm_count() * 16;  // more CTAs than are resident at once: measured faster than one wave
    if (grid > cap) grid = cap;
    const int64_t iters = (nblocks + grid * per_pass - 1) / (grid * per_pass);
    if (nblocks + grid * per_pass < 0x7FFFFFFF)
        mxq::quantize_kernel<uint32_t><<<(unsigned)grid, mxq::kQuantThreads, 0, (cudaStream_t)stream>>>(
            (const uint4 *)W_bf16, (uint4 *)codes, scales, nonfinite_blocks, (uint32_t)nblocks, (uint32_t)iters);
    else
        mxq::quantize_kernel<int64_t><<<(unsigned)grid, mxq::kQuantThreads, 0, (cudaStream_t)stream>>>(
            (const uint4 *)W_bf16, (uint4 *)codes, scales, nonfinite_blocks, nblocks, iters);
    return mxq::launch_status();
}

int mxq_dequantize(const uint8_t *codes, const uint8_t *scales, int64_t N, int64_t K, void *W_bf16_out,
                   void *stream) {
    if (!codes || !scales || !W_bf16_out) return MXQ_ERR_NULL;
    if (!mxq::shape_ok(N, K)) return MXQ_ERR_SHAPE;
    if (!mxq::aligned16(codes) || !mxq::aligned16(scales) || !mxq::aligned16(W_bf16_out)) return MXQ_ERR_ALIGN;
    const int64_t nblocks = N * K / 32;
    const int64_t grid = (nblocks + 255) / 256;
    mxq::dequantize_kernel<<<(unsigned)grid, 256, 0, (cudaStream_t)stream>>>((const uint4 *)codes, scales,
                                                                             (uint4 *)W_bf16_out, nblocks);
    return mxq::launch_status();
}

#pragma GCC visibility pop
}  // extern "C"
