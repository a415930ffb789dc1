// Device-side helpers shared by the mxq kernels (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxq.h"

#if defined(__CUDA_ARCH__) && !defined(__CUDA_ARCH_FEAT_SM100_ALL)
#error "mxq kernels use sm_100a-only conversions; compile with -gencode arch=compute_100a,code=sm_100a"
#endif

namespace mxq {

constexpr int kBlock = 32;  // weights per scale (MX block), Sec. III-D-3

// ---- programmatic dependent launch ---------------------------------------------------
// wait: block until the kernel launched before this one in the stream has completed and
// its writes are visible.  trigger: allow the next kernel in the stream to start launching.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- bounds-checked build (-DMXQ_DEBUG_BOUNDS; the stand-in for a memory checker) -------------------------------
// MXQ_AT(p, n, base, extent) stands where a kernel forms the address of a plain global load or store of n bytes into
// the buffer [base, base + extent).  The ordinary build compiles it to p.  The checked build tests the range first;
// an access outside it is counted, the first one is recorded (source line, byte offset from base, extent), and the
// access is redirected to a scratch area, so that a wrong index shows up as a report and never as a fault.  (Copies
// made by TMA are clipped by the hardware against the tensor map and need no check.)  Every translation unit keeps its
// own record; mxq_debug_bounds_report adds them up.
#ifdef MXQ_DEBUG_BOUNDS
namespace {
__device__ unsigned long long g_bounds[4];   // violations; of the first one: source line, offset, extent
__device__ uint4 g_bounds_sink[2048];   // (32 KB: the largest single access is a bulk copy of 17 KB)
}  // namespace
template <class T>
__device__ __forceinline__ T *bounds_checked(T *p, size_t n, const void *base, size_t extent, int line) {
    const uintptr_t a = (uintptr_t)p, b = (uintptr_t)base;
    if (a >= b && a + n <= b + extent) return p;
    if (atomicAdd(&g_bounds[0], 1ull) == 0ull) {
        g_bounds[1] = (unsigned long long)line;
        g_bounds[2] = (unsigned long long)(a - b);
        g_bounds[3] = (unsigned long long)extent;
    }
    return reinterpret_cast<T *>(reinterpret_cast<uintptr_t>(g_bounds_sink) + (a & 15u));   // (keeps the access's alignment)
}
#define MXQ_AT(p, n, base, extent) ::mxq::bounds_checked((p), (size_t)(n), (base), (size_t)(extent), __LINE__)
// host: this translation unit's record, cleared by the read
static int bounds_take_tu(unsigned long long *out) {
    unsigned long long zero[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(out, g_bounds, sizeof(zero)) != cudaSuccess) return MXQ_ERR_CUDA;
    return cudaMemcpyToSymbol(g_bounds, zero, sizeof(zero)) == cudaSuccess ? MXQ_OK : MXQ_ERR_CUDA;
}
#define MXQ_BOUNDS_TU(name) \
    int name(unsigned long long *out) { return bounds_take_tu(out); }
#else
#define MXQ_AT(p, n, base, extent) (p)
#define MXQ_BOUNDS_TU(name)                     \
    int name(unsigned long long *out) {         \
        out[0] = out[1] = out[2] = out[3] = 0;  \
        return MXQ_OK;                          \
    }
#endif

// ---- loads of data that the PREVIOUS kernel in the stream may have written (X, a residual, a workspace) -------------
// With programmatic dependent launch a kernel is running before its predecessor has finished, and only what it reads
// AFTER griddepcontrol.wait through the ordinary (coherent) path is guaranteed to be the predecessor's output.  A plain
// C++ dereference of a `const __restrict__` pointer may be compiled to ld.global.nc, whose cache is outside that
// guarantee: a line left there by an earlier kernel on the same SM can be served instead (seen as a layer of a chain
// computing from the previous layer's activations).  So such data is always read through these.
__device__ __forceinline__ uint4 ld_dep_u4(const void *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_dep_u32(const void *p) {
    uint32_t v;
    asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ld_dep_f32(const void *p) { return __uint_as_float(ld_dep_u32(p)); }
__device__ __forceinline__ float ld_dep_bf16(const void *p) {
    unsigned short h;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(h) : "l"(p) : "memory");
    return __uint_as_float((uint32_t)h << 16);
}

// ---- loads that bypass L1 allocation (weights are read exactly once) -------------------
__device__ __forceinline__ uint4 ld_stream_u4(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ld_stream_u32(const void *p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// ---- E2M1 / E8M0 decode ---------------------------------------------------------------
// One code byte (element 2j in the low nibble, 2j+1 in the high nibble) -> the two values
// as packed halves (.x = low nibble).  Exact: every E2M1 value is an FP16 number.
__device__ __forceinline__ __half2 e2m1x2_to_half2(uint32_t byte) {
    uint32_t out;
    asm("{\n\t.reg .b8 b;\n\tcvt.u8.u32 b, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, b;\n\t}" : "=r"(out) : "r"(byte));
    return *reinterpret_cast<__half2 *>(&out);
}

// E8M0 byte -> 2^(b-127) as FP32.  b = 0 is the subnormal 2^-127, b = 255 is NaN.
__device__ __forceinline__ float e8m0_to_float(uint32_t b) {
    uint32_t bits = (b == 0u) ? 0x00400000u : (b == 255u ? 0x7FC00000u : (b << 23));
    return __uint_as_float(bits);
}

// two FP32 -> one code byte: `lo` lands in the low nibble, `hi` in the high nibble.
// Round to nearest even, magnitudes above 6 clamp to 6.
__device__ __forceinline__ uint32_t float2_to_e2m1x2(float lo, float hi) {
    uint32_t out;
    asm("{\n\t.reg .b8 b;\n\tcvt.rn.satfinite.e2m1x2.f32 b, %1, %2;\n\tcvt.u32.u8 %0, b;\n\t}"
        : "=r"(out)
        : "f"(hi), "f"(lo));
    return out;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace mxq
