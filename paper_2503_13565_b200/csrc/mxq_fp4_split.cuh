// The exact rewriting of BF16 token rows as packed 4-bit operands of tcgen05.mma kind::mxf4.block_scale, shared by the
// packed-FP4 kernels (mxq_linear_fp4.cu writes the operand into its own shared memory; mxq_linear_batch.cu writes it
// once per distinct X into global memory, from where every CTA fetches it with bulk copies).
//
// Within a block of 32 along K every BF16 element is an integer multiple of a common power of two: relative to the
// block's largest exponent it is a 32-bit fixed-point number, i.e. 16 radix-4 digits.  Digit plane p (the digits 0..3
// are the E2M1 codes of 0, 0.5, 1, 1.5, so a digit is its own code; the element's sign goes into bit 3) is one row of
// the operand with block scale 2^(top - 2p - guard).  The tensor core multiplies every plane with the weights
// exactly; the kernel's epilogue adds a token's 16 accumulator columns.  Elements more than 24 binades below their
// block's maximum would lose bits (so would Inf / NaN): the functions report such blocks and the caller computes the
// affected sums with scalar FP32 code instead.
#pragma once
#include <stdint.h>

#include "mxq_device.cuh"

namespace mxq {

// Every partial sum is bounded by sum |x w^|, which cancellation can leave up to 1/2e-3 = 500 times larger than a
// result that still has to come out finite.  So the token operand's scales carry an extra 2^-kGuard, all sums are
// formed 2^kGuard too small, and the factor is restored once, at the final store.  (What this costs at the bottom of
// the FP32 range is far below the layer's absolute tolerance.)
constexpr int kGuard = 10;
constexpr float kGuardUp = 1024.f, kGuardDown = 1.f / 1024.f;

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t mask, uint32_t c) {   // (a & mask) | c
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(c));
    return d;
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
        x[i] = lop3_and_or(a, 0x0F0F0F0Fu, (b & 0x0F0F0F0Fu) << 4);
        x[i + 1] = lop3_and_or(b, 0xF0F0F0F0u, (a >> 4) & 0x0F0F0F0Fu);
    }
}

// Where the operand goes: a shared-window address (st.shared) or a global pointer (plain stores).
struct SplitToShared {
    uint32_t base;
    __device__ __forceinline__ void u32(uint32_t off, uint32_t v) const {
        asm volatile("st.shared.u32 [%0], %1;" ::"r"(base + off), "r"(v) : "memory");
    }
    __device__ __forceinline__ void u8(uint32_t off, uint32_t v) const {
        asm volatile("st.shared.u8 [%0], %1;" ::"r"(base + off), "r"(v) : "memory");
    }
};
struct SplitToGlobal {
    uint8_t *base;
    const uint8_t *whole;   // the buffer `base` points into and its size (bounds-checked build)
    size_t whole_bytes;
    __device__ __forceinline__ void u32(uint32_t off, uint32_t v) const { *MXQ_AT(reinterpret_cast<uint32_t *>(base + off), 4, whole, whole_bytes) = v; }
    __device__ __forceinline__ void u8(uint32_t off, uint32_t v) const { *MXQ_AT(base + off, 1, whole, whole_bytes) = (uint8_t)v; }
};

// Half of one 8-element unit of X (16 bytes `raw`; token slot m; k offset kin inside a 256-k stage): the lane with
// half = 0 writes digit planes 0..7, its neighbour with half = 1 planes 8..15; the two lanes of a 32-block's first
// unit also write the planes' scale bytes.  Lane layout inside a warp: lane = 8 * block + 2 * unit + half; all 32
// lanes call together (the block maximum is formed with shuffles).  `b` addresses the stage's operand rows (NB rows
// of 128 bytes in 8-row groups of 1024 bytes, no swizzle), `sf` the stage's two 512-byte scale atoms.  Returns
// whether this lane met an element that cannot be written exactly.
// With `rem` (8 floats, may be nullptr) the function also says what is missing: the planes then hold each element
// truncated to the block's 32-bit fixed point (all zeros for a block that contains an Inf or a NaN), and rem[i] is
// element i minus what the planes hold -- exactly, in FP32 -- so that the caller can add rem[i] * w to the sums.
template <class Dst>
__device__ __forceinline__ bool split_half_unit_to(const uint4 raw, int m, uint32_t kin, int half, int lane, const Dst b, const Dst sf,
                                                   float *rem = nullptr) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    // largest exponent field of the 32-block: both halves of a word at once, then across the block's four units
    uint32_t e2 = (w[0] >> 7) & 0x00FF00FFu;
#pragma unroll
    for (int i = 1; i < 4; ++i) e2 = __vmaxu2(e2, (w[i] >> 7) & 0x00FF00FFu);
    uint32_t emax = max(e2 & 0xFFFFu, e2 >> 16);
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 2));
    emax = max(emax, __shfl_xor_sync(0xffffffffu, emax, 4));
    bool inexact = emax == 255u;                        // Inf or NaN in the block
    // 32-bit fixed point under the block maximum: plane p holds bits 31-2p, 30-2p, worth digit * 2^(top - 128 - 2p)
    const uint32_t top = min(max(emax, 31u + kGuard), 254u);
    const float up = __uint_as_float((285u - top) << 23);   // 2^(158 - top), a normal number for every top in 41..254
    const float down = __uint_as_float((top - 31u) << 23);  // 2^(top - 158)
    const bool nonfinite = emax == 255u;
    const uint32_t pick = half ? 0x4140u : 0x4342u;          // bytes (b0, 0, b1, 0) of this lane's 16 bits of the fixed point
    uint32_t pl[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t word = w[i >> 1];
        const uint32_t mag = (i & 1) ? (word & 0x7FFF0000u) : ((word << 16) & 0x7FFF0000u);   // |x| as FP32 bits
        // |x| * 2^(158 - top) is the fixed-point value (bit 31 is worth 2^(top - 127)); it is below 2^32, and any
        // fraction it has is exactly the bits that would fall off the bottom
        const float scaled = __uint_as_float(mag) * up;
        uint32_t f = __float2uint_rz(scaled);
        const float lost = scaled - __uint2float_rn(f);   // (exact: both have at most 8 significant bits)
        if (lost != 0.f) inexact = true;
        const uint32_t sbit = ((i & 1) ? word : (word << 16)) & 0x80000000u;
        if (rem != nullptr) {
            if (nonfinite) {
                f = 0u;                                    // the block contributes nothing through the planes
                rem[i] = __uint_as_float(mag | sbit);      // ... and everything through the remainder
            } else {
                rem[i] = __uint_as_float(__float_as_uint(lost * down) | sbit);
            }
        }
        const uint32_t sgn = (uint32_t)((int32_t)((i & 1) ? word : (word << 16)) >> 31) & 0x88888888u;
        uint32_t v = __byte_perm(f, 0u, pick);            // 8 digits in bytes 0 and 2
        v = (v | (v << 4)) & 0x0F0F0F0Fu;                 // 2 digits per byte
        pl[i] = lop3_and_or(v | (v << 2), 0x33333333u, sgn);   // one digit (its own code) per nibble, nibble j = plane 8 half + 7 - j
    }
    transpose_nibbles8(pl);   // now pl[j] = plane 8 * half + 7 - j, nibble i = element i
    const uint32_t dst = (uint32_t)(m * 2 + half) * 1024u + (kin >> 5) * 128u + ((kin & 31u) >> 1);
#pragma unroll
    for (int q = 0; q < 8; ++q) b.u32(dst + (7 - q) * 16, pl[q]);   // row group 2m + half, row 7 - q
    if ((lane & 6) == 0) {
        const uint32_t kb = kin >> 5;
        const uint32_t row0 = (uint32_t)(16 * m + 8 * half);   // first of this lane's eight planes (rows of the operand)
        const uint32_t at = (kb >> 2) * 512u + (kb & 3u) + (row0 & 31u) * 16u + (row0 >> 5) * 4u;
        const uint32_t byte0 = top - kGuard - 16u * half;   // digit d is stored as the code of d / 2: one above 2^(top-128-2p), less the guard
#pragma unroll
        for (int q = 0; q < 8; ++q) sf.u8(at + q * 16, byte0 - 2 * q);
    }
    return inexact;
}

}  // namespace mxq
