// TMA tensor maps over the canonical codes array [N][K/2] (host side).
#pragma once
#include <cuda.h>   // CUtensorMap and its enums only; the encoder is looked up at run time (no libcuda link)
#include <stdint.h>

namespace mxq {

// whether the driver's tensor-map encoder could be found (false without a driver)
bool tensor_map_available();

// A map whose box is one 128-row stage of weights, 128-byte swizzled:
//   expand_fp4 = true : 128 codes per row, each 8 code bytes widened into the 16-byte slot that the
//                       kind::mxf8f6f4 MMA reads (needs K % 128 == 0 and a 32-byte aligned base)
//   expand_fp4 = false: 128 packed bytes (256 codes) per row, as they are, for kind::mxf4
//                       (needs K % 32 == 0 and a 16-byte aligned base)
// Maps depend only on (device, pointer, N, K, kind); recent ones are cached.  False if encoding fails.
bool codes_tensor_map(const uint8_t *codes, int64_t N, int64_t K, bool expand_fp4, CUtensorMap *out);

// A map over a BF16 matrix [rows][K] (K % 64 == 0, 16-byte aligned base) whose box is box_rows rows x 64 elements
// (128 bytes), 128-byte swizzled; rows of the box beyond the matrix read as zeros.  Cached like the maps above.
bool bf16_tensor_map(const void *base, int64_t rows, int64_t K, int box_rows, CUtensorMap *out);

}  // namespace mxq
