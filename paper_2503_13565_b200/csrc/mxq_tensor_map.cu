// Host-side cache of TMA tensor maps over the canonical codes array.
#include "mxq_tensor_map.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>

namespace mxq {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        (void)cudaGetLastError();
        return (EncodeTiledFn)p;
    }();
    return fn;
}

struct MapSlot {
    int dev;
    const void *ptr;
    int64_t N, K;
    bool expand, valid;
    CUtensorMap map;
};
constexpr int kMapSlots = 1024;
MapSlot g_maps[kMapSlots];
std::mutex g_maps_mutex;

}  // namespace

bool tensor_map_available() { return encode_fn() != nullptr; }

bool codes_tensor_map(const uint8_t *codes, int64_t N, int64_t K, bool expand_fp4, CUtensorMap *out) {
    int dev = 0;
    cudaGetDevice(&dev);
    const uint64_t h = (reinterpret_cast<uintptr_t>(codes) >> 8) * 0x9E3779B97F4A7C15ull + (uint64_t)N * 31 + (uint64_t)K * 2 +
                       (expand_fp4 ? 1 : 0);
    MapSlot &slot = g_maps[(h >> 40) % kMapSlots];
    std::lock_guard<std::mutex> lock(g_maps_mutex);
    if (slot.valid && slot.dev == dev && slot.ptr == codes && slot.N == N && slot.K == K && slot.expand == expand_fp4) {
        *out = slot.map;
        return true;
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    // expanded: dimension 0 counts codes (the type packs two per byte); packed: dimension 0 counts bytes
    const cuuint64_t gdim[2] = {(cuuint64_t)(expand_fp4 ? K : K / 2), (cuuint64_t)N};
    const cuuint64_t gstr[1] = {(cuuint64_t)(K / 2)};
    const cuuint32_t box[2] = {128, 128};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(&slot.map, expand_fp4 ? CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                          const_cast<uint8_t *>(codes), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (std::getenv("MXQ_DEBUG"))
            std::fprintf(stderr, "mxq: tensor map encode failed (%d) for N=%lld K=%lld\n", (int)r, (long long)N, (long long)K);
        slot.valid = false;
        return false;
    }
    slot.dev = dev;
    slot.ptr = codes;
    slot.N = N;
    slot.K = K;
    slot.expand = expand_fp4;
    slot.valid = true;
    *out = slot.map;
    return true;
}

bool bf16_tensor_map(const void *base, int64_t rows, int64_t K, int box_rows, CUtensorMap *out) {
    int dev = 0;
    cudaGetDevice(&dev);
    const uint64_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 0x9E3779B97F4A7C15ull + (uint64_t)rows * 131 + (uint64_t)K * 2 +
                       (uint64_t)box_rows * 7 + 3;
    MapSlot &slot = g_maps[(h >> 40) % kMapSlots];
    std::lock_guard<std::mutex> lock(g_maps_mutex);
    // (kind of map in the slot: N holds rows, expand holds false, K holds -(K + box_rows) to keep BF16 maps apart from code maps)
    const int64_t tag = -(K * 1024 + box_rows);
    if (slot.valid && slot.dev == dev && slot.ptr == base && slot.N == rows && slot.K == tag && !slot.expand) {
        *out = slot.map;
        return true;
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t gstr[1] = {(cuuint64_t)(K * 2)};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(&slot.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstr, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (std::getenv("MXQ_DEBUG"))
            std::fprintf(stderr, "mxq: BF16 tensor map encode failed (%d) for rows=%lld K=%lld\n", (int)r, (long long)rows, (long long)K);
        slot.valid = false;
        return false;
    }
    slot.dev = dev;
    slot.ptr = base;
    slot.N = rows;
    slot.K = tag;
    slot.expand = false;
    slot.valid = true;
    *out = slot.map;
    return true;
}

}  // namespace mxq
