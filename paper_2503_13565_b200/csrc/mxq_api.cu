// Entry points that launch nothing: version, status text, sizes, options.
#include <atomic>

#include "mxq_host.h"

namespace mxq {

static std::atomic<int> g_pdl{1};
bool pdl_enabled() { return g_pdl.load(std::memory_order_relaxed) != 0; }

static std::atomic<int> g_layout[7] = {{0}, {0}, {0}, {-1}, {0}, {0}, {0}};
LayoutOverride layout_override() {
    LayoutOverride o;
    o.split = g_layout[0].load(std::memory_order_relaxed);
    o.ring = g_layout[1].load(std::memory_order_relaxed);
    o.tiles = g_layout[2].load(std::memory_order_relaxed);
    o.operand_through_ring = g_layout[3].load(std::memory_order_relaxed);
    o.presplit_min_m = g_layout[4].load(std::memory_order_relaxed);
    o.batch_ring = g_layout[5].load(std::memory_order_relaxed);
    o.batch_ctas_per_sm = g_layout[6].load(std::memory_order_relaxed);
    return o;
}

int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace mxq

extern "C" {
#pragma GCC visibility push(default)

int mxq_version(void) { return MXQ_VERSION; }

const char *mxq_status_string(int status) {
    switch (status) {
        case MXQ_OK: return "ok";
        case MXQ_ERR_NULL: return "a required pointer is NULL";
        case MXQ_ERR_SHAPE: return "a size is out of range";
        case MXQ_ERR_ALIGN: return "a base pointer is not 16-byte aligned";
        case MXQ_ERR_DTYPE: return "unknown dtype selector";
        case MXQ_ERR_WORKSPACE: return "workspace missing or too small";
        case MXQ_ERR_CUDA: return "CUDA runtime error at launch";
        default: return "unknown status";
    }
}

int mxq_set_pdl(int enabled) { return mxq::g_pdl.exchange(enabled ? 1 : 0); }

int mxq_set_linear_layout(int what, int value) {
    if (what < 0 || what >= 7) return MXQ_ERR_SHAPE;
    mxq::g_layout[what].store(value, std::memory_order_relaxed);
    return MXQ_OK;
}

size_t mxq_codes_bytes(int64_t N, int64_t K) { return mxq::shape_ok(N, K) ? (size_t)N * (size_t)K / 2 : 0; }
size_t mxq_scales_bytes(int64_t N, int64_t K) { return mxq::shape_ok(N, K) ? (size_t)N * (size_t)K / 32 : 0; }

#pragma GCC visibility pop
}  // extern "C"
