// mxq_linear_batch: several MXFP4 layers in one persistent launch (mxq_linear_batch.cu).  Plain integers and PODs
// only, so that the host (sizing, launch), the device code and the tests' mirror of the arithmetic agree.
#pragma once
#include <cuda.h>   // CUtensorMap only
#include <stddef.h>
#include <stdint.h>

#ifdef __CUDACC__
#define MXQ_BATCH_HD __host__ __device__
#else
#define MXQ_BATCH_HD
#endif

namespace mxq {

constexpr int kBatchMaxDescs = 64;       // layers per call (the table travels as a kernel parameter, 15 KB of the 32 KB allowed)
constexpr int kBatchMaxM = 8;            // token rows: 16 digit planes each, 128 operand columns at most
constexpr int kBatchThreads = 320;       // MMA warp, producer warp, four split / epilogue warps, four scale warps
constexpr int kBatchTileRows = 128;      // weight rows per tile = M of one tcgen05.mma
constexpr int kBatchStageK = 256;        // k per unit = 128 packed bytes per row = 8 MX blocks = 4 MMAs of K = 64
constexpr uint32_t kBatchCodesBytes = 16384;   // 128 rows x 128 bytes
constexpr uint32_t kBatchSfBytes = 1024;       // two 512-byte scale atoms (4 blocks each)
constexpr uint32_t kBatchSmemLimit = 227 * 1024;
constexpr int kBatchMaxGrid = 1024;      // CTAs (ticket counters in the workspace header)
constexpr int kBatchMaxGroups = 8;       // groups of layers per call (a layer that depends on earlier ones opens a group)

// ---- workspace ------------------------------------------------------------------------------------------------------
// [0, kBatchHeaderBytes)  counters, all zero between calls; every counter that many CTAs wait for has a 128-byte line
//                          to itself (kBatchCounterStride words from one to the next):
//      u32 ready[64]   split tasks delivered per token-operand image            (words 0, 32, 64, ...)
//      u32 bad[64]     an image's list of corrections overflowed (the word after its ready counter)
//      u32 fixes[64]   entries on an image's list of corrections (the word after that)
//      u32 done[8]     tiles stored, per group                                  (words 2048, 2080, ...)
//      u32 task[8]     rewriting tasks handed out, per group                    (the word after the group's done counter)
//      u32 exit        CTAs that have finished                                  (word 2304)
//      u32 ticket[kBatchMaxGrid] at word 2560: contributors that have delivered their share of a tile split between CTAs
// [kBatchHeaderBytes, ...) partial sums: [grid][2 (at the head / at the tail of the CTA's range)][token slots][128] floats
// then the token-operand images, one per distinct X: [stage][operand rows NB x 128 bytes | 1024 bytes of scale atoms]
// then the lists of corrections, kBatchMaxFixes entries per image
constexpr size_t kBatchHeaderBytes = 16384;
constexpr int kBatchCounterStride = 32;
constexpr int kBatchWordReady = 0, kBatchWordBad = 1, kBatchWordDone = 2048, kBatchWordTask = 2049, kBatchWordExit = 2304, kBatchWordTicket = 2560;

inline int batch_nb(int M) { return M == 1 ? 16 : (M == 2 ? 32 : (M <= 4 ? 64 : 128)); }   // operand columns: 16 planes per token slot
inline uint32_t batch_image_stage_bytes(int nb) { return (uint32_t)nb * 128u + kBatchSfBytes; }
inline uint32_t batch_slot_bytes(int nb) { return kBatchCodesBytes + kBatchSfBytes + batch_image_stage_bytes(nb); }
inline size_t batch_partials_bytes(int grid, int nb) { return (size_t)grid * 2u * (size_t)(nb / 16) * 128u * 4u; }

// accumulator slots in tensor memory (at most 4; the SM's 512 columns are shared by the CTAs on it, and 32 columns go
// to the scale factors) and the columns to allocate (a power of two >= slots * nb + 32)
inline int batch_acc_slots(int nb, int ctas_per_sm) {
    const int a = (512 / ctas_per_sm - 32) / nb;
    return a < 1 ? 0 : (a > 4 ? 4 : a);
}
inline int batch_tmem_cols(int nb, int ctas_per_sm) {
    const int need = batch_acc_slots(nb, ctas_per_sm) * nb + 32;
    int cols = 32;
    while (cols < need) cols *= 2;
    return cols;
}
inline uint32_t batch_smem_bytes(int nb, int ring) {
    const uint32_t b = 1024u /* alignment slack */ + (uint32_t)ring * batch_slot_bytes(nb) +
                       (uint32_t)(2 * ring + 2 * 4) * 8u /* mbarriers */ + 128u /* tensor-memory address, flags, the CTA's ranges */;
    return (b + 15u) & ~15u;
}

// ---- partition: the call's units (layer, tile, stage), tile-major, are cut into `grid` contiguous ranges -------------
MXQ_BATCH_HD inline int64_t batch_range_lo(int64_t cta, int64_t units, int64_t grid) { return cta * units / grid; }
// the CTA whose range holds unit u (grid <= units, so no range is empty)
MXQ_BATCH_HD inline int64_t batch_owner(int64_t u, int64_t units, int64_t grid) { return ((u + 1) * grid - 1) / units; }

constexpr int kBatchMaxFixes = 256;      // elements per image that may fall outside their block's fixed point
struct BatchFix {                        // one such element: what the operand planes do not hold of X[m][k]
    int32_t m, k;
    float rem;
    uint32_t pad;
};

struct BatchDesc {
    const uint8_t *codes, *scales;
    const void *X;          // [M][K] BF16
    void *Y;
    const void *residual;   // epilogue 1
    int32_t N, K;
    int32_t ks, tiles;      // ceil(K / 256), ceil(N / 128)
    int32_t unit_base;      // first unit of this layer in the call's sequence
    int32_t img;            // its token-operand image
    int32_t y_dtype, epi;   // epi: 0 store, 1 + residual, 2 silu(gate) * up over interleaved rows
};
struct BatchImg {
    const void *X;
    int32_t K, ks;
    int32_t task_base, ntasks;   // tasks = M * K / 128 (128 k of one token row each)
    uint32_t offset;             // bytes from the workspace base
    uint32_t pad;
};
struct BatchTable {
    CUtensorMap maps[kBatchMaxDescs];
    BatchDesc desc[kBatchMaxDescs];
    BatchImg img[kBatchMaxDescs];
    uint8_t *ws;
    int32_t ndesc, nimg, M;
    int32_t units, tasks;
    int32_t ngroups;
    int32_t group_unit[kBatchMaxGroups + 1];   // first unit of every group (and the end)
    int32_t group_task[kBatchMaxGroups + 1];   // first rewriting task of every group (and the end)
    int32_t group_tiles[kBatchMaxGroups];      // tiles of every group
    int32_t ring, tmem_cols, acc_slots;
    int32_t fault_unit;          // test hook: the producer skips this unit's weight copy (-1: none)
    uint32_t wait_us;            // limit of every wait inside the kernel
    uint32_t partials_offset;    // bytes from the workspace base
    uint32_t fix_offset;         // lists of corrections, bytes from the workspace base
    uint64_t ws_bytes;           // size of the workspace (bounds-checked build)
};

}  // namespace mxq
