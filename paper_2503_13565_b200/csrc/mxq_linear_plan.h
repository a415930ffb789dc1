// Work decomposition of the tensor-core mxq_linear kernel, shared by host (sizing, launch)
// and device (index arithmetic).  Plain integers only.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define MXQ_HD __host__ __device__ __forceinline__
#else
#define MXQ_HD inline
#endif

namespace mxq {

constexpr int kTileRows = 16;        // weight rows per tile = rows of one m16n8k16 A operand
constexpr int kMmaWarps = 8;         // warps per CTA; each takes 8 of a stage's 64 MX blocks
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kWarpBlocks = 8;       // MX blocks per warp per stage (their 8 scale bytes are one 64-bit word)
constexpr int kStageBlocks = kMmaWarps * kWarpBlocks;    // 64 blocks = 2048 weights per row per stage
// one warp's slice of one stage in shared memory: codes as [row][8 chunks of 16 bytes], chunk c of row r
// stored at position c ^ (r & 7) (copies and fragment reads are both bank-conflict free), then
// 16 rows x 8 scale bytes; slots are 128-byte aligned
constexpr int kWarpCodeBytes = kTileRows * kWarpBlocks * 16;               // 2048
constexpr int kWarpStageBytes = kWarpCodeBytes + kTileRows * kWarpBlocks;  // 2176
constexpr int kMaxStages = 3;        // ring depth
constexpr int kMaxCtaStages = 128;   // stage-table entries per CTA (16 bytes each)
constexpr int kRedSlots = 4;         // tiles whose per-warp partial results can be pending at once
constexpr uint32_t kSmemQuarterSm = 56 * 1024;   // 4 CTAs per SM: two kernels, two CTAs each, can be resident
constexpr uint32_t kSmemThirdSm = 75 * 1024;     // 3 CTAs per SM
constexpr uint32_t kSmemHalfSm = 113 * 1024;     // 2 CTAs per SM
constexpr uint32_t kOffMisc = 0;
constexpr uint32_t kOffTable = 256;              // uint4[kMaxCtaStages]
constexpr uint32_t kOffRed = kOffTable + kMaxCtaStages * 16;

struct LinearPlan {
    int M;            // token rows
    int nt8;          // 8-token column tiles: 1 (M <= 8) or 2
    int kb;           // K / 32, MX blocks per row
    int nwin;         // K windows (X for one window fits in shared memory)
    int bw;           // blocks per window (multiple of 4); the last window has bw_last
    int bw_last;
    int grid;         // CTAs; CTA c owns weight rows [row_begin(c), row_begin(c+1))
    int nstage;       // ring depth
    int max_tiles;    // most 16-row tiles any CTA owns
    uint32_t x_stride;                 // bytes between token rows of X in shared memory
    uint32_t off_acc, off_x, off_ring, smem_bytes;
    int64_t N, K;
};

MXQ_HD int64_t row_begin(const LinearPlan &p, int c) { return (p.N * (int64_t)c) / p.grid; }

// ---- stage table --------------------------------------------------------------------------
// A CTA walks: for each K window, for each of its tiles, the window's blocks in stages of at most
// kStageBlocks.  stage_lookup maps a stage number to what it covers, in closed form.
struct StageInfo {
    int w, tile, b, nblk;   // window, tile (local to the CTA), first block within the window, blocks
    int seg_last, win_first;
};

// number of stages of a CTA that owns `tiles` tiles; if 0 <= q < that, also describes stage q
MXQ_HD int stage_lookup(const LinearPlan &p, int tiles, int q, StageInfo &out) {
    int total = 0;
    for (int w = 0; w < p.nwin; ++w) {
        const int bwid = (w == p.nwin - 1) ? p.bw_last : p.bw;
        const int spp = (bwid + kStageBlocks - 1) / kStageBlocks;   // stages per (window, tile) pair
        const int here = tiles * spp;
        if (q >= total && q < total + here) {
            const int ql = q - total;
            out.w = w;
            out.tile = ql / spp;
            const int chunk = ql - out.tile * spp;
            out.b = chunk * kStageBlocks;
            out.nblk = bwid - out.b < kStageBlocks ? bwid - out.b : kStageBlocks;
            out.seg_last = chunk == spp - 1;
            out.win_first = ql == 0;
        }
        total += here;
    }
    return total;
}

}  // namespace mxq
