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
constexpr int kMmaWarps = 16;        // warps per CTA; each takes 4 of a stage's 64 MX blocks
constexpr int kMmaThreads = kMmaWarps * 32;
constexpr int kWarpBlocks = 4;       // MX blocks per warp per stage (their 4 scale bytes are one 32-bit word)
constexpr int kStageBlocks = kMmaWarps * kWarpBlocks;    // 64 blocks = 2048 weights per row per stage
// one warp's slice of one stage in shared memory: 16 rows x 64 code bytes (16-byte chunks XOR-swizzled by
// row so that fragment reads are bank-conflict free) followed by 16 rows x 4 scale bytes
constexpr int kWarpCodeBytes = kTileRows * kWarpBlocks * 16;   // 1024
constexpr int kWarpStageBytes = kWarpCodeBytes + kTileRows * 4;  // 1088
constexpr int kMaxStages = 4;
constexpr int kMaxCtaStages = 384;   // stage-table entries per CTA (16 bytes each)
constexpr int kTicketCap = 65536;    // tiles that can be tracked: N <= 16 * kTicketCap
constexpr uint32_t kSmemBudget = 113 * 1024;             // half an SM, so that two kernels can be resident
constexpr uint32_t kOffMisc = 0;
constexpr uint32_t kOffTable = 256;                      // uint4[kMaxCtaStages]
constexpr uint32_t kOffRed = kOffTable + kMaxCtaStages * 16;

// workspace layout
constexpr size_t kWsErrorOff = 0;                        // reserved, stays zero
constexpr size_t kWsFallbackOff = 4;                     // uint32: CTAs that took the exact scalar path (cumulative)
constexpr size_t kWsTicketOff = 256;
constexpr size_t kWsPartialOff = kWsTicketOff + (size_t)kTicketCap * 4;

struct LinearPlan {
    int M;            // token rows
    int nt8;          // 8-token column tiles: 1 (M <= 8) or 2
    int tiles;        // ceil(N / 16)
    int kb;           // K / 32, MX blocks per row
    int nwin;         // K windows (X for one window fits in shared memory)
    int bw;           // blocks per window (multiple of 4); the last window has bw_last
    int bw_last;
    int grid;         // CTAs
    int nstage;       // ring depth
    int slots;        // partial-result slots per CTA
    uint32_t units;   // tiles * kb: one unit = 16 rows x 32 k
    uint32_t x_stride;    // bytes between token rows of X in shared memory
    uint32_t off_x, off_ring, smem_bytes;   // ring: [warp][stage][kWarpStageBytes]
    int64_t N, K;
};

// unit order: window-major, then tile, then block within the window (k fastest)
MXQ_HD void unit_decode(const LinearPlan &p, uint32_t u, int &w, int &tile, int &b) {
    const uint32_t head = (uint32_t)(p.nwin - 1) * (uint32_t)p.tiles * (uint32_t)p.bw;
    if (u < head) {
        const uint32_t per_win = (uint32_t)p.tiles * (uint32_t)p.bw;
        w = (int)(u / per_win);
        const uint32_t r = u % per_win;
        tile = (int)(r / (uint32_t)p.bw);
        b = (int)(r % (uint32_t)p.bw);
    } else {
        const uint32_t r = u - head;
        w = p.nwin - 1;
        tile = (int)(r / (uint32_t)p.bw_last);
        b = (int)(r % (uint32_t)p.bw_last);
    }
}

MXQ_HD uint32_t pair_begin(const LinearPlan &p, int w, int tile) {  // first unit of (window, tile)
    if (w < p.nwin - 1) return ((uint32_t)w * (uint32_t)p.tiles + (uint32_t)tile) * (uint32_t)p.bw;
    return (uint32_t)(p.nwin - 1) * (uint32_t)p.tiles * (uint32_t)p.bw + (uint32_t)tile * (uint32_t)p.bw_last;
}

// CTA c owns units [cta_begin(c), cta_begin(c+1)); boundaries are multiples of 4 blocks
MXQ_HD uint32_t cta_begin(const LinearPlan &p, int c) {
    return (uint32_t)(((uint64_t)(p.units / 4) * (uint64_t)c) / (uint64_t)p.grid) * 4u;
}

MXQ_HD int cta_of(const LinearPlan &p, uint32_t u) {  // the CTA whose range holds unit u
    const uint64_t g4 = p.units / 4;
    const uint64_t gu = u / 4;
    int c = (int)(((gu + 1) * (uint64_t)p.grid + g4 - 1) / g4) - 1;
    if (c > p.grid - 1) c = p.grid - 1;
    return c;
}

// ---- stage table --------------------------------------------------------------------------
// A CTA walks its unit range in stages of at most kStageBlocks blocks that never cross a
// (window, tile) pair.  stage_lookup maps a stage number to what it covers, in closed form.
struct StageInfo {
    int w, tile, b, nblk;   // window, tile, first block within the window, blocks
    int seg_first, seg_last, win_first;
};

// stages needed for the units [u0, u1) of CTA range; if q >= 0 also describes stage q
MXQ_HD int stage_lookup(const LinearPlan &p, uint32_t u0, uint32_t u1, int q, StageInfo &out) {
    int total = 0;
    for (int w = 0; w < p.nwin; ++w) {
        const int bwid = (w == p.nwin - 1) ? p.bw_last : p.bw;
        const uint32_t wb = (uint32_t)w * (uint32_t)p.tiles * (uint32_t)p.bw;       // first unit of the window
        const uint32_t we = wb + (uint32_t)p.tiles * (uint32_t)bwid;
        const uint32_t a = u0 > wb ? u0 : wb, e = u1 < we ? u1 : we;
        if (a >= e) continue;
        const int spp = (bwid + kStageBlocks - 1) / kStageBlocks;                     // stages per whole pair
        const int t_first = (int)((a - wb) / (uint32_t)bwid), b_first = (int)((a - wb) % (uint32_t)bwid);
        const uint32_t span = e - a;
        const int len0 = (span < (uint32_t)(bwid - b_first)) ? (int)span : bwid - b_first;
        const int n0 = (len0 + kStageBlocks - 1) / kStageBlocks;
        const uint32_t rest = span - (uint32_t)len0;                                  // whole pairs, then a partial one
        const int whole = (int)(rest / (uint32_t)bwid), tail = (int)(rest % (uint32_t)bwid);
        const int ntail = (tail + kStageBlocks - 1) / kStageBlocks;
        const int here = n0 + whole * spp + ntail;
        if (q >= total && q < total + here) {
            const int ql = q - total;
            int seg_len, chunk;
            if (ql < n0) {
                out.tile = t_first;
                chunk = ql;
                out.b = b_first + chunk * kStageBlocks;
                seg_len = len0;
            } else {
                const int q2 = ql - n0;
                const int seg = q2 / spp;
                chunk = q2 - seg * spp;
                out.tile = t_first + 1 + seg;
                out.b = chunk * kStageBlocks;
                seg_len = seg < whole ? bwid : tail;
            }
            const int done = chunk * kStageBlocks;
            out.w = w;
            out.nblk = seg_len - done < kStageBlocks ? seg_len - done : kStageBlocks;
            out.seg_first = chunk == 0;
            out.seg_last = done + out.nblk == seg_len;
            out.win_first = ql == 0;
        }
        total += here;
    }
    return total;
}

}  // namespace mxq
