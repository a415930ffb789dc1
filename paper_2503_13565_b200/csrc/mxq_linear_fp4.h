// Work decomposition and shared-memory layout of the packed-FP4 tcgen05 mxq_linear kernel (mxq_linear_fp4.cu).
// Plain integers only, so the host (sizing, launch) and the tests' mirror of it agree with the device code.
#pragma once
#include <stdint.h>

namespace mxq {

constexpr int kFp4TileRows = 128;    // weight rows per CTA = M of one tcgen05.mma
constexpr int kFp4StageK = 256;      // k per ring stage = 128 packed bytes per row = 8 MX blocks = 4 MMAs of K = 64
constexpr int kFp4Threads = 192;     // MMA warp, producer warp, four activation / epilogue warps
constexpr int kFp4Planes = 16;       // radix-4 digit planes per token (32 bits of fixed point under the block maximum)
constexpr int kFp4MaxM = 4;          // 16 planes x 4 tokens = 64 columns of the token operand
constexpr uint32_t kFp4StageBytes = 16384;        // 128 rows x 128 bytes; also what the copy engine counts
constexpr uint32_t kFp4SfStageBytes = 1024;       // two 512-byte scale atoms (4 blocks each) per stage
constexpr int kFp4MaxRing = 8;
constexpr int kFp4MaxSplit = 8;                   // portable cluster size
constexpr uint32_t kFp4RecvRows = 136;            // >= split * ceil(128 / split) for every split <= 8
constexpr uint32_t kFp4SmemLimit = 227 * 1024;

struct Fp4Plan {
    int M;           // token rows (1..4)
    int nb;          // columns of the token operand: 16, 32 or 64 (sixteen planes per token)
    int ks;          // ceil(K / 256), stages per tile; the last one is half full when K % 256 == 128
    int tiles;       // ceil(N / 128)
    int split;       // CTAs (cluster size) sharing one tile; CTA r takes stages [r*ks/split, (r+1)*ks/split)
    int ring;        // stages in flight per CTA
    int chunk_max;   // most stages any CTA owns = ceil(ks / split)
    int grid;        // tiles * split
    int tmem_cols;   // tensor-memory columns allocated per CTA
    uint32_t smem_bytes;
    int64_t N, K;
};

inline uint32_t fp4_smem_bytes(int nb, int chunk, int ring) {
    const uint32_t recv = (uint32_t)(nb / kFp4Planes) * kFp4RecvRows * 4u;   // partial results pushed by the cluster's CTAs
    const uint32_t b = 1024u /* alignment slack */ + (uint32_t)ring * (kFp4StageBytes + kFp4SfStageBytes) +
                       (uint32_t)chunk * ((uint32_t)nb * 128u + kFp4SfStageBytes) + recv +
                       (uint32_t)(2 * ring + 2 + chunk) * 8u /* mbarriers */ + 16u /* tensor-memory address, flags */;
    return (b + 15u) & ~15u;
}

// how many CTAs of `bytes` dynamic shared memory fit on one SM (each also takes 1 KB of system use)
inline int fp4_ctas_per_sm(uint32_t bytes) { return (int)((228u * 1024u) / (bytes + 1024u)); }

// Chooses split and ring for p.{M, nb, ks, tiles}; false if no choice fits in shared memory.
// Measured on B200: a call is fastest when all of its CTAs are resident at once (one wave) and there are about
// two per SM, so that one CTA's serial phases (activation split, epilogue, cluster sum) hide behind another's
// weight stream; small CTAs also leave room for the next kernel's CTAs to start their weight stream early.
// force_split / force_ring (> 0) override the heuristic where they are feasible.
inline bool fp4_layout(Fp4Plan &p, int sms, int force_split, int force_ring) {
    int best_split = 0, best_ring = 0;
    long best_cost = -1;
    const int smax = p.ks < kFp4MaxSplit ? p.ks : kFp4MaxSplit;
    for (int s = 1; s <= smax; ++s) {
        if (force_split > 0 && s != (force_split < smax ? force_split : smax)) continue;
        const int chunk = (p.ks + s - 1) / s;
        const long ctas = (long)p.tiles * s;
        // deepest ring up to 4 stages that still lets every CTA be resident at once; if none does, 4 stages
        int ring = chunk < 4 ? chunk : 4;
        if (force_ring > 0) ring = force_ring < chunk ? force_ring : chunk;
        else
            while (ring > 2 && ctas > (long)sms * fp4_ctas_per_sm(fp4_smem_bytes(p.nb, chunk, ring))) --ring;
        while (ring > 1 && fp4_smem_bytes(p.nb, chunk, ring) > kFp4SmemLimit) --ring;
        const uint32_t bytes = fp4_smem_bytes(p.nb, chunk, ring);
        if (bytes > kFp4SmemLimit) continue;
        const long slots = (long)sms * fp4_ctas_per_sm(bytes);
        const long waves = (ctas + slots - 1) / slots;
        const long off = ctas > 2L * sms ? ctas - 2L * sms : 2L * sms - ctas;   // distance from two CTAs per SM
        long cost = (waves - 1) * 100000 + off;
        if (waves > 1) cost = 100000 + (chunk > 8 ? chunk - 8 : 8 - chunk);      // many waves: about 8 stages per CTA
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best_split = s;
            best_ring = ring;
        }
    }
    if (best_cost < 0) return false;
    p.split = best_split;
    p.ring = best_ring;
    p.chunk_max = (p.ks + best_split - 1) / best_split;
    p.grid = p.tiles * best_split;
    p.smem_bytes = fp4_smem_bytes(p.nb, p.chunk_max, best_ring);
    p.tmem_cols = p.nb + 32 <= 64 ? 64 : 128;   // accumulator + two slots of (8 + 8) scale columns
    return true;
}

}  // namespace mxq
