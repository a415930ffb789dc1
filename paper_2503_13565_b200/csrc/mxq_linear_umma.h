// Work decomposition and shared-memory layout of the tcgen05 mxq_linear kernel (mxq_linear_umma.cu).
// Plain integers only, so the host (sizing, launch) and the tests' mirror of it agree with the device code.
#pragma once
#include <stdint.h>

namespace mxq {

constexpr int kUmmaTileRows = 128;   // weight rows per CTA = M of one tcgen05.mma
constexpr int kUmmaStageK = 128;     // k per ring stage = 4 MX blocks = 4 MMAs of K = 32
constexpr int kUmmaThreads = 128;
constexpr uint32_t kUmmaStageSmemBytes = 16384;   // 128 rows x 128 codes, each 8 code bytes in a 16-byte slot
constexpr uint32_t kUmmaStageTxBytes = 8192;      // what the copy engine counts for one stage: the packed bytes
constexpr uint32_t kUmmaSfAtomBytes = 512;        // scale bytes of 128 rows x 4 blocks in tensor-core order
constexpr int kUmmaMaxRing = 8;
constexpr int kUmmaMaxSplit = 8;                  // portable cluster size
constexpr uint32_t kUmmaRecvRows = 136;           // >= split * ceil(128 / split) for every split <= 8
constexpr uint32_t kUmmaSmemLimit = 227 * 1024;
constexpr uint32_t kUmmaSmemHalf = 113 * 1024;    // two CTAs per SM
constexpr uint32_t kUmmaSmemThird = 75 * 1024;    // three CTAs per SM

struct UmmaPlan {
    int M;           // token rows
    int nb;          // columns of the B operand: 16, 32 or 48 (three per token)
    int ks;          // K / 128, stages per tile
    int tiles;       // ceil(N / 128)
    int split;       // CTAs (cluster size) sharing one tile; CTA r takes stages [r*ks/split, (r+1)*ks/split)
    int ring;        // stages in flight per CTA
    int chunk_max;   // most stages any CTA owns = ceil(ks / split)
    int grid;        // tiles * split
    int tmem_cols;   // tensor-memory columns allocated per CTA
    uint32_t smem_bytes;
    int64_t N, K;
};

inline uint32_t umma_smem_bytes(int nb, int chunk, int ring) {
    const uint32_t recv = (uint32_t)(nb / 3) * kUmmaRecvRows * 4u;   // partial results pushed by the cluster's CTAs
    const uint32_t b = 1024u /* alignment slack */ + (uint32_t)ring * (kUmmaStageSmemBytes + kUmmaSfAtomBytes) +
                       (uint32_t)chunk * ((uint32_t)nb * 128u + kUmmaSfAtomBytes) + recv + (uint32_t)(2 * ring + 2) * 8u;
    return (b + 15u) & ~15u;
}

// Chooses split and ring for p.{M, nb, ks, tiles}; false if no choice fits in shared memory.
// force_split / force_ring (> 0) override the heuristic where they are feasible.
inline bool umma_layout(UmmaPlan &p, int sms, int force_split, int force_ring) {
    int best_split = 0, best_ring = 0;
    long best_cost = -1;
    const int smax = p.ks < kUmmaMaxSplit ? p.ks : kUmmaMaxSplit;
    for (int s = 1; s <= smax; ++s) {
        if (force_split > 0 && s != (force_split < smax ? force_split : smax)) continue;
        const int chunk = (p.ks + s - 1) / s;
        int ring = chunk < kUmmaMaxRing ? chunk : kUmmaMaxRing;
        if (force_ring > 0 && force_ring < ring) ring = force_ring;
        const int ring_floor = force_ring > 0 ? ring : (ring < 4 ? ring : 4);
        while (ring > ring_floor && umma_smem_bytes(p.nb, chunk, ring) > kUmmaSmemHalf) --ring;
        if (umma_smem_bytes(p.nb, chunk, ring) > kUmmaSmemHalf) {
            // one CTA per SM: as deep a ring as fits
            ring = chunk < kUmmaMaxRing ? chunk : kUmmaMaxRing;
            if (force_ring > 0 && force_ring < ring) ring = force_ring;
            while (ring > 2 && umma_smem_bytes(p.nb, chunk, ring) > kUmmaSmemLimit) --ring;
            if (umma_smem_bytes(p.nb, chunk, ring) > kUmmaSmemLimit) continue;
        }
        const uint32_t bytes = umma_smem_bytes(p.nb, chunk, ring);
        const int occ = bytes <= kUmmaSmemThird ? 3 : (bytes <= kUmmaSmemHalf ? 2 : 1);
        const long ctas = (long)p.tiles * s;
        const long per_sm = (ctas + sms - 1) / sms;                 // CTAs the busiest SM runs in total
        const long waves = (ctas + (long)sms * occ - 1) / ((long)sms * occ);
        const long cost = per_sm * chunk * 4 + (s > 1 ? 4 : 0) + (waves - 1) * 8;   // in quarter stages
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
    p.smem_bytes = umma_smem_bytes(p.nb, p.chunk_max, best_ring);
    p.tmem_cols = p.nb + 8 * best_ring <= 64 ? 64 : 128;
    return true;
}

}  // namespace mxq
