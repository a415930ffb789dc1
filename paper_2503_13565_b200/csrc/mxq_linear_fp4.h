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
constexpr int kFp4MaxSplit = 8;                   // portable cluster size
constexpr uint32_t kFp4RecvRows = 136;            // >= split * ceil(128 / split) for every split <= 8
constexpr uint32_t kFp4SmemLimit = 227 * 1024;

struct Fp4Plan {
    int M;           // token rows (1..4)
    int nb;          // columns of the token operand per tile: 16, 32 or 64 (sixteen planes per token)
    int ks;          // ceil(K / 256), stages per tile; the last one is half full when K % 256 == 128
    int tiles;       // ceil(N / 128)
    int split;       // CTAs (cluster size) sharing a group of tiles; CTA r takes stages [r*ks/split, (r+1)*ks/split)
    int groups;      // tile groups; group g owns tiles [g*tiles/groups, (g+1)*tiles/groups)
    int tiles_max;   // most tiles in a group = ceil(tiles / groups)
    int ring;        // (tile, stage) units in flight per CTA
    int chunk_max;   // most stages any CTA owns = ceil(ks / split)
    int grid;        // groups * split
    int tmem_cols;   // tensor-memory columns allocated per CTA
    int pow2_split;  // in: only cluster sizes 1, 2, 4, 8 (the gate / up epilogue pairs rows inside a warp)
    uint32_t smem_bytes;
    int64_t N, K;
};

constexpr int kFp4MaxUnitsResident = 12;   // most ring slots (16 KB of codes + 1 KB of scales each)

inline uint32_t fp4_smem_bytes(int nb, int M, int tiles_max, int chunk, int ring, int split) {
    const uint32_t recv = split > 1 ? (uint32_t)(tiles_max * M) * kFp4RecvRows * 4u : 0u;   // partial results pushed by the cluster's CTAs
    const uint32_t b = 1024u /* alignment slack */ + (uint32_t)ring * (kFp4StageBytes + kFp4SfStageBytes) +
                       (uint32_t)chunk * ((uint32_t)nb * 128u + kFp4SfStageBytes) + recv +
                       (uint32_t)(2 * ring + 2 + chunk) * 8u /* mbarriers */ + 16u /* tensor-memory address, three flags */ + 208u /* fused verification: keys, tokens, flag */;
    return (b + 15u) & ~15u;
}

inline int fp4_tmem_cols(int nb, int tiles_max) {
    const int need = nb * tiles_max + 32;   // one accumulator per tile + two slots of (8 + 8) scale columns
    int cols = 32;
    while (cols < need) cols *= 2;
    return cols;
}

// CTAs of this kernel that fit on one SM: shared memory (each CTA also takes 1 KB of system use) and tensor-memory
// columns (512 per SM).  The occupancy calculator reports 1 for any kernel that contains tcgen05.alloc, but the hardware
// does place several such CTAs on an SM when these two resources allow (checked on B200 by recording %smid and
// residency intervals).
inline int fp4_ctas_per_sm(uint32_t smem_bytes, int tmem_cols) {
    const int by_smem = (int)((228u * 1024u) / (smem_bytes + 1024u)), by_tmem = 512 / tmem_cols;
    return by_smem < by_tmem ? by_smem : by_tmem;
}

// CTA slots of the whole GPU that a one-wave launch may count on: a grid that fills more than about 95 % of them ran as
// if in two waves (clusters are placed inside one GPC, and the last ones find no GPC with room): 12288 x 4096 as 288 CTAs
// on 296 slots took 12.8 us, as 384 on 444 slots 8.3 us; 13824 x 5120 as 432 on 444 13.3 us, as 540 on 592 10.3 us.
inline long fp4_usable_slots(int sms, uint32_t smem_bytes, int tmem_cols) {
    return (long)sms * fp4_ctas_per_sm(smem_bytes, tmem_cols) * 92 / 100;
}

// Chooses split, groups and ring for p.{M, nb, ks, tiles}; false if nothing fits.
//
// Two regimes, both measured on B200:
//  - up to 2 * SMs tiles (the transformer layers themselves): one tile per CTA; the deepest ring up to 4 stages that
//    still lets every CTA of the call be resident at once; the split that leaves the fewest stages per SM outside
//    the rings.  Small CTAs matter twice: the call runs as one wave, and what it leaves free of an SM's shared memory is taken
//    by the CTAs of the next call (programmatic dependent launch), which start their weight stream early.
//  - more tiles (vocabulary projections): one CTA per SM walking several tiles with a deep ring, so that the
//    activations of a K range are split once per CTA and the pipeline never drains between tiles; the cost of a
//    choice is the number of (tile, stage) units per CTA, weighted as the code below says.
// force_split / force_ring (> 0) override the heuristic where they are feasible.
inline bool fp4_layout(Fp4Plan &p, int sms, int force_split, int force_ring, int force_tiles = 0) {
    const int tcap = (512 - 32) / p.nb;   // tiles whose accumulators fit in tensor memory beside the scale columns
    // (one token row: up to 2 * SMs tiles; more rows: up to SMs tiles, because every CTA of the first regime splits the
    // token rows over all of K before its stream can run ahead: 32000 x 4096 at M = 2 ran at 2.4 TB/s there)
    const bool layer_regime = p.tiles <= (p.nb == 16 ? 2 * sms : sms);
    long best_cost = -1;
    int best_split = 0, best_groups = 0, best_ring = 0;
    const int smax = p.ks < kFp4MaxSplit ? p.ks : kFp4MaxSplit;
    for (int s = 1; s <= smax; ++s) {
        if (force_split > 0 && s != (force_split < smax ? force_split : smax)) continue;
        if (p.pow2_split && (s & (s - 1)) != 0) continue;
        if (force_split <= 0 && s == 7) continue;   // clusters of 7 measured up to 1.5 times slower than of 6 or 8 (5120 x 5120, 5120 x 13824)
        const int chunk = (p.ks + s - 1) / s;
        // Matrices of more tiles than SMs are also tried with two tiles per CTA (half as much of X to split per tile;
        // taken only where the cost below is strictly lower: 32000 x 4096 at M = 1 16.2 -> 15.4 us, 22016 x 4096 13.1 ->
        // 12.6 us; on 11008 x 4096, a tie, two tiles per CTA measured 8.6 against 8.2 us).
        const int tries = layer_regime && force_tiles <= 0 && p.tiles > sms ? 2 : 1;
        for (int tp = 1; tp <= tries; ++tp) {
        int groups, ring;
        long cost;
        if (layer_regime) {
            int tper = force_tiles > 0 ? (force_tiles < tcap ? force_tiles : tcap) : tp;
            groups = (p.tiles + tper - 1) / tper;
            tper = (p.tiles + groups - 1) / groups;
            const long ctas = (long)groups * s;
            const int tm = fp4_tmem_cols(p.nb, tper);
            const int units = tper * chunk;
            ring = units < 4 ? units : 4;
            if (force_ring > 0) ring = force_ring < units ? force_ring : units;
            else
                while (ring > 2 && ctas > fp4_usable_slots(sms, fp4_smem_bytes(p.nb, p.M, tper, chunk, ring, s), tm)) --ring;
            while (ring > 1 && fp4_smem_bytes(p.nb, p.M, tper, chunk, ring, s) > kFp4SmemLimit) --ring;
            const uint32_t bytes = fp4_smem_bytes(p.nb, p.M, tper, chunk, ring, s);
            if (bytes > kFp4SmemLimit) continue;
            const long slots = fp4_usable_slots(sms, bytes, tm);
            const long waves = (ctas + slots - 1) / slots;
            // What a CTA cannot request before the activations arrive -- its stages beyond the ring -- is streamed
            // inside the dependent chain: the cost is that remainder per SM (in hundredths of a stage).  Measured at
            // M = 1: 11008 x 4096 8.05 us (split 4, 2.3 stages per SM left) / 8.23 (split 3, 3.5) / 8.80 (split 6, 3.5) /
            // 9.37 (split 2, 4.6); 12288 x 4096 8.3 us (split 4, 2.6) / 9.95 (split 3 with three slots, 5.8) / 9.4 (split 2, 5.2).
            cost = (waves - 1) * 100000 + (long)(units - ring) * ctas * 100 / sms;
        } else {
            groups = sms / s < 1 ? 1 : sms / s;          // one CTA per SM
            if (groups > p.tiles) groups = p.tiles;
            if ((p.tiles + groups - 1) / groups > tcap) groups = (p.tiles + tcap - 1) / tcap;
            const int tmax = (p.tiles + groups - 1) / groups;
            const int units = tmax * chunk;
            ring = units < kFp4MaxUnitsResident ? units : kFp4MaxUnitsResident;
            if (force_ring > 0 && force_ring < ring) ring = force_ring;
            while (ring > 1 && fp4_smem_bytes(p.nb, p.M, tmax, chunk, ring, s) > kFp4SmemLimit) --ring;
            if (fp4_smem_bytes(p.nb, p.M, tmax, chunk, ring, s) > kFp4SmemLimit) continue;
            // time ~ units per CTA; a K range narrower than half a row of codes costs almost twice as much per byte
            // (the parts of a row are then fetched by three or more SMs at unrelated times: 64000 x 4096 ran at
            // 2.6 TB/s with split 4 and at 5.0 TB/s with split 2); a ring too shallow to cover the latency costs too
            const long waves = ((long)groups * s + sms - 1) / sms;
            const long by_ring = (long)ring * 16384 / 1500, rate = by_ring < 40 ? by_ring : 40;   // GB/s: bytes in flight per 1.5 us, one requester
            cost = waves * units * 1000 / rate * (s <= 2 ? 10 : 19) + s;
        }
        // layer regime: ties go to the larger split (less of X per CTA) as long as that does not put more than two CTAs
        // on an SM (32000 x 768 at M = 1: 250 CTAs of one tile and all of K 5.0 us, 750 CTAs in clusters of 3 7.7 us)
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && layer_regime && tp == 1 && (long)groups * s <= 2L * sms)) {
            best_cost = cost;
            best_split = s;
            best_groups = groups;
            best_ring = ring;
        }
        }
    }
    if (best_cost < 0) return false;
    p.split = best_split;
    p.groups = best_groups;
    p.tiles_max = (p.tiles + best_groups - 1) / best_groups;
    p.ring = best_ring;
    p.chunk_max = (p.ks + best_split - 1) / best_split;
    p.grid = best_groups * best_split;
    p.smem_bytes = fp4_smem_bytes(p.nb, p.M, p.tiles_max, p.chunk_max, best_ring, best_split);
    p.tmem_cols = fp4_tmem_cols(p.nb, p.tiles_max);
    return true;
}

}  // namespace mxq
