// Work decomposition and shared-memory layout of the FP8-operand tcgen05 mxq_linear kernel (mxq_linear_umma.cu).
// Plain integers only, so the host (sizing, launch) and the tests' mirror of it agree with the device code.
#pragma once
#include <stdint.h>

namespace mxq {

#ifdef __CUDACC__
#define MXQ_UMMA_HD __host__ __device__
#else
#define MXQ_UMMA_HD
#endif

constexpr int kUmmaTileRows = 128;   // weight rows per tile = M of one tcgen05.mma
constexpr int kUmmaStageK = 128;     // k per ring stage = 4 MX blocks = 4 MMAs of K = 32
constexpr int kUmmaThreads = 192;    // MMA warp, producer warp, four activation / epilogue warps
constexpr int kUmmaParts = 3;        // E5M2 parts (columns of the token operand) per token
constexpr int kUmmaMaxM = 16;
constexpr uint32_t kUmmaStageBytes = 16384;       // shared memory per stage: 128 rows x 128 codes, 8 code bytes per 16-byte slot
constexpr uint32_t kUmmaStageTxBytes = 8192;      // what the copy engine counts for one stage: the packed bytes
constexpr uint32_t kUmmaSfStageBytes = 512;       // one scale atom: 128 rows x 4 blocks in tensor-core order
constexpr int kUmmaMaxSplit = 8;                  // portable cluster size
constexpr uint32_t kUmmaRecvRows = 136;           // >= split * ceil(128 / split) for every split <= 8
constexpr uint32_t kUmmaSmemLimit = 227 * 1024;
constexpr int kUmmaMaxUnitsResident = 12;         // most ring slots (16 KB of expanded codes + 512 B of scales each)

// The token operand split ahead of the weight kernel, in the caller's workspace: one 32-bit "cannot be split
// exactly" flag per stage (padded to 1 KB), then one 512-byte scale atom per stage, then one image of the stage's
// nb x 128 bytes of E5M2 parts per stage -- atoms and images exactly as the weight kernel keeps them in shared memory,
// so that a CTA fetches its K range with two bulk copies per 256 k.
constexpr int kUmmaPresplitMinM = 3;              // fewer token rows: splitting inside the weight kernel is as fast ...
constexpr int64_t kUmmaPresplitTwoRowsMinWeights = 1 << 23;   // ... except at two rows on matrices from 8 M weights on (2-8 % faster;
                                                              // the small draft model's layers lose 5-15 % to the extra launch)
MXQ_UMMA_HD inline size_t umma_ws_flags_bytes(int ks) { return (((size_t)ks * 4u) + 1023u) & ~(size_t)1023u; }
MXQ_UMMA_HD inline size_t umma_ws_bytes(int nb, int ks) {
    return umma_ws_flags_bytes(ks) + (size_t)ks * kUmmaSfStageBytes + (size_t)ks * (size_t)nb * 128u;
}
inline int umma_nb(int M) { return 3 * M <= 16 ? 16 : (3 * M <= 32 ? 32 : 48); }

struct UmmaPlan {
    int M;           // token rows (1..16)
    int nb;          // columns of the token operand per tile: 16, 32 or 48 (three per token)
    int ks;          // K / 128, stages per tile
    int tiles;       // ceil(N / 128)
    int split;       // CTAs (cluster size) sharing a group of tiles; CTA r takes stages [r*ks/split, (r+1)*ks/split)
    int groups;      // tile groups; group g owns tiles [g*tiles/groups, (g+1)*tiles/groups)
    int tiles_max;   // most tiles in a group = ceil(tiles / groups)
    int ring;        // (tile, stage) units in flight per CTA
    int chunk_max;   // most stages any CTA owns = ceil(ks / split)
    int grid;        // groups * split
    int tmem_cols;   // tensor-memory columns allocated per CTA
    int presplit;    // planned for a token operand split ahead of the weight kernel (needs the workspace)
    int bring;       // ... and fetched stage by stage into the ring slots instead of whole K ranges
    long cost;       // the layout heuristic's figure for the chosen decomposition (comparable within a regime)
    int pow2_split;  // in: only cluster sizes 1, 2, 4, 8 (the gate / up epilogue pairs rows inside a warp)
    int one_wave;    // in: no layout of more CTAs than are resident at once
    int layer_tiles; // most tiles for the one-tile-per-CTA regime (0: one per SM); set by umma_layout
    uint32_t smem_bytes;
    int64_t N, K;
};

inline uint32_t umma_smem_bytes(int nb, int M, int tiles_max, int chunk, int ring, int split, int bring = 0) {
    const uint32_t recv = split > 1 ? (uint32_t)(tiles_max * M) * kUmmaRecvRows * 4u : 0u;   // partial results pushed by the cluster's CTAs
    const uint32_t b = 1024u /* alignment slack */ + (uint32_t)ring * (kUmmaStageBytes + kUmmaSfStageBytes) +
                       (uint32_t)(bring ? ring : chunk) * ((uint32_t)nb * 128u + kUmmaSfStageBytes) + recv +
                       (uint32_t)(2 * ring + 2 + (chunk + 1) / 2) * 8u /* mbarriers */ + 16u /* tensor-memory address, flags */ + 208u /* fused verification: keys, tokens, flag */;
    return (b + 15u) & ~15u;
}

inline int umma_tmem_cols(int nb, int tiles_max) {
    const int need = nb * tiles_max + 16;   // one accumulator per tile + two slots of (4 + 4) scale columns
    int cols = 32;
    while (cols < need) cols *= 2;
    return cols;
}

// CTAs of this kernel that fit on one SM (shared memory incl. 1 KB of system use each; 512 tensor-memory columns)
inline int umma_ctas_per_sm(uint32_t smem_bytes, int tmem_cols) {
    const int by_smem = (int)((228u * 1024u) / (smem_bytes + 1024u)), by_tmem = 512 / tmem_cols;
    return by_smem < by_tmem ? by_smem : by_tmem;
}

// CTA slots a one-wave launch may count on (see fp4_usable_slots: grids filling more than about 95 % of the slots ran as
// two waves; 12288 x 4096 at M = 8 as 288 CTAs on 296 slots took 16.9 us, as 384 on 444 slots 11.8 us)
// (not applied to matrices of more tiles than SMs, which measured best with every slot counted: 27648 x 5120 as 432 CTAs)
inline long umma_usable_slots(int derate_sms, int sms, uint32_t smem_bytes, int tmem_cols) {
    const long slots = (long)sms * umma_ctas_per_sm(smem_bytes, tmem_cols);
    return derate_sms > 0 ? slots * 92 / 100 : slots;
}

// Chooses split, groups and ring for p.{M, nb, ks, tiles}; false if nothing fits.  Same two regimes as the packed-FP4
// kernel: up to one tile per SM -> one tile per CTA, every CTA resident at once, the split that leaves the fewest stages
// per SM outside the rings (ties to the larger split: splitting the activations is this kernel's main cost from M = 4
// on, and it shrinks with the K range);
// more tiles -> one CTA per SM walking several tiles.
// force_split / force_ring / force_tiles (> 0) override the heuristic where they are feasible.
inline bool umma_layout_one(UmmaPlan &p, int sms, int force_split, int force_ring, int force_tiles, bool allow_bring) {
    // p.presplit (set by the caller): the token operand comes ready-made from the workspace; a CTA of one tile may then
    // fetch it stage by stage with the weights (p.bring), so that its K range does not eat the ring's shared memory
    const int tcap = (512 - 16) / p.nb;   // tiles whose accumulators fit in tensor memory beside the scale columns
    const bool layer_regime = p.tiles <= (p.layer_tiles > 0 ? p.layer_tiles : sms);
    // Tiles per CTA in the layer regime: one, except for the widest token operand on matrices of many tiles, where
    // the operand's K range of a CTA (6.5 KB per stage) leaves too little shared memory for weights unless two
    // tiles share it (11008 x 4096 at M = 16: 21.5 -> 16 us).
    int tper = p.nb == 48 && 2 * p.tiles >= sms && !allow_bring ? 2 : 1;
    if (force_tiles > 0) tper = force_tiles < tcap ? force_tiles : tcap;
    long best_cost = -1;
    int best_split = 0, best_groups = 0, best_ring = 0;
    const int smax = p.ks < kUmmaMaxSplit ? p.ks : kUmmaMaxSplit;
    for (int s = 1; s <= smax; ++s) {
        if (force_split > 0 && s != (force_split < smax ? force_split : smax)) continue;
        if (p.pow2_split && (s & (s - 1)) != 0) continue;
        if (force_split <= 0 && s == 7) continue;   // clusters of 7 measured up to 1.5 times slower than of 6 or 8 (5120 x 5120, 5120 x 13824)
        const int chunk = (p.ks + s - 1) / s;
        int groups, ring;
        long cost;
        if (layer_regime) {
            groups = (p.tiles + tper - 1) / tper;
            const int tmax = (p.tiles + groups - 1) / groups;
            const long ctas = (long)groups * s;
            const int tm = umma_tmem_cols(p.nb, tmax);
            const int units = tmax * chunk;
            const int br = allow_bring && p.presplit && tmax == 1 ? 1 : 0;
            ring = units < kUmmaMaxUnitsResident ? units : kUmmaMaxUnitsResident;
            if (tper == 1 && ring > 8) ring = 8;
            if (force_ring > 0) ring = force_ring < units ? force_ring : units;
            else
                while (ring > 2 && ctas > (long)sms * umma_ctas_per_sm(umma_smem_bytes(p.nb, p.M, tmax, chunk, ring, s, br), tm)) --ring;
            while (ring > 1 && umma_smem_bytes(p.nb, p.M, tmax, chunk, ring, s, br) > kUmmaSmemLimit) --ring;
            const uint32_t bytes = umma_smem_bytes(p.nb, p.M, tmax, chunk, ring, s, br);
            if (bytes > kUmmaSmemLimit) continue;
            const long slots = umma_usable_slots(p.tiles > sms ? 0 : sms, sms, bytes, tm);
            const long waves = (ctas + slots - 1) / slots;
            // more tiles than SMs: the stages the fullest SM has to stream, with the vocabulary regime's penalty for K
            // ranges under half a row
            const long per_sm = (ctas + sms - 1) / sms * chunk * (s <= 2 ? 10 : 19);
            // Up to one tile per SM: as in the packed-FP4 kernel, the stages per SM that do not fit in the rings (they
            // are streamed inside the dependent chain; hundredths of a stage), but never with fewer than three ring
            // slots (a slot holds 8 KB here: two do not cover the latency) nor with one fat CTA per SM (which keeps the
            // next call's CTAs out) while another split avoids both.  Against "closest to two CTAs per SM", which this
            // replaced, the 13B layer set takes 98.6 instead of 116.8 us at M = 16 and 68.0 instead of 71.5 us at M = 2
            // (13824 x 5120 at M = 16: 24.9 -> 15.5 us, 8192 x 8192: 23.9 -> 15.5 us); the 7B layer set is unchanged.
            const long left = (long)(units - ring) * ctas * 100 / sms + (ring < 3 && units >= 3 ? 50000 : 0) +
                              (umma_ctas_per_sm(bytes, tm) < 2 ? 50000 : 0);
            cost = (waves - 1) * 100000 + (p.tiles > sms ? per_sm : left);
        } else {
            groups = sms / s < 1 ? 1 : sms / s;          // one CTA per SM
            if (groups > p.tiles) groups = p.tiles;
            if ((p.tiles + groups - 1) / groups > tcap) groups = (p.tiles + tcap - 1) / tcap;
            const int tmax = (p.tiles + groups - 1) / groups;
            const int units = tmax * chunk;
            ring = units < kUmmaMaxUnitsResident ? units : kUmmaMaxUnitsResident;
            if (force_ring > 0 && force_ring < ring) ring = force_ring;
            const int br = allow_bring && p.presplit ? 1 : 0;   // (every tile then fetches the token operand's stages again, from L2)
            while (ring > 1 && umma_smem_bytes(p.nb, p.M, tmax, chunk, ring, s, br) > kUmmaSmemLimit) --ring;
            if (umma_smem_bytes(p.nb, p.M, tmax, chunk, ring, s, br) > kUmmaSmemLimit) continue;
            // Time ~ units per CTA / the rate its stream reaches: two requesters at 25 GB/s each, the ring's bytes in
            // flight (8 KB of packed codes per slot) per 1.5 us of latency, the SM's share of the memory bandwidth;
            // nearly doubled for K ranges under half a row of codes (see the packed-FP4 kernel).
            const long waves = ((long)groups * s + sms - 1) / sms;
            const long by_ring = (long)ring * 8192 / 1500, rate = by_ring < 41 ? by_ring : 41;   // GB/s
            cost = waves * units * 1000 / rate * (s <= 2 ? 10 : 19) * (br ? 17 : 10) / 10 + s;   // (the operand fetched again per tile: measured)
        }
        if (best_cost < 0 || cost < best_cost || (cost == best_cost && layer_regime && p.tiles <= sms)) {   // layers: ties to the larger split
            best_cost = cost;
            best_split = s;
            best_groups = groups;
            best_ring = ring;
        }
    }
    if (best_cost < 0) return false;
    p.split = best_split;
    p.groups = best_groups;
    p.tiles_max = (p.tiles + best_groups - 1) / best_groups;
    p.ring = best_ring;
    p.chunk_max = (p.ks + best_split - 1) / best_split;
    p.grid = best_groups * best_split;
    p.bring = allow_bring && p.presplit && (!layer_regime || p.tiles_max == 1) ? 1 : 0;
    p.cost = best_cost;
    p.smem_bytes = umma_smem_bytes(p.nb, p.M, p.tiles_max, p.chunk_max, best_ring, best_split, p.bring);
    p.tmem_cols = umma_tmem_cols(p.nb, p.tiles_max);
    return true;
}

// With the token operand split ahead of the kernel there are two ways to hold it.  Whole K range resident: measured
// faster (by 0.5 us on the 7B layer shapes at M = 8) when that still leaves three ring slots and the plan fills at least
// 5/6 of the SMs.  Stage by stage through the ring otherwise (13824 x 5120 at M = 8: 22 -> 15 us).
inline bool umma_layout(UmmaPlan &p, int sms, int force_split, int force_ring, int force_tiles = 0, int force_bring = -1) {
    if (!p.presplit || force_bring == 0) return umma_layout_one(p, sms, force_split, force_ring, force_tiles, false);
    UmmaPlan r = p;
    const bool have_r = force_bring < 0 && umma_layout_one(r, sms, force_split, force_ring, force_tiles, false);
    if (p.tiles <= (p.layer_tiles > 0 ? p.layer_tiles : sms)) {
        if (have_r && r.tiles_max == 1 && r.ring >= 3 && 6 * r.grid >= 5 * sms) {
            p = r;
            return true;
        }
        if (umma_layout_one(p, sms, force_split, force_ring, force_tiles, true)) return true;
        if (have_r) p = r;
        return have_r;
    }
    // Up to two tiles per SM with the token operand coming through the ring: still one tile per CTA, all CTAs resident
    // at once (two or three small CTAs per SM), if that leaves three ring slots.  Measured against one fat CTA per SM:
    // 32000 x 4096 at M = 8: 23.4 -> 19.1 us, 22016 x 4096 at M = 8: 18.9 -> 16.8 us; small CTAs also let the next call's
    // CTAs in early.
    if (p.tiles <= 2 * sms && force_bring != 0 && force_tiles <= 0) {
        UmmaPlan l = p;
        l.layer_tiles = 2 * sms;
        if (umma_layout_one(l, sms, force_split, force_ring, 0, true) && l.tiles_max == 1 && l.ring >= 3 && l.cost < 100000) {
            p = l;
            return true;
        }
    }
    // From 6 token rows on (32 or 48 operand columns), any number of tiles: one tile and all of K per CTA, the operand
    // through the ring, the deepest ring with which two CTAs fit on an SM, as many waves as it takes.  One fat CTA per SM
    // leaves the weight stream idle while its tensor core works (the block-scaled FP8 MMA at N = 32 takes 34 ns, four per
    // stage); with two CTAs per SM one streams while the other multiplies.  128256 x 4096: 70.0 -> 64.1 us at M = 8,
    // 75.3 -> 68.0 us at M = 16; 64000 x 4096: 37.3 -> 34.6 and 43.6 -> 36.8 us.  (At M = 4 the fat CTAs win: 59.9 against
    // 63.4 us; a ring that leaves room for one CTA per SM only: 88 us.)
    if (p.nb >= 32 && force_bring != 0 && force_tiles <= 0 && force_split <= 0 && !(p.one_wave && p.tiles > 2 * sms)) {
        const int chunk = p.ks, tm = umma_tmem_cols(p.nb, 1);
        int ring = chunk < kUmmaMaxUnitsResident ? chunk : kUmmaMaxUnitsResident;
        if (ring > 8) ring = 8;
        while (ring > 1 && umma_ctas_per_sm(umma_smem_bytes(p.nb, p.M, 1, chunk, ring, 1, 1), tm) < 2) --ring;
        if (force_ring > 0 && force_ring < ring) ring = force_ring;
        const uint32_t bytes = umma_smem_bytes(p.nb, p.M, 1, chunk, ring, 1, 1);
        if (ring >= 3 && bytes <= kUmmaSmemLimit && umma_ctas_per_sm(bytes, tm) >= 2) {
            p.split = 1;
            p.groups = p.tiles;
            p.tiles_max = 1;
            p.ring = ring;
            p.chunk_max = chunk;
            p.grid = p.tiles;
            p.bring = 1;
            p.cost = (long)((p.tiles + 2L * sms - 1) / (2L * sms)) * chunk;
            p.smem_bytes = bytes;
            p.tmem_cols = tm;
            return true;
        }
    }
    // vocabulary regime: the modelled cost decides (resident on ties: no second fetch of the operand per tile)
    UmmaPlan b = p;
    const bool have_b = umma_layout_one(b, sms, force_split, force_ring, force_tiles, true);
    if (!have_r && !have_b) return false;
    p = have_r && (!have_b || r.cost <= b.cost) ? r : b;
    return true;
}

}  // namespace mxq
