"""Host logic of mxq_linear's decomposition, checked on the CPU.

The library reports its plan for a shape (mxq_linear_plan_info); this test replays the index
arithmetic the kernel uses -- row ranges per CTA, tiles, the closed-form stage table -- in plain
Python and checks the invariants the kernel relies on.
"""
import pytest

import paper_2503_13565_b200 as mxq

SMEM_HALF_SM, SMEM_QUARTER_SM = 113 * 1024, 56 * 1024
STAGE_BLOCKS, MAX_CTA_STAGES, SMS = 64, 128, 148

SHAPES = [(1, 4096, 4096), (8, 4096, 4096), (1, 11008, 4096), (8, 4096, 11008), (1, 4096, 11008),
          (16, 5120, 13824), (16, 13824, 5120), (4, 32000, 768), (1, 128256, 4096), (16, 128256, 4096),
          (1, 512, 256), (3, 203, 1408), (1, 1, 128), (16, 7, 128), (2, 16, 256), (9, 129, 5120), (5, 8192, 8192),
          (8, 1000000, 128)]


def stage_lookup(p, tiles, q):
    """Python port of the closed form the kernel uses to describe stage q of a CTA with `tiles` tiles."""
    total, out = 0, None
    for w in range(p["windows"]):
        bwid = p["bw_last"] if w == p["windows"] - 1 else p["bw"]
        spp = -(-bwid // STAGE_BLOCKS)
        here = tiles * spp
        if total <= q < total + here:
            ql = q - total
            tile, chunk = divmod(ql, spp)
            b = chunk * STAGE_BLOCKS
            out = dict(w=w, tile=tile, b=b, nblk=min(STAGE_BLOCKS, bwid - b), seg_last=chunk == spp - 1,
                       win_first=ql == 0)
        total += here
    return total, out


@pytest.mark.parametrize("m,n,k", SHAPES)
def test_plan_invariants(m, n, k):
    p = mxq.mxq_linear_plan_info(m, n, k, "mma")
    assert p["kernel"] == "mma"
    assert p["smem_bytes"] <= SMEM_HALF_SM
    assert p["kb"] == k // 32
    assert p["bw"] % 4 == 0 and p["bw_last"] % 4 == 0 and p["bw_last"] > 0
    assert (p["windows"] - 1) * p["bw"] + p["bw_last"] == p["kb"]
    assert p["stages"] in (2, 3)
    assert p["grid"] == min(n, p["grid"]) and (p["grid"] == n or p["grid"] % (2 * SMS) == 0)
    assert mxq.mxq_linear_workspace_bytes(m, n, k) == 0

    # row ranges partition [0, N) and differ by at most one row
    bounds = [n * c // p["grid"] for c in range(p["grid"] + 1)]
    assert bounds[0] == 0 and bounds[-1] == n
    sizes = {b1 - b0 for b0, b1 in zip(bounds, bounds[1:])}
    assert min(sizes) >= 1 and max(sizes) - min(sizes) <= 1
    assert -(-max(sizes) // 16) == p["max_tiles"]

    # the stage table of the largest CTA fits, and the closed form matches a sequential walk
    tiles = p["max_tiles"]
    walk = []
    for w in range(p["windows"]):
        bwid = p["bw_last"] if w == p["windows"] - 1 else p["bw"]
        first = True
        for t in range(tiles):
            b = 0
            while b < bwid:
                nb = min(STAGE_BLOCKS, bwid - b)
                walk.append(dict(w=w, tile=t, b=b, nblk=nb, seg_last=b + nb == bwid, win_first=first))
                first = False
                b += nb
    total, _ = stage_lookup(p, tiles, -1)
    assert total == len(walk) <= MAX_CTA_STAGES
    for q in list(range(min(total, 60))) + list(range(max(0, total - 60), total)):
        assert stage_lookup(p, tiles, q)[1] == walk[q], q
    # every block of every window is covered exactly once per tile
    covered = {}
    for s in walk:
        covered[(s["w"], s["tile"])] = covered.get((s["w"], s["tile"]), 0) + s["nblk"]
    assert sum(v for (w, t), v in covered.items() if t == 0) == p["kb"]


def test_shapes_outside_the_tensor_core_paths_use_the_generic_kernel():
    assert mxq.mxq_linear_plan_info(1, 3, 1 << 20, "mma")["kernel"] is None      # a single row would overflow the stage table
    for kernel in ("mma", "umma", "fp4"):
        assert mxq.mxq_linear_plan_info(1, 64, 96, kernel)["kernel"] is None      # K % 128 != 0
        assert mxq.mxq_linear_plan_info(1, 203, 1440, kernel)["kernel"] is None
    assert mxq.mxq_linear_workspace_bytes(1, 64, 96) == 0
    assert mxq.mxq_linear_plan_info(1, 64, 96)["kernel"] == "generic"
    assert mxq.mxq_linear_plan_info(1, 64, 96, "generic") == {"kernel": "generic", "grid": 8}


def test_headline_shapes_run_two_ctas_per_sm():
    """M=1 on the 7B layers with the mma.sync kernel: one window, two or three stages, two CTAs per SM."""
    for n, k, limit in [(4096, 4096, SMEM_HALF_SM), (11008, 4096, SMEM_HALF_SM), (4096, 11008, SMEM_HALF_SM)]:
        p = mxq.mxq_linear_plan_info(1, n, k, "mma")
        assert (p["windows"], p["grid"]) == (1, 2 * SMS) and p["stages"] in (2, 3), p
        assert p["smem_bytes"] <= limit, p


UMMA_SHAPES = SHAPES + [(1, 32000, 4096), (1, 1000, 65536), (16, 4096, 28672), (4, 300, 128)]


@pytest.mark.parametrize("m,n,k", UMMA_SHAPES)
def test_tcgen05_plan_invariants(m, n, k):
    """FP8-operand tcgen05 kernel: a CTA owns a K range (its rank in a cluster of `split` <= 8) of a group of 128-row
    tiles; everything it keeps in shared and tensor memory fits."""
    p = mxq.mxq_linear_plan_info(m, n, k, "umma")
    assert p["kernel"] == "umma"
    ks = k // 128
    tiles = -(-n // 128)
    assert p["kb"] == k // 32 and p["tiles"] == tiles
    assert 1 <= p["split"] <= min(8, ks)
    assert 1 <= p["groups"] <= tiles and p["grid"] == p["groups"] * p["split"]
    assert p["tiles_max"] == -(-tiles // p["groups"])
    assert p["chunk_max"] == -(-ks // p["split"])
    assert 1 <= p["ring"] <= min(12, p["tiles_max"] * p["chunk_max"])
    assert p["nb"] in (16, 32, 48) and p["nb"] >= 3 * m and (p["nb"] == 16 or p["nb"] - 16 < 3 * m)
    assert p["smem_bytes"] <= 227 * 1024
    assert p["tmem_cols"] in (32, 64, 128, 256, 512) and p["tmem_cols"] >= p["nb"] * p["tiles_max"] + 16
    # the stage ranges of a cluster's CTAs partition [0, K/128) and none is empty
    bounds = [r * ks // p["split"] for r in range(p["split"] + 1)]
    sizes = [b1 - b0 for b0, b1 in zip(bounds, bounds[1:])]
    assert bounds[0] == 0 and bounds[-1] == ks and min(sizes) >= 1 and max(sizes) <= p["chunk_max"]
    tb = [g * tiles // p["groups"] for g in range(p["groups"] + 1)]
    tsz = [b1 - b0 for b0, b1 in zip(tb, tb[1:])]
    assert tb[0] == 0 and tb[-1] == tiles and min(tsz) >= 1 and max(tsz) == p["tiles_max"]
    # rows of a tile are shared out among the cluster's CTAs for the final sum
    rb = [r * 128 // p["split"] for r in range(p["split"] + 1)]
    assert rb[-1] == 128 and p["split"] * max(b1 - b0 for b0, b1 in zip(rb, rb[1:])) <= 136
    for row in range(128):
        owner = ((row + 1) * p["split"] - 1) // 128
        assert rb[owner] <= row < rb[owner + 1]


def test_tcgen05_kernel_needs_whole_stages():
    assert mxq.mxq_linear_plan_info(1, 4096, 4096 + 64, "umma")["kernel"] is None
    assert mxq.mxq_linear_plan_info(1, 4096, 96, "umma")["kernel"] is None


@pytest.mark.parametrize("m,n,k", [(m, n, k) for (m, n, k) in UMMA_SHAPES if m <= 4] + [(2, 11008, 4096), (3, 5000, 1408),
                                   (1, 128256, 4096), (4, 128256, 4096), (2, 1000000, 128)])
def test_packed_fp4_plan_invariants(m, n, k):
    """Stages of 256 k (the last one half full when K % 256 == 128), sixteen digit planes per token; a CTA owns a K
    range (its rank in the cluster) of a group of tiles."""
    p = mxq.mxq_linear_plan_info(m, n, k, "fp4")
    assert p["kernel"] == "fp4"
    ks = -(-k // 256)
    tiles = -(-n // 128)
    assert p["kb"] == k // 32 and p["tiles"] == tiles
    assert 1 <= p["split"] <= min(8, ks)
    assert 1 <= p["groups"] <= tiles and p["grid"] == p["groups"] * p["split"]
    assert p["tiles_max"] == -(-tiles // p["groups"])
    assert p["chunk_max"] == -(-ks // p["split"])
    assert 1 <= p["ring"] <= min(12, p["tiles_max"] * p["chunk_max"])
    slots = {1: 1, 2: 2, 3: 4, 4: 4}[m]
    assert p["nb"] == 16 * slots
    assert p["smem_bytes"] <= 227 * 1024
    assert p["tmem_cols"] in (32, 64, 128, 256, 512) and p["tmem_cols"] >= p["nb"] * p["tiles_max"] + 32
    # stage ranges of a cluster's CTAs partition [0, ks); tile ranges of the groups partition [0, tiles)
    bounds = [r * ks // p["split"] for r in range(p["split"] + 1)]
    sizes = [b1 - b0 for b0, b1 in zip(bounds, bounds[1:])]
    assert bounds[0] == 0 and bounds[-1] == ks and min(sizes) >= 1 and max(sizes) <= p["chunk_max"]
    tb = [g * tiles // p["groups"] for g in range(p["groups"] + 1)]
    tsz = [b1 - b0 for b0, b1 in zip(tb, tb[1:])]
    assert tb[0] == 0 and tb[-1] == tiles and min(tsz) >= 1 and max(tsz) == p["tiles_max"]


def test_packed_fp4_kernel_is_for_few_tokens_and_whole_half_stages():
    assert mxq.mxq_linear_plan_info(5, 4096, 4096, "fp4")["kernel"] is None
    assert mxq.mxq_linear_plan_info(1, 4096, 4096 + 64, "fp4")["kernel"] is None


def test_packed_fp4_regimes():
    """Transformer-layer shapes: one tile per CTA, every CTA of the call resident at once with room to spare for the
    next call's CTAs.  Vocabulary projection with a thousand tiles: one CTA per SM, each walking several tiles."""
    for n, k in [(4096, 4096), (11008, 4096), (4096, 11008), (5120, 5120), (13824, 5120), (5120, 13824)]:
        p = mxq.mxq_linear_plan_info(1, n, k, "fp4")
        assert p["tiles_max"] == 1 and p["groups"] == p["tiles"]
        per_sm = min((228 * 1024) // (p["smem_bytes"] + 1024), 512 // p["tmem_cols"])
        assert per_sm >= 2 and p["grid"] <= SMS * per_sm, p
        assert SMS < p["grid"] <= 4 * SMS and p["ring"] <= 4
    p = mxq.mxq_linear_plan_info(1, 128256, 4096, "fp4")
    assert p["tiles_max"] > 1 and p["grid"] <= SMS


def test_one_wave_layouts_leave_slack():
    """One tile per CTA (two, for packed-FP4 matrices of more tiles than SMs) with every CTA resident at once: the grid may
    count on 92 % of the CTA slots only (fuller grids were measured to run as two waves)."""
    for m, kernel, shapes in [(1, "fp4", [(4096, 4096), (11008, 4096), (4096, 11008), (12288, 4096), (22016, 4096), (5120, 5120),
                                          (13824, 5120), (5120, 13824), (8192, 8192)]),
                              (8, "umma", [(4096, 4096), (11008, 4096), (4096, 11008), (12288, 4096), (5120, 5120), (13824, 5120),
                                           (5120, 13824), (8192, 8192)])]:
        for n, k in shapes:
            p = mxq.mxq_linear_plan_info(m, n, k, kernel)
            assert p["tiles_max"] == 1 or (kernel == "fp4" and p["tiles_max"] == 2 and p["tiles"] > SMS), p
            per_sm = min((228 * 1024) // (p["smem_bytes"] + 1024), 512 // p["tmem_cols"])
            assert p["grid"] <= SMS * per_sm * 92 // 100, (n, k, p)
            if kernel == "umma":
                assert p["ring"] >= 3 and per_sm >= 2, (n, k, p)
