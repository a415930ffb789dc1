"""Host logic of mxq_linear's stream-K decomposition, checked on the CPU.

The library reports its plan for a shape (mxq_linear_plan_info); this test replays the index
arithmetic the kernel uses -- unit ranges per CTA, segments, partial-slot numbering, ticket
totals -- in plain Python and checks the invariants the kernel relies on.
"""
import pytest

import paper_2503_13565_b200 as mxq

SMEM_HALF_SM = 113 * 1024

SHAPES = [(1, 4096, 4096), (8, 4096, 4096), (1, 11008, 4096), (8, 4096, 11008), (1, 4096, 11008),
          (16, 5120, 13824), (16, 13824, 5120), (4, 32000, 768), (1, 128256, 4096), (16, 128256, 4096),
          (1, 512, 256), (3, 203, 1408), (1, 1, 128), (16, 7, 128), (2, 16, 256), (9, 129, 5120), (5, 8192, 8192)]


def decode(p, u):
    head = (p["windows"] - 1) * p["tiles"] * p["bw"]
    if u < head:
        per = p["tiles"] * p["bw"]
        return u // per, (u % per) // p["bw"], (u % per) % p["bw"]
    r = u - head
    return p["windows"] - 1, r // p["bw_last"], r % p["bw_last"]


def pair_begin(p, w, t):
    if w < p["windows"] - 1:
        return (w * p["tiles"] + t) * p["bw"]
    return (p["windows"] - 1) * p["tiles"] * p["bw"] + t * p["bw_last"]


def cta_begin(p, c):
    return (p["units"] // 4) * c // p["grid"] * 4


def cta_of(p, u):
    g4 = p["units"] // 4
    return min(((u // 4 + 1) * p["grid"] + g4 - 1) // g4 - 1, p["grid"] - 1)


@pytest.mark.parametrize("m,n,k", SHAPES)
def test_plan_invariants(m, n, k):
    p = mxq.mxq_linear_plan_info(m, n, k)
    assert p["tensor_core"] == 1
    assert p["smem_bytes"] <= SMEM_HALF_SM
    assert p["tiles"] == (n + 15) // 16 and p["kb"] == k // 32 and p["units"] == p["tiles"] * p["kb"]
    assert p["bw"] % 4 == 0 and p["bw_last"] % 4 == 0 and p["bw_last"] > 0
    assert (p["windows"] - 1) * p["bw"] + p["bw_last"] == p["kb"]
    assert p["stages"] in (2, 3, 4) and 1 <= p["grid"] <= 148
    assert mxq.mxq_linear_workspace_bytes(m, n, k) >= 256 + 65536 * 4 + p["grid"] * p["slots"] * p["nt8"] * 8 * 16 * 4

    # ranges partition the units, on multiples of 4
    bounds = [cta_begin(p, c) for c in range(p["grid"] + 1)]
    assert bounds[0] == 0 and bounds[-1] == p["units"]
    assert all(b % 4 == 0 for b in bounds) and all(b1 > b0 for b0, b1 in zip(bounds, bounds[1:]))
    sizes = [b1 - b0 for b0, b1 in zip(bounds, bounds[1:])]
    assert max(sizes) - min(sizes) <= 4

    # walk every CTA's range the way the kernel does
    done = {}      # tile -> blocks accounted
    slots = {}     # (cta, segment index) -> (window, tile)
    step = max(1, p["grid"] // 20)
    ctas = sorted(set(list(range(0, p["grid"], step)) + [p["grid"] - 1])) if p["units"] > 200000 else range(p["grid"])
    for c in ctas:
        u, seg = bounds[c], 0
        while u < bounds[c + 1]:
            w, t, b0 = decode(p, u)
            bwid = p["bw_last"] if w == p["windows"] - 1 else p["bw"]
            seg_end = min(bwid, b0 + bounds[c + 1] - u)
            assert b0 % 4 == 0 and (seg_end - b0) % 4 == 0
            assert seg < p["slots"]
            slots[(c, seg)] = (w, t)
            assert cta_of(p, u) == c and cta_of(p, u + (seg_end - b0) - 1) == c
            done[t] = done.get(t, 0) + seg_end - b0
            u += seg_end - b0
            seg += 1
    if len(ctas) == p["grid"]:
        assert all(done[t] == p["kb"] for t in range(p["tiles"]))
        # the final reduction finds every share of a tile through the slot numbering
        for t in list(range(0, p["tiles"], max(1, p["tiles"] // 50))) + [p["tiles"] - 1]:
            total = 0
            for w in range(p["windows"]):
                pb = pair_begin(p, w, t)
                pe = pb + (p["bw_last"] if w == p["windows"] - 1 else p["bw"])
                for c in range(cta_of(p, pb), cta_of(p, pe - 1) + 1):
                    fw, ft, _ = decode(p, bounds[c])
                    slot = (w * p["tiles"] + t) - (fw * p["tiles"] + ft)
                    assert slots[(c, slot)] == (w, t)
                    total += min(pe, bounds[c + 1]) - max(pb, bounds[c])
            assert total == p["kb"]


def test_shapes_outside_the_tensor_core_path_use_the_generic_kernel():
    assert mxq.mxq_linear_plan_info(1, 64, 96)["tensor_core"] == 0          # K % 128 != 0
    assert mxq.mxq_linear_workspace_bytes(1, 64, 96) == 0
    assert mxq.mxq_linear_plan_info(1, 203, 1440)["tensor_core"] == 0


def test_headline_shapes_run_in_one_window_with_three_stages():
    for n, k in [(4096, 4096), (11008, 4096), (4096, 11008)]:
        p = mxq.mxq_linear_plan_info(1, n, k)
        assert (p["windows"], p["stages"], p["grid"]) == (1, 4, 148)
