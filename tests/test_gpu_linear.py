"""GPU parity of mxq_linear against the oracle: |y - y64| <= 2e-3 * sum|x w^| + 1e-6 element by element."""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from golden_io import direct_cast_blocks, linear_block_a
from paper_2503_13565_b200 import synth
from parity import check_linear, gpu_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["auto", "fp4", "umma", "mma"])
def linear_kernel(request):
    """Every case runs four times: with the library's own choice of kernel (by measured speed), and with the choice
    capped at the packed-FP4 tcgen05 kernel (used for up to 4 token rows wherever it covers the shape), at the
    FP8-operand tcgen05 kernel, and at the mma.sync kernel (else the generic one)."""
    prev = mxq.mxq_set_linear_kernel(request.param)
    yield request.param
    mxq.mxq_set_linear_kernel(prev)
    assert mxq.mxq_linear_device_status() == 0, "a bounded wait inside the tcgen05 kernel gave up"


def run_case(wbits, xbits, out_dtype=torch.float32, rows=None, what=""):
    """Quantise on the oracle side, run the layer on both sides from the same bytes."""
    codes, scales, _ = oracle.quantize(wbits)
    y64, a64 = oracle.linear(xbits, codes, scales, rows=rows)
    n, k = wbits.shape
    m = xbits.shape[0]
    ws = mxq.new_workspace(mxq.mxq_linear_workspace_bytes(m, n, k))
    y = mxq.mxq_linear(gpu_bf16(xbits), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(),
                       out_dtype=out_dtype, workspace=ws)
    torch.cuda.synchronize()
    if rows is not None:
        y = y[:, torch.as_tensor(rows, device="cuda")]
    return check_linear(y, y64, a64, what), y


def test_config1_tiny():
    w = synth.bits_of(synth.weight(1, 0, 512, 256))
    x = synth.bits_of(synth.activations(1, 0, 1, 256))
    run_case(w, x, what="config1")


@pytest.mark.parametrize("m", [1, 4])
@pytest.mark.parametrize("idx,n,k", [(0, 768, 768), (4, 3072, 768), (6, 768, 3072), (7, 32000, 768)])
def test_config2_small_draft(idx, n, k, m):
    w = synth.bits_of(synth.weight(2, idx, n, k))
    x = synth.bits_of(synth.activations(2, idx, m, k))
    run_case(w, x, what="config2 %dx%d M=%d" % (n, k, m))


@pytest.mark.parametrize("m", [1, 8])
@pytest.mark.parametrize("idx,n,k", [(0, 4096, 4096), (4, 11008, 4096), (6, 4096, 11008)])
def test_config3_7b_layers_sampled_rows(idx, n, k, m):
    """Full-size layers in the launch configuration the benchmark times; the oracle checks a seeded
    sample of output rows (first, last, and rows spread over every tile)."""
    w = synth.bits_of(synth.weight(3, idx, n, k))
    x = synth.bits_of(synth.activations(3, idx, m, k))
    rng = np.random.default_rng(idx)
    rows = np.unique(np.concatenate([[0, 1, n - 1, n - 2], rng.integers(0, n, 700)])).astype(np.int64)
    run_case(w, x, rows=rows, what="config3 %dx%d M=%d" % (n, k, m))


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 8, 9, 12, 15, 16])
def test_every_token_count_on_a_ragged_shape(m):
    n, k = 203, 1440   # N not a multiple of any tile, K = 45 blocks
    w = synth.bits_of(synth.weight(3, 10, n, k))
    x = synth.bits_of(synth.activations(3, 10, m, k))
    run_case(w, x, what="ragged M=%d" % m)


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 8, 9, 12, 15, 16])
def test_every_token_count_on_a_ragged_shape_tensor_core_path(m):
    n, k = 203, 1408   # N not a multiple of 16, K = 44 blocks (a multiple of 128: tensor-core kernel)
    w = synth.bits_of(synth.weight(3, 14, n, k))
    x = synth.bits_of(synth.activations(3, 14, m, k))
    assert mxq.mxq_linear_plan_info(m, n, k)["kernel"] in ("fp4", "umma", "mma")
    run_case(w, x, what="ragged tc M=%d" % m)


@pytest.mark.parametrize("m,n,k", [(8, 4096, 11008), (16, 512, 13824), (16, 1000, 4096), (12, 333, 5120)])
def test_shapes_that_split_k_into_windows(m, n, k):
    assert mxq.mxq_linear_plan_info(m, n, k, "mma")["windows"] > 1
    w = synth.bits_of(synth.weight(3, 15, n, k))
    x = synth.bits_of(synth.activations(3, 15, m, k))
    rows = np.unique(np.concatenate([[0, n - 1], np.random.default_rng(5).integers(0, n, 200)])).astype(np.int64)
    run_case(w, x, rows=rows, what="windows %dx%d M=%d" % (n, k, m))


@pytest.mark.parametrize("n,k", [(1, 32), (2, 64), (7, 32), (9, 4096), (300, 96), (16, 13824), (129, 5120), (1, 128),
                                 (17, 128), (5000, 256)])
@pytest.mark.parametrize("m", [1, 3, 16])
def test_small_and_extreme_shapes(n, k, m):
    w = synth.bits_of(synth.weight(5, 2, n, k))
    x = synth.bits_of(synth.activations(5, 2, m, k))
    run_case(w, x, what="%dx%d M=%d" % (n, k, m))


@pytest.mark.parametrize("m", [1, 2, 4, 8, 16])
def test_config4_lm_head_sampled_rows(m):
    n, k = 32000, 4096
    w = synth.bits_of(synth.weight(4, 0, n, k))
    x = synth.bits_of(synth.activations(4, 0, m, k))
    rows = np.unique(np.concatenate([[0, n - 1], np.random.default_rng(4).integers(0, n, 300)])).astype(np.int64)
    run_case(w, x, rows=rows, what="lm_head M=%d" % m)


@pytest.mark.parametrize("m,n", [(1, 128256), (2, 128256), (4, 128256), (8, 128256), (16, 128256), (16, 50304), (3, 64000)])
def test_largest_vocabularies_sampled_rows(m, n):
    """The launch configurations of the largest projections bench.py times: one CTA per SM walking up to 14 tiles, the
    token operand resident or riding the ring.  Codes and scale bytes are drawn directly (seeded), so no cast of half a
    billion weights is needed; the oracle checks a seeded sample of rows from every part of the matrix."""
    k = 4096
    g = torch.Generator().manual_seed(1000 * 4 + m)
    codes = torch.randint(0, 256, (n, k // 2), dtype=torch.uint8, generator=g)
    scales = torch.randint(110, 126, (n, k // 32), dtype=torch.uint8, generator=g)
    x = synth.bits_of(synth.activations(4, 1, m, k))
    rows = np.unique(np.concatenate([[0, 1, 127, 128, n - 129, n - 128, n - 1],
                                     np.random.default_rng(m).integers(0, n, 250)])).astype(np.int64)
    y64, a64 = oracle.linear(x, codes.numpy(), scales.numpy(), rows=rows)
    ws = mxq.new_workspace(mxq.mxq_linear_workspace_bytes(m, n, k))
    y = mxq.mxq_linear(gpu_bf16(x), codes.cuda(), scales.cuda(), workspace=ws)
    torch.cuda.synchronize()
    check_linear(y[:, torch.as_tensor(rows, device="cuda")], y64, a64, "vocabulary %d M=%d" % (n, m))


@pytest.mark.parametrize("force", [0, 1])
@pytest.mark.parametrize("m,n,k", [(5, 203, 1408), (8, 4096, 4096), (16, 1000, 4096), (3, 300, 5120), (8, 32000, 4096), (16, 32000, 768)])
def test_token_operand_resident_and_through_the_ring(m, n, k, force):
    """With a workspace the FP8-operand kernel keeps the pre-split token operand of a CTA's whole K range in shared
    memory, or fetches it stage by stage into the ring slots; the layout heuristic picks one, mxq_set_linear_layout
    forces either.  Both must give the layer's result for every operand width, with one tile per CTA and with several."""
    mxq.mxq_set_linear_layout("operand_through_ring", force)
    prev = mxq.mxq_set_linear_kernel("umma")
    try:
        w = synth.bits_of(synth.weight(3, 16, n, k))
        x = synth.bits_of(synth.activations(3, 16, m, k))
        rows = None if n * k < 4e6 else np.unique(np.random.default_rng(3).integers(0, n, 250)).astype(np.int64)
        run_case(w, x, rows=rows, what="bring=%s" % force)
    finally:
        mxq.mxq_set_linear_kernel(prev)
        mxq.mxq_set_linear_layout("operand_through_ring", -1)


def test_bf16_output_is_the_rounded_fp32_output():
    w = synth.bits_of(synth.weight(3, 11, 515, 2048))
    x = synth.bits_of(synth.activations(3, 11, 5, 2048))
    _, y32 = run_case(w, x, torch.float32, what="fp32 out")
    _, y16 = run_case(w, x, torch.bfloat16, what="bf16 out")
    assert torch.equal(y16, y32.to(torch.bfloat16))   # round to nearest even of the same FP32 sums


def test_results_are_bit_reproducible():
    w = synth.bits_of(synth.weight(3, 12, 1000, 4096))
    for m in (1, 8):
        x = synth.bits_of(synth.activations(3, 12, m, 4096))
        _, y1 = run_case(w, x)
        _, y2 = run_case(w, x)
        assert torch.equal(y1, y2)


@pytest.mark.parametrize("m,n,k", [(3, 203, 1408), (8, 4096, 4096), (16, 1000, 4096), (6, 130, 1024), (16, 11008, 4096)])
def test_workspace_is_optional(m, n, k):
    """From 3 token rows on the FP8-operand kernel splits the token rows ahead of the weight kernel when it is given
    a workspace, and inside every CTA when it is not: the same parts, and the same sums in the same order whenever
    the two variants lay the work out alike (they may not: without the workspace a CTA keeps its whole K range of the
    token operand in shared memory, which can change the best decomposition)."""
    w = synth.bits_of(synth.weight(3, 15, n, k))
    x = synth.bits_of(synth.activations(3, 15, m, k))
    if (n, k) == (130, 1024):   # a K range that cannot be split exactly: both variants must take the scalar path
        x[2, 100] = 0x0001
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    need = mxq.mxq_linear_workspace_bytes(m, n, k)
    assert need > 0
    xg = gpu_bf16(x)
    y_ws = mxq.mxq_linear(xg, gc, gs, workspace=mxq.new_workspace(need))
    y_small = mxq.mxq_linear(xg, gc, gs, workspace=mxq.new_workspace(need - 16))   # too small: ignored
    y_reuse_ws = mxq.new_workspace(need + 4096)
    y_reuse_ws.fill_(0xFF)                                                          # contents are scratch
    y_dirty = mxq.mxq_linear(xg, gc, gs, workspace=y_reuse_ws[16:])                 # 16-byte aligned, not more
    torch.cuda.synchronize()
    assert torch.equal(y_ws, y_dirty)
    rows = None if n * k < 4e6 else np.unique(np.random.default_rng(2).integers(0, n, 200)).astype(np.int64)
    codes, scales, _ = oracle.quantize(w)
    y64, a64 = oracle.linear(x, codes, scales, rows=rows)
    for y, what in ((y_ws, "workspace"), (y_small, "no workspace")):
        check_linear(y if rows is None else y[:, torch.as_tensor(rows, device="cuda")], y64, a64, what)


def test_hand_block_a():
    blk = [b for b in direct_cast_blocks() if b["name"] == "A"][0]
    fx = linear_block_a()
    x = np.zeros((1, 32), np.float32)
    x[0, : len(fx["x"])] = fx["x"]
    xbits = (x.view(np.uint32) >> 16).astype(np.uint16)
    gc, gs = mxq.mxq_quantize(gpu_bf16(blk["bits"].reshape(1, 32)))
    y = mxq.mxq_linear(gpu_bf16(xbits), gc, gs)
    assert float(y[0, 0]) == fx["y"][0]   # every partial sum here is exact in FP32


def test_all_codes_under_extreme_scales():
    """Every code next to every scale byte the cast can produce (0..252), in one matrix; X picks out
    single weights so each output is one product."""
    n = 253
    codes = np.zeros((n, 16), np.uint8)
    for j in range(8):
        codes[:, j] = (2 * j) | ((2 * j + 1) << 4)
    scales = np.arange(n, dtype=np.uint8).reshape(n, 1)
    xs = np.zeros((16, 32), np.float32)
    xs[np.arange(16), np.arange(16)] = 1.0
    xbits = (xs.view(np.uint32) >> 16).astype(np.uint16)
    y64, a64 = oracle.linear(xbits, codes, scales)
    y = mxq.mxq_linear(gpu_bf16(xbits), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
    got = y.cpu().numpy().astype(np.float64)
    assert np.array_equal(got, y64)      # single exact products, FP32-representable: no tolerance needed


def test_nan_scale_gives_nan_row_only():
    w = synth.bits_of(synth.weight(1, 0, 64, 256))
    codes, scales, _ = oracle.quantize(w)
    scales[5, 3] = 0xFF
    x = synth.bits_of(synth.activations(1, 0, 2, 256))
    y64, a64 = oracle.linear(x, codes, scales)
    y = mxq.mxq_linear(gpu_bf16(x), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
    check_linear(y, y64, a64, "nan scale")
    assert torch.isnan(y[:, 5]).all() and torch.isfinite(y[:, :5]).all()


def test_wide_range_activations():
    """Activations spanning many binades, including BF16 subnormals and zeros: more than FP16 can hold
    next to the row maximum, so the tensor-core kernel must take its exact scalar path."""
    rng = np.random.default_rng(7)
    n, k, m = 130, 1024, 6
    w = synth.bits_of(synth.weight(3, 13, n, k))
    x = rng.standard_normal((m, k)) * np.exp2(rng.integers(-40, 30, (m, k)))
    x[0, ::3] = 0
    xbits = (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    xbits[1, :64] = (rng.integers(1, 128, 64) | (rng.integers(0, 2, 64) << 15)).astype(np.uint16)  # subnormals
    run_case(w, xbits, what="wide range")


def test_host_variant_matches_device_variant():
    n, k, m = 768, 3072, 4
    w = synth.bits_of(synth.weight(2, 6, n, k))
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    x = synth.activations(2, 6, m, k)
    y_dev = mxq.mxq_linear(x.cuda(), gc, gs)
    xh = x.pin_memory()
    yh = torch.empty((m, n), dtype=torch.float32).pin_memory()
    mxq.mxq_linear_host(xh, gc, gs, yh, torch.empty_like(x, device="cuda"),
                        torch.empty((m, n), dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(yh, y_dev.cpu())


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("m,n,k,dtype", [(1, 4096, 4096, torch.float32), (8, 1000, 2048, torch.bfloat16), (16, 203, 1408, torch.float32)])
def test_host_variant_pinned_and_pageable(m, n, k, dtype, pinned):
    """Page-locked buffers are moved by the GPU itself (a staging kernel for X, Y stored straight into host memory),
    pageable ones by the copy engine: the same bits either way, and nothing written around Y."""
    w = synth.bits_of(synth.weight(3, 21, n, k))
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    x = synth.activations(3, 21, m, k)
    y_dev = mxq.mxq_linear(x.cuda(), gc, gs, out_dtype=dtype)
    buf = torch.full((m * n + 64,), 3.0, dtype=dtype)
    xh = x.clone()
    if pinned:
        buf, xh = buf.pin_memory(), xh.pin_memory()
    yh = buf[32:32 + m * n].view(m, n)
    for _ in range(2):   # twice: the second call's staging must wait for the first call's reads
        mxq.mxq_linear_host(xh, gc, gs, yh, torch.empty_like(x, device="cuda"), torch.empty((m, n), dtype=dtype, device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(yh, y_dev.cpu())
    assert (buf[:32] == 3.0).all() and (buf[32 + m * n:] == 3.0).all()


def test_canaries_around_the_output_survive():
    n, k, m = 203, 1440, 3
    w = synth.bits_of(synth.weight(3, 10, n, k))
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    x = synth.activations(3, 10, m, k).cuda()
    buf = torch.full((m * n + 64,), 12345.0, dtype=torch.float32, device="cuda")
    out = buf[32: 32 + m * n].view(m, n)
    mxq.mxq_linear(x, gc, gs, out=out)
    torch.cuda.synchronize()
    assert (buf[:32] == 12345.0).all() and (buf[32 + m * n:] == 12345.0).all()


# ---- the launch plans bench.py times on the 13B layer shapes, the paper's 8192 x 8192 and the fused q/k/v matrix -------

import functools


@functools.lru_cache(maxsize=2)
def _big_case(idx, n, k):
    """Weights of one full-size matrix, cast by the oracle once and shared by the token counts (and kernel settings)."""
    w = synth.bits_of(synth.weight(5 if k in (5120, 13824) else 3, idx, n, k))
    codes, scales, _ = oracle.quantize(w)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, n - 129, n - 128, n - 1],
                                     np.random.default_rng(idx).integers(0, n, 160)])).astype(np.int64)
    return codes, scales, rows, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()


def _run_big(idx, n, k, m):
    codes, scales, rows, gc, gs = _big_case(idx, n, k)
    x = synth.bits_of(synth.activations(5, idx, m, k))
    y64, a64 = oracle.linear(x, codes, scales, rows=rows)
    ws = mxq.new_workspace(mxq.mxq_linear_workspace_bytes(m, n, k))
    y = mxq.mxq_linear(gpu_bf16(x), gc, gs, workspace=ws)
    torch.cuda.synchronize()
    check_linear(y[:, torch.as_tensor(rows, device="cuda")], y64, a64, "%dx%d M=%d" % (n, k, m))


@pytest.mark.parametrize("m", list(range(1, 17)))
@pytest.mark.parametrize("idx,n,k", [(0, 5120, 5120), (4, 13824, 5120), (6, 5120, 13824)])
def test_config5_13b_layer_shapes_every_token_count(idx, n, k, m):
    """Config 5: the three 13B layer shapes at every M in 1..16, in the launch plans the benchmark's curves time
    (e.g. 13824 x 5120 as 540 CTAs on 592 slots); sampled rows spread over the first, the last and random tiles."""
    _run_big(idx, n, k, m)


@pytest.mark.parametrize("m", [1, 8])
@pytest.mark.parametrize("idx,n,k", [(20, 8192, 8192), (21, 12288, 4096), (22, 22016, 4096)])
def test_micro_benchmark_and_fused_projection_shapes(idx, n, k, m):
    """8192 x 8192 (the paper's micro-benchmark shape) and the fused q/k/v (12288 x 4096) and gate/up (22016 x 4096)
    matrices of the four-call layer, as bench.py times them."""
    _run_big(idx, n, k, m)
