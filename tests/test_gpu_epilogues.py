"""GPU parity of the fused layer epilogues (mxq_linear_residual, mxq_linear_swiglu) against their oracles.

Bounds, element by element, with t(A) = 2e-3 * A + 1e-6 the plain layer's tolerance on a sum whose sum_k |x w^| is A:
  residual   |y - (r + y64)| <= t(A) + 2^-23 |r + y64|                      (one more FP32 addition)
  gate / up  |y - silu(g) u| <= 1.1 t(A_g) (|u| + t(A_u)) + |silu(g)| t(A_u) + 1e-6 |silu(g) u| + 1e-30
             (|silu'| < 1.1 everywhere; the exponential, the quotient and the product are FP32 operations)
A BF16 output adds 2^-8 of the exact value (one rounding to 8 significant bits).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth
from parity import ABS, REL, gpu_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["auto", "fp4", "umma", "mma"])
def linear_kernel(request):
    """Every case runs with the library's own choice of kernel and with the choice capped at each tcgen05 kernel (the
    epilogue then runs inside it) and at the mma.sync kernel (the sums pass through the workspace)."""
    prev = mxq.mxq_set_linear_kernel(request.param)
    yield request.param
    mxq.mxq_set_linear_kernel(prev)
    assert mxq.mxq_linear_device_status() == 0, "a bounded wait inside the tcgen05 kernel gave up"


def values(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def within(got, want, tol, out_dtype, what):
    tol = tol + (np.abs(want) * 2.0 ** -8 if out_dtype == torch.bfloat16 else 0.0)
    assert np.isfinite(got).all(), what
    worst = float((np.abs(got - want) / tol).max())
    assert worst <= 1.0, "%s: error/tolerance = %.3g" % (what, worst)


def quantised(cfg, idx, n, k):
    codes, scales, _ = oracle.quantize(synth.bits_of(synth.weight(cfg, idx, n, k)))
    return codes, scales


def run_residual(m, n, k, idx, out_dtype=torch.float32, rows=None, in_place=False):
    codes, scales = quantised(3, idx, n, k)
    x = synth.bits_of(synth.activations(3, idx, m, k))
    g = torch.Generator().manual_seed(100 + idx)
    res = (torch.randn(m, n, generator=g) * 0.5).to(out_dtype).cuda()
    r64 = values(res)
    sel = slice(None) if rows is None else np.asarray(rows)
    want, a = oracle.linear_residual(x, codes, scales, r64[:, sel], rows=rows)
    out = res.clone() if in_place else None
    y = mxq.mxq_linear_residual(gpu_bf16(x), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(),
                                out if in_place else res, out=out)
    torch.cuda.synchronize()
    assert y.dtype == out_dtype and y.shape == (m, n)
    if not in_place:
        assert torch.equal(res, torch.from_numpy(r64).to(out_dtype).cuda()), "the residual was written to"
    within(values(y)[:, sel], want, REL * a + ABS + 2.0 ** -23 * np.abs(want), out_dtype,
           "residual %dx%d M=%d" % (n, k, m))
    return y


def run_swiglu(m, f, k, idx, out_dtype=torch.bfloat16, rows=None):
    codes, scales = quantised(3, idx, 2 * f, k)
    x = synth.bits_of(synth.activations(3, idx, m, k))
    want, g, u, ag, au = oracle.linear_swiglu(x, codes, scales, rows=rows)
    y = mxq.mxq_linear_swiglu(gpu_bf16(x), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(),
                              out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert y.dtype == out_dtype and y.shape == (m, f)
    tg, tu = REL * ag + ABS, REL * au + ABS
    tol = 1.1 * tg * (np.abs(u) + tu) + np.abs(oracle.silu(g)) * tu + 1e-6 * np.abs(want) + 1e-30
    got = values(y) if rows is None else values(y)[:, np.asarray(rows)]
    within(got, want, tol, out_dtype, "swiglu F=%d K=%d M=%d" % (f, k, m))
    return y


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 8, 9, 16])
def test_residual_ragged_shape(m):
    run_residual(m, 203, 1408, idx=m)          # K = 11 stages of 128: odd cluster sizes; N not a multiple of a tile


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 8, 9, 16])
def test_swiglu_ragged_shape(m):
    run_swiglu(m, 203, 1408, idx=m)            # 406 weight rows: the last tile is ragged, pairs never straddle it


@pytest.mark.parametrize("m", [1, 4, 7])
@pytest.mark.parametrize("f,k", [(64, 128), (1, 128), (300, 256), (1000, 2048), (515, 96)])
def test_swiglu_small_shapes(f, k, m):
    """One stage (no cluster), one pair, two stages, many tiles with a power-of-two cluster, and a K outside the
    tensor-core kernels (the sums pass through the workspace)."""
    run_swiglu(m, f, k, idx=3, out_dtype=torch.float32)


@pytest.mark.parametrize("m", [1, 4, 7])
@pytest.mark.parametrize("n,k", [(64, 128), (1, 128), (300, 256), (1000, 2048), (515, 96)])
def test_residual_small_shapes(n, k, m):
    run_residual(m, n, k, idx=4, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("m", [1, 8])
def test_7b_feed_forward_sampled_rows(m):
    """The 7B feed-forward block as the benchmark runs it: gate / up as one 22016 x 4096 matrix, down with the residual."""
    rows = np.unique(np.concatenate([[0, 1, 11006, 11007], np.random.default_rng(1).integers(0, 11008, 300)])).astype(np.int64)
    run_swiglu(m, 11008, 4096, idx=4, rows=rows)
    rows = np.unique(np.concatenate([[0, 4095], np.random.default_rng(2).integers(0, 4096, 300)])).astype(np.int64)
    run_residual(m, 4096, 11008, idx=6, out_dtype=torch.bfloat16, rows=rows)
    run_residual(m, 4096, 4096, idx=0, out_dtype=torch.float32, rows=rows)


@pytest.mark.parametrize("m", [1, 3])
def test_many_tiles_per_cta(m):
    """Vocabulary-sized N: a CTA walks several tiles (the epilogue runs tile by tile)."""
    rows = np.unique(np.random.default_rng(3).integers(0, 20000, 400)).astype(np.int64)
    run_swiglu(m, 20000, 768, idx=7, rows=rows, out_dtype=torch.float32)
    rows = np.unique(np.random.default_rng(4).integers(0, 40000, 400)).astype(np.int64)
    run_residual(m, 40000, 768, idx=7, rows=rows)


def test_residual_in_place_and_equal_to_the_plain_layer_plus_the_residual():
    """Y may be the residual itself; and, the decomposition being the plain layer's, the fused FP32 result is the plain
    layer's FP32 result plus the residual, bit for bit."""
    for m, n, k in [(1, 4096, 4096), (8, 1000, 2048), (2, 203, 1408)]:
        y = run_residual(m, n, k, idx=5)
        z = run_residual(m, n, k, idx=5, in_place=True)
        assert torch.equal(y, z)
        codes, scales = quantised(3, 5, n, k)
        x = synth.bits_of(synth.activations(3, 5, m, k))
        ws = mxq.new_workspace(mxq.mxq_linear_workspace_bytes(m, n, k))
        plain = mxq.mxq_linear(gpu_bf16(x), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(), workspace=ws)
        g = torch.Generator().manual_seed(105)
        res = (torch.randn(m, n, generator=g) * 0.5).cuda()
        assert torch.equal(y, plain + res)


def test_canaries_and_workspace_contract():
    m, f, k = 4, 515, 2048
    codes, scales = quantised(3, 8, 2 * f, k)
    x = gpu_bf16(synth.bits_of(synth.activations(3, 8, m, k)))
    c, s = torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()
    buf = torch.full((m * f + 64,), 777.0, dtype=torch.float32, device="cuda")
    need = mxq.mxq_linear_fused_workspace_bytes(m, 2 * f, k)
    ws = torch.full((need + 512,), 0xAB, dtype=torch.uint8, device="cuda")      # a dirty workspace, with a canary behind it
    y = mxq.mxq_linear_swiglu(x, c, s, out=buf[32:32 + m * f].view(m, f), workspace=ws[:need])
    torch.cuda.synchronize()
    assert (buf[:32] == 777.0).all() and (buf[32 + m * f:] == 777.0).all()
    assert (ws[need:] == 0xAB).all()
    assert torch.equal(y, mxq.mxq_linear_swiglu(x, c, s, out_dtype=torch.float32))   # reproducible, whatever the workspace held
    with pytest.raises(mxq.MxqError):
        mxq.mxq_linear_swiglu(x, c, s, workspace=ws[:need - 256])
    with pytest.raises(mxq.MxqError):
        mxq.mxq_linear_swiglu(x, c[:-1], s[:-1])                                     # an odd number of weight rows
