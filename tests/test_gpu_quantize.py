"""GPU parity of mxq_quantize / mxq_dequantize against the oracle: bytes must be identical."""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from golden_io import direct_cast_blocks
from paper_2503_13565_b200 import synth
from parity import gpu_bf16, to_np_u8

pytestmark = pytest.mark.gpu


def quantize_both(bits: np.ndarray):
    oc, os_, obad = oracle.quantize(bits)
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    gc, gs = mxq.mxq_quantize(gpu_bf16(bits), nonfinite_blocks=cnt)
    torch.cuda.synchronize()
    return (oc, os_, obad), (to_np_u8(gc), to_np_u8(gs), int(cnt.item()))


def assert_same(o, g):
    assert np.array_equal(o[1], g[1]), "scales differ at %s" % (np.argwhere(o[1] != g[1])[:5],)
    assert np.array_equal(o[0], g[0]), "codes differ at %s" % (np.argwhere(o[0] != g[0])[:5],)
    assert o[2] == g[2]


def test_config1_tiny():
    bits = synth.bits_of(synth.weight(1, 0, 512, 256))
    assert_same(*quantize_both(bits))


@pytest.mark.parametrize("idx,n,k", [(0, 768, 768), (4, 3072, 768), (6, 768, 3072), (7, 32000, 768)])
def test_config2_small_draft_layers(idx, n, k):
    bits = synth.bits_of(synth.weight(2, idx, n, k))
    assert_same(*quantize_both(bits))


@pytest.mark.parametrize("n,k", [(1, 32), (3, 64), (5, 96), (1, 4096), (37, 11008), (4096, 4096)])
def test_config3_shapes_and_ragged_sizes(n, k):
    bits = synth.bits_of(synth.weight(3, 0, n, k))
    assert_same(*quantize_both(bits))


def test_config5_injected_zero_and_subnormal_blocks():
    w = synth.weight(5, 0, 1024, 5120)
    bits = synth.bits_of(w)
    o, g = quantize_both(bits)
    assert_same(o, g)
    assert (o[1] == 0).sum() > 50 and (o[1] == 1).sum() >= 1   # the injection really produced bytes 0 and 1


def test_hand_blocks():
    blocks = direct_cast_blocks()
    bits = np.stack([b["bits"] for b in blocks])
    o, g = quantize_both(bits)
    assert_same(o, g)
    for i, b in enumerate(blocks):
        assert g[1][i, 0] == b["scale"]
        assert list(g[0][i, : len(b["bytes"])]) == b["bytes"]


def test_every_bf16_value_under_every_scale():
    """Exhaustive: for each shared exponent the cast can produce, every finite BF16 pattern that can
    share a block with it, 31 per block next to an element that pins the block maximum."""
    finite = np.array([b for b in range(1 << 16) if (b >> 7) & 0xFF != 0xFF], np.uint16)
    exp_field = (finite.astype(np.int64) >> 7) & 0xFF
    chunks = []
    for se in range(-127, 126):
        top_field = se + 2 + 127
        cand = finite[exp_field <= top_field]
        pad = (-len(cand)) % 31
        vals = np.concatenate([cand, np.zeros(pad, np.uint16)]).reshape(-1, 31)
        blocks = np.empty((vals.shape[0], 32), np.uint16)
        blocks[:, 0] = np.uint16(top_field << 7)
        blocks[:, 1:] = vals
        chunks.append(blocks)
    bits = np.concatenate(chunks)
    # shuffle the block maximum's position so that every lane of a quad gets to hold it
    rng = np.random.default_rng(0)
    pos = rng.integers(0, 32, bits.shape[0])
    rows = np.arange(bits.shape[0])
    tmp = bits[rows, pos].copy()
    bits[rows, pos] = bits[rows, 0]
    bits[rows, 0] = tmp
    o, g = quantize_both(bits)
    assert_same(o, g)
    assert bits.size > 8_000_000


def test_nonfinite_blocks_and_counter():
    bits = synth.bits_of(synth.weight(1, 0, 64, 256)).copy()
    bits[3, 40] = 0x7F80
    bits[3, 41] = 0xFF80
    bits[9, 255] = 0x7FC1
    bits[63, 0] = 0xFFFF
    o, g = quantize_both(bits)
    assert_same(o, g)
    assert g[2] == 3


def test_dequantize_is_exact():
    rng = np.random.default_rng(1)
    codes = rng.integers(0, 256, (33, 160), dtype=np.uint8)
    scales = rng.integers(0, 253, (33, 10), dtype=np.uint8)
    scales[0, 0], scales[1, 1] = 0, 252
    scales[2, 2] = 0xFF
    want = oracle.dequantize(codes, scales)
    got = mxq.mxq_dequantize(torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda())
    got = got.float().cpu().numpy().astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(got[~nan], want[~nan]) and np.isnan(got[nan]).all()
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_quantize_then_dequantize_matches_oracle_values():
    bits = synth.bits_of(synth.weight(2, 1, 768, 768))
    gc, gs = mxq.mxq_quantize(gpu_bf16(bits))
    got = mxq.mxq_dequantize(gc, gs).float().cpu().numpy().astype(np.float64)
    oc, os_, _ = oracle.quantize(bits)
    assert np.array_equal(got, oracle.dequantize(oc, os_))


def test_config5_direct_cast_of_all_forty_13b_layers():
    """Config 5 at scale: the 40 x 7 weight matrices of a 13B-shaped model (12.69 G weights: q, k, v, o 5120 x 5120;
    gate, up 13824 x 5120; down 5120 x 13824), Student-t with zeroed blocks, blocks pushed into the BF16 subnormals
    and the hand blocks planted, drawn on the GPU from per-matrix seeds.  Every matrix is cast by mxq_quantize and by
    the oracle from the same bits; codes, scales and the non-finite counter must agree byte for byte, layer by layer.
    (One block per layer is overwritten with an Inf and a NaN here, so that the counter is exercised at scale too.)"""
    shapes = [(n, k) for _, n, k in synth.LAYERS_13B]
    total = 0
    for layer in range(40):
        for j, (n, k) in enumerate(shapes):
            w = synth.weight(5, 100 + layer * len(shapes) + j, n, k, device="cuda")
            if j == layer % len(shapes):
                blk = w.view(-1, 32)
                blk[(layer * 7919 + 13) % blk.shape[0], 3] = float("inf")
                blk[(layer * 104729 + 5) % blk.shape[0], 31] = float("nan")
            cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
            gc, gs = mxq.mxq_quantize(w, nonfinite_blocks=cnt)
            bits = synth.bits_of(w)
            oc, os_, obad = oracle.quantize(bits)
            torch.cuda.synchronize()
            assert np.array_equal(os_, to_np_u8(gs)), "scales differ in layer %d matrix %d" % (layer, j)
            assert np.array_equal(oc, to_np_u8(gc)), "codes differ in layer %d matrix %d" % (layer, j)
            assert obad == int(cnt.item()), "non-finite counter differs in layer %d matrix %d" % (layer, j)
            total += n * k
            del w, gc, gs, bits, oc, os_
    assert total == 40 * 317194240
