"""Pins for the oracle's direct cast and dequantisation (CPU only).

Each test checks the oracle against something that is not the oracle: the
hand-written fixtures, exact integer / rational arithmetic, closed forms, or
invariants of the format.  Section references are to the paper (Sec. III-D-3).
"""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from golden_io import direct_cast_blocks, e2m1_values

GRID2 = np.array([0, 1, 2, 3, 4, 6, 8, 12], np.int64)  # twice the E2M1 magnitudes, as integers


def f32_to_bf16_bits(x):
    """float32 values that are exactly BF16-representable -> uint16 bits (asserts exactness)."""
    u = np.asarray(x, np.float32).view(np.uint32)
    assert not (u & 0xFFFF).any(), "value is not BF16-representable"
    return (u >> 16).astype(np.uint16)


def bits_to_f64(b):
    return (np.asarray(b, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def unpack_codes(codes):
    c = np.asarray(codes, np.uint8)
    out = np.empty(c.shape[:-1] + (c.shape[-1] * 2,), np.uint8)
    out[..., 0::2] = c & 0xF
    out[..., 1::2] = c >> 4
    return out


def bits_fraction(b):
    """BF16 bit pattern -> exact Fraction (finite patterns only)."""
    b = int(b)
    s, e, m = b >> 15, (b >> 7) & 0xFF, b & 0x7F
    assert e != 0xFF
    mag = Fraction(m, 128) * Fraction(2) ** (-126) if e == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -mag if s else mag


# ---- value set -----------------------------------------------------------------


def test_value_set_matches_fixture():
    want = e2m1_values()
    codes = np.zeros((1, 16), np.uint8)
    for j in range(8):
        codes[0, j] = (2 * j) | ((2 * j + 1) << 4)
    scales = np.full((1, 1), 127, np.uint8)
    got = oracle.dequantize(codes, scales)[0, :16]
    for c in range(16):
        assert got[c] == want[c], (c, got[c], want[c])
        assert np.signbit(got[c]) == np.signbit(want[c])
    assert sorted(set(abs(got))) == [0, 0.5, 1, 1.5, 2, 3, 4, 6]


@pytest.mark.parametrize("byte", [0, 1, 2, 100, 126, 127, 128, 200, 252, 253, 254])
def test_scale_byte_is_a_biased_exponent(byte):
    codes = np.zeros((1, 16), np.uint8)
    codes[0, 0] = 0x2 | (0xF << 4)  # +1, -6
    got = oracle.dequantize(codes, np.full((1, 1), byte, np.uint8))
    assert Fraction(got[0, 0]) == Fraction(2) ** (byte - 127)
    assert Fraction(got[0, 1]) == -6 * Fraction(2) ** (byte - 127)


def test_scale_byte_ff_is_nan():
    got = oracle.dequantize(np.zeros((1, 16), np.uint8), np.full((1, 1), 0xFF, np.uint8))
    assert np.isnan(got).all()


# ---- hand-worked blocks ------------------------------------------------------------


@pytest.mark.parametrize("blk", direct_cast_blocks(), ids=lambda b: b["name"])
def test_hand_blocks(blk):
    codes, scales, bad = oracle.quantize(blk["bits"].reshape(1, 32))
    assert bad == 0
    assert int(scales[0, 0]) == blk["scale"]
    got = unpack_codes(codes)[0]
    n = len(blk["codes"])
    assert list(got[:n]) == blk["codes"]
    assert not got[n:].any()
    assert list(codes[0, : len(blk["bytes"])]) == blk["bytes"]


# ---- brute force over every BF16 value and every scale ------------------------------


def expected_codes_nearest(bits, se):
    """Nearest E2M1 neighbour of |v| / 2^se by exact integer comparison, ties to the even code,
    anything above 6 clamps; sign bit copied.  bits: uint16 array; se: scalar shared exponent."""
    b = bits.astype(np.int64)
    sign = (b >> 15) & 1
    e = (b >> 7) & 0xFF
    m = b & 0x7F
    mant = np.where(e == 0, m, 128 + m)            # |v| = mant * 2^p
    p = np.where(e == 0, -133, e - 134)
    sh = p - se + 1                                 # 2|v|/2^se = mant * 2^sh
    code = np.zeros(b.shape, np.int64)
    tiny = sh < -20                                 # 2r < 256 * 2^-21: rounds to 0
    big = sh > 8
    ok = ~tiny & ~big
    up = np.clip(sh, 0, 8)
    dn = np.clip(-sh, 0, 20)
    lhs = mant << up                                # compare lhs against GRID2 << dn
    best = np.full(b.shape, -1, np.int64)
    bestd = np.full(b.shape, np.iinfo(np.int64).max, np.int64)
    for j in range(8):
        d = np.abs(lhs - (GRID2[j] << dn))
        better = (d < bestd) | ((d == bestd) & (j % 2 == 0) & (best % 2 == 1))
        best = np.where(better, j, best)
        bestd = np.where(better, d, bestd)
    over = lhs > (12 << dn)
    best = np.where(over, 7, best)
    code = np.where(ok, best, code)
    code = np.where(big & (mant > 0), 7, code)
    return (code | (sign << 3)).astype(np.uint8)


def test_rounding_brute_force_all_values_all_scales():
    """Every finite BF16 pattern that can share a block with a given scale, for every scale the
    cast can produce (shared exponent -127..125): the oracle's rounding agrees with an exact
    nearest-neighbour search."""
    finite = np.array([b for b in range(1 << 16) if (b >> 7) & 0xFF != 0xFF], np.uint16)
    exp_field = (finite.astype(np.int64) >> 7) & 0xFF
    total = 0
    for se in range(-127, 126):
        # the block maximum is 2^(se+2) (bits: exponent field se+2+127), unless the clamp binds
        top_field = se + 2 + 127
        setter = np.uint16(top_field << 7)           # exactly 4 * 2^se
        cand = finite[exp_field <= top_field] if se > -127 else finite[exp_field <= 2]
        if se == -127:
            setter = np.uint16(2 << 7)               # 2^-125 = 4 * 2^-127
        pad = (-len(cand)) % 31
        vals = np.concatenate([cand, np.zeros(pad, np.uint16)]).reshape(-1, 31)
        blocks = np.empty((vals.shape[0], 32), np.uint16)
        blocks[:, 0] = setter
        blocks[:, 1:] = vals
        codes, scales, bad = oracle.quantize(blocks)
        assert bad == 0
        assert (scales == se + 127).all(), se
        got = unpack_codes(codes)
        assert (got[:, 0] == 6).all()
        want = expected_codes_nearest(vals.reshape(-1), se).reshape(-1, 31)
        assert np.array_equal(got[:, 1:], want), se
        total += vals.size
    assert total > 8_000_000


def test_rounding_ties_go_to_even_code():
    # scaled values 0.25 0.75 1.25 1.75 2.5 3.5 5.0 and the block maximum 4 (scale byte 127)
    v = np.array([4, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -5.0] + [0] * 21, np.float32)
    codes, scales, _ = oracle.quantize(f32_to_bf16_bits(v).reshape(1, 32))
    assert scales[0, 0] == 127
    assert list(unpack_codes(codes)[0, :11]) == [6, 0, 2, 2, 4, 4, 6, 6, 8, 0xA, 0xE]


# ---- scale closed form ---------------------------------------------------------------


def test_scale_closed_form_for_every_positive_value():
    """A block whose only non-zero is a: byte = max(floor(log2 a) - 2, -127) + 127, with floor(log2 a)
    read off the bit fields (normal: exponent field - 127; subnormal m*2^-133: bit length of m - 134)."""
    pats = np.array([b for b in range(1, 0x7F80)], np.uint16)
    blocks = np.zeros((pats.size, 32), np.uint16)
    blocks[:, 7] = pats
    _, scales, _ = oracle.quantize(blocks)
    e = pats.astype(np.int64) >> 7
    m = pats.astype(np.int64) & 0x7F
    bitlen = np.floor(np.log2(np.maximum(m, 1))).astype(np.int64)  # exact for 1..127
    flog = np.where(e == 0, bitlen - 133, e - 127)
    want = np.maximum(flog - 2, -127) + 127
    assert np.array_equal(scales[:, 0].astype(np.int64), want)
    # a negative maximum gives the same scale
    blocks[:, 7] |= 0x8000
    _, scales2, _ = oracle.quantize(blocks)
    assert np.array_equal(scales, scales2)


def test_block_maximum_lands_on_4_or_6():
    rng = np.random.default_rng(1)
    w = (rng.standard_normal((64, 256)) * 0.02).astype(np.float32)
    bits = (w.view(np.uint32) >> 16).astype(np.uint16)  # truncation is fine: any BF16 input will do
    codes, scales, _ = oracle.quantize(bits)
    mags = (unpack_codes(codes) & 7).reshape(64, 8, 32).max(axis=2)
    assert set(np.unique(mags)) <= {6, 7}


# ---- invariants ------------------------------------------------------------------------


def random_bf16(rng, shape, spread=6.0):
    x = rng.standard_normal(shape) * np.exp2(rng.integers(-int(spread), int(spread), shape))
    return (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_round_trip_of_representable_blocks():
    """Blocks made of grid values times a power of two survive quantise -> dequantise unchanged,
    provided the block maximum is 4 or 6 times the scale (as the cast itself always produces)."""
    rng = np.random.default_rng(2)
    n, k = 97, 160
    codes = rng.integers(0, 256, (n, k // 2), dtype=np.uint8)
    # force one element per block to magnitude 4 or 6 so the scale is recovered
    cu = unpack_codes(codes).reshape(n, k // 32, 32)
    cu[:, :, 3] = rng.choice(np.array([6, 7, 14, 15], np.uint8), (n, k // 32))
    cu = cu.reshape(n, k)
    codes = (cu[:, 0::2] | (cu[:, 1::2] << 4)).astype(np.uint8)
    scales = rng.integers(0, 253, (n, k // 32), dtype=np.uint8)
    w = oracle.dequantize(codes, scales)
    bits = f32_to_bf16_bits(w.astype(np.float32))
    assert np.array_equal(bits_to_f64(bits), w)
    codes2, scales2, bad = oracle.quantize(bits)
    assert bad == 0
    assert np.array_equal(scales2, scales)
    assert np.array_equal(codes2, codes)


def test_idempotence():
    rng = np.random.default_rng(3)
    bits = random_bf16(rng, (50, 320))
    bits[0, :32] = 0
    bits[1, 5] = 0x8000
    bits[2, :32] = random_bf16(rng, 32) & 0x807F  # BF16 subnormals
    codes, scales, _ = oracle.quantize(bits)
    w = oracle.dequantize(codes, scales)
    bits2 = f32_to_bf16_bits(w.astype(np.float32))
    codes2, scales2, _ = oracle.quantize(bits2)
    assert np.array_equal(codes2, codes)
    # the scale is reproduced wherever the block is not all zero after the cast
    nonzero = (unpack_codes(codes) & 7).reshape(50, 10, 32).any(axis=2)
    assert np.array_equal(scales2[nonzero], scales[nonzero])
    assert (scales2[~nonzero] == 0).all()


def test_error_bound():
    """|w^ - v| <= half a grid step (times X) below the clamp, < 2X above it."""
    rng = np.random.default_rng(4)
    bits = random_bf16(rng, (40, 512), spread=3)
    codes, scales, _ = oracle.quantize(bits)
    v = bits_to_f64(bits)
    w = oracle.dequantize(codes, scales)
    x = np.repeat(np.exp2(scales.astype(np.float64) - 127), 32, axis=1)
    r = np.abs(v) / x
    err = np.abs(w - v) / x
    assert (r < 8).all()
    assert (err[r < 2] <= 0.25).all()
    assert (err[(r >= 2) & (r < 4)] <= 0.5).all()
    assert (err[(r >= 4) & (r <= 6)] <= 1.0).all()
    assert (err[r > 6] < 2.0).all()
    assert (np.sign(w) * np.sign(v) >= 0).all()


def test_random_blocks_against_rational_arithmetic():
    """Whole cast, both steps, against a Fraction-based restatement on a few hundred blocks."""
    rng = np.random.default_rng(5)
    bits = random_bf16(rng, (6, 64), spread=4)
    bits[0, :32] = random_bf16(rng, 32) & 0x807F
    codes, scales, _ = oracle.quantize(bits)
    got = unpack_codes(codes)
    grid = [Fraction(g, 2) for g in GRID2.tolist()]
    for n in range(bits.shape[0]):
        for j in range(bits.shape[1] // 32):
            vals = [bits_fraction(b) for b in bits[n, 32 * j: 32 * j + 32]]
            amax = max(abs(v) for v in vals)
            se = -127
            if amax > 0:
                fl = 0
                while Fraction(2) ** (fl + 1) <= amax:
                    fl += 1
                while Fraction(2) ** fl > amax:
                    fl -= 1
                se = max(fl - 2, -127)
            assert scales[n, j] == se + 127
            for i, v in enumerate(vals):
                r = abs(v) / Fraction(2) ** se
                if r > 6:
                    c = 7
                else:
                    dist = [abs(r - g) for g in grid]
                    dmin = min(dist)
                    cands = [c for c in range(8) if dist[c] == dmin]
                    c = cands[0] if len(cands) == 1 else [c for c in cands if c % 2 == 0][0]
                sign = int(bits[n, 32 * j + i]) >> 15
                assert got[n, 32 * j + i] == (sign << 3 | c)


def test_nonfinite_blocks():
    bits = np.zeros((2, 64), np.uint16)
    bits[0, :32] = (np.linspace(-1, 1, 32, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)
    bits[0, 40] = 0x7F80   # +Inf
    bits[1, 3] = 0xFFC0    # NaN
    bits[1, 33] = 0x3F80
    codes, scales, bad = oracle.quantize(bits)
    assert bad == 2
    assert scales[0, 1] == 0xFF and scales[1, 0] == 0xFF
    assert not codes[0, 16:].any() and not codes[1, :16].any()
    assert scales[0, 0] != 0xFF and scales[1, 1] == 125  # 1.0 -> 2^(0-2)


def test_storage_is_4_25_bits_per_weight():
    n, k = 24, 1024
    codes, scales, _ = oracle.quantize(np.zeros((n, k), np.uint16))
    assert (codes.nbytes + scales.nbytes) * 8 == n * k * 4.25
    assert abs(n * k * 2 / (codes.nbytes + scales.nbytes) - 3.7647) < 1e-4  # the paper's 3.76x


def test_layout_even_element_in_low_nibble():
    v = np.zeros((1, 64), np.float32)
    v[0, 0], v[0, 1], v[0, 33] = 4.0, -1.0, 6.0
    codes, scales, _ = oracle.quantize(f32_to_bf16_bits(v))
    assert codes[0, 0] == (6 | (0xA << 4))
    assert codes[0, 16] == (0 | (7 << 4))
    assert codes.shape == (1, 32) and scales.shape == (1, 2)
