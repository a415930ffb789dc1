"""Pins for the oracle's linear layer Y = X . dequant(W)^T (CPU only).

The oracle is the plain definition (Sec. III-D-3; Eq. 2 allows the scale to be
applied per element or per 32-long partial sum).  It is checked against exact
integer / rational arithmetic, a hand-worked block, and a library matrix
product over an independently decoded weight matrix.
"""
from fractions import Fraction

import numpy as np

import oracle
from golden_io import direct_cast_blocks, e2m1_values, linear_block_a
from test_oracle_quantize import bits_fraction, bits_to_f64, f32_to_bf16_bits, unpack_codes


def pack(cu):
    return (cu[:, 0::2] | (cu[:, 1::2] << 4)).astype(np.uint8)


def decode_with_fixture(codes, scales):
    """Independent decode: value table from the hand-written fixture, scale by exp2."""
    table = np.array([e2m1_values()[c] for c in range(16)], np.float64)
    w = table[unpack_codes(codes)]
    return w * np.repeat(np.exp2(scales.astype(np.float64) - 127.0), 32, axis=1)


def test_hand_block_a_dot_product():
    blk = [b for b in direct_cast_blocks() if b["name"] == "A"][0]
    fx = linear_block_a()
    codes, scales, _ = oracle.quantize(blk["bits"].reshape(1, 32))
    x = np.zeros((1, 32), np.float32)
    x[0, : len(fx["x"])] = fx["x"]
    y, a = oracle.linear(f32_to_bf16_bits(x), codes, scales)
    assert y[0, 0] == fx["y"][0]
    assert a[0, 0] == fx["sum_abs"][0]


def test_all_ones_counts_k_and_alternating_signs_cancel():
    n, k = 5, 256
    cu = np.full((n, k), 2, np.uint8)  # +1.0
    x = f32_to_bf16_bits(np.ones((3, k), np.float32))
    s = np.full((n, k // 32), 127, np.uint8)
    y, a = oracle.linear(x, pack(cu), s)
    assert (y == k).all() and (a == k).all()
    cu[:, 1::2] = 0xA  # -1.0 at odd k
    y, a = oracle.linear(x, pack(cu), s)
    assert (y == 0).all() and (a == k).all()


def test_integer_valued_case_is_an_integer_matvec():
    rng = np.random.default_rng(10)
    m, n, k = 4, 37, 320
    cu = rng.integers(0, 16, (n, k), dtype=np.uint8)
    s = np.full((n, k // 32), 127, np.uint8)
    xi = rng.integers(-8, 9, (m, k))
    two_w = np.array([0, 1, 2, 3, 4, 6, 8, 12, 0, -1, -2, -3, -4, -6, -8, -12], np.int64)[cu]  # 2 * value
    want2 = xi.astype(np.int64) @ two_w.T
    wantabs2 = np.abs(xi).astype(np.int64) @ np.abs(two_w).T
    y, a = oracle.linear(f32_to_bf16_bits(xi.astype(np.float32)), pack(cu), s)
    assert np.array_equal(y * 2, want2.astype(np.float64))
    assert np.array_equal(a * 2, wantabs2.astype(np.float64))


def test_rational_arithmetic_small():
    rng = np.random.default_rng(11)
    m, n, k = 2, 3, 64
    cu = rng.integers(0, 16, (n, k), dtype=np.uint8)
    s = rng.integers(100, 140, (n, k // 32), dtype=np.uint8)
    xb = (rng.standard_normal((m, k)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    y, a = oracle.linear(xb, pack(cu), s)
    vals = e2m1_values()
    for mm in range(m):
        for nn in range(n):
            acc, accabs = Fraction(0), Fraction(0)
            for kk in range(k):
                w = Fraction(vals[int(cu[nn, kk])]) * Fraction(2) ** (int(s[nn, kk // 32]) - 127)
                p = bits_fraction(xb[mm, kk]) * w
                acc += p
                accabs += abs(p)
            assert abs(Fraction(y[mm, nn]) - acc) <= Fraction(1, 10 ** 13) * accabs
            assert abs(Fraction(a[mm, nn]) - accabs) <= Fraction(1, 10 ** 13) * accabs


def test_against_library_matmul_with_distinct_m_n_k():
    """M, N and K all different and X rows distinct, so a transposed operand or a swapped index fails."""
    rng = np.random.default_rng(12)
    m, n, k = 5, 129, 416
    wbits = ((rng.standard_normal((n, k)) * 0.02).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    codes, scales, _ = oracle.quantize(wbits)
    xb = (rng.standard_normal((m, k)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    y, a = oracle.linear(xb, codes, scales)
    wd = decode_with_fixture(codes, scales)
    x = bits_to_f64(xb)
    want = x @ wd.T
    wanta = np.abs(x) @ np.abs(wd).T
    assert y.shape == (m, n)
    assert np.all(np.abs(y - want) <= 1e-12 * wanta)
    assert np.all(np.abs(a - wanta) <= 1e-12 * wanta)
    # the dequantised matrix itself agrees with the independent decode
    assert np.array_equal(oracle.dequantize(codes, scales), wd)
    # and the quantised product is close to the unquantised one (direct cast keeps ~1 significant digit+)
    ref = x @ bits_to_f64(wbits).T
    assert np.abs(y - ref).mean() < 0.2 * np.abs(ref).mean() + 1e-3


def test_rows_subset_matches_full():
    rng = np.random.default_rng(13)
    m, n, k = 3, 40, 96
    codes = rng.integers(0, 256, (n, k // 2), dtype=np.uint8)
    scales = rng.integers(110, 130, (n, k // 32), dtype=np.uint8)
    xb = (rng.standard_normal((m, k)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    y, a = oracle.linear(xb, codes, scales)
    rows = np.array([39, 0, 7, 7, 21], np.int64)
    ys, as_ = oracle.linear(xb, codes, scales, rows=rows)
    assert np.array_equal(ys, y[:, rows]) and np.array_equal(as_, a[:, rows])


def test_nan_scale_poisons_only_its_row():
    codes = np.full((2, 32), 0x22, np.uint8)
    scales = np.full((2, 2), 127, np.uint8)
    scales[1, 1] = 0xFF
    x = f32_to_bf16_bits(np.ones((1, 64), np.float32))
    y, _ = oracle.linear(x, codes, scales)
    assert y[0, 0] == 64 and np.isnan(y[0, 1])


def test_smallest_and_largest_scales():
    codes = np.zeros((2, 16), np.uint8)
    codes[0, 0] = 0x01  # +0.5 at k=0
    codes[1, 0] = 0x07  # +6 at k=0
    scales = np.array([[0], [252]], np.uint8)
    x = f32_to_bf16_bits(np.ones((1, 32), np.float32))
    y, _ = oracle.linear(x, codes, scales)
    assert Fraction(y[0, 0]) == Fraction(1, 2) * Fraction(2) ** -127
    assert Fraction(y[0, 1]) == 6 * Fraction(2) ** 125
