"""Pins for the oracle of the unquantised comparison layer (oracle.linear_bf16): special cases with closed forms and a
brute-force loop, so that a transposed operand, a wrong decode of the BF16 bits or a dropped |.| fails."""
import numpy as np

import oracle


def bf16_bits(a):
    a = np.asarray(a, np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)   # exact for values that are BF16 numbers


def test_one_hot_weights_pick_elements_of_x():
    k, n = 64, 5
    x = np.arange(1, k + 1, dtype=np.float32).reshape(1, k)          # integers up to 64 are BF16 numbers
    w = np.zeros((n, k), np.float32)
    for r in range(n):
        w[r, 7 * r + 3] = -2.0
    y, a = oracle.linear_bf16(bf16_bits(x), bf16_bits(w))
    assert y.shape == (1, n) and a.shape == (1, n)
    assert y[0].tolist() == [-2.0 * (7 * r + 4) for r in range(n)]
    assert a[0].tolist() == [2.0 * (7 * r + 4) for r in range(n)]


def test_rectangular_shapes_are_not_transposed_and_rows_select_outputs():
    m, n, k = 3, 4, 2
    x = np.array([[1, 2], [3, 4], [5, 6]], np.float32)
    w = np.array([[1, 0], [0, 1], [1, 1], [-1, 0.5]], np.float32)
    y, a = oracle.linear_bf16(bf16_bits(x), bf16_bits(w))
    assert y.tolist() == [[1, 2, 3, 0], [3, 4, 7, -1], [5, 6, 11, -2]]
    assert a.tolist() == [[1, 2, 3, 2], [3, 4, 7, 5], [5, 6, 11, 8]]
    y2, a2 = oracle.linear_bf16(bf16_bits(x), bf16_bits(w), rows=[3, 0])
    assert y2.tolist() == [[0, 1], [-1, 3], [-2, 5]] and a2.shape == (m, 2)


def test_against_a_python_loop_on_random_bf16_bits():
    rng = np.random.default_rng(5)
    m, n, k = 2, 6, 40
    xb = rng.integers(0x3C00, 0x4100, (m, k)).astype(np.uint16) | (rng.integers(0, 2, (m, k)) << 15).astype(np.uint16)
    wb = rng.integers(0x3A00, 0x3F80, (n, k)).astype(np.uint16) | (rng.integers(0, 2, (n, k)) << 15).astype(np.uint16)
    def val(b):   # BF16 decode written out: sign, 8-bit exponent, 7-bit fraction (normal numbers only here)
        s, e, f = b >> 15, (b >> 7) & 0xFF, b & 0x7F
        return (-1.0) ** s * 2.0 ** (e - 127) * (1 + f / 128.0)
    y, a = oracle.linear_bf16(xb, wb)
    for i in range(m):
        for j in range(n):
            acc = sum(val(int(xb[i, t])) * val(int(wb[j, t])) for t in range(k))
            assert abs(y[i, j] - acc) <= 1e-12 * a[i, j]
            assert abs(a[i, j] - sum(abs(val(int(xb[i, t])) * val(int(wb[j, t]))) for t in range(k))) <= 1e-12 * a[i, j]
