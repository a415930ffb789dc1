"""Pins for the oracle of the fused layer epilogues (oracle.silu, oracle.linear_residual, oracle.linear_swiglu):
closed forms and identities of the activation, and layers whose outputs are known by construction, so that a swapped
gate / up row, a missing activation, a wrong sign in the exponent or a dropped residual fails."""
import math

import numpy as np

import oracle


def bf16_bits(a):
    a = np.asarray(a, np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)   # exact for values that are BF16 numbers


def test_silu_closed_forms_and_identities():
    assert oracle.silu(np.array([0.0]))[0] == 0.0
    # silu(1) = 1 / (1 + 1/e), silu(-1) = -1 / (1 + e), silu(ln 3) = ln 3 * 3/4
    assert abs(oracle.silu(np.array([1.0]))[0] - 1.0 / (1.0 + 1.0 / math.e)) < 1e-15
    assert abs(oracle.silu(np.array([-1.0]))[0] + 1.0 / (1.0 + math.e)) < 1e-15
    assert abs(oracle.silu(np.array([math.log(3.0)]))[0] - 0.75 * math.log(3.0)) < 1e-15
    g = np.linspace(-30, 30, 2001)
    s = oracle.silu(g)
    assert np.allclose(s - oracle.silu(-g), g, rtol=0, atol=1e-13)      # x sigma(x) + x sigma(-x) = x
    assert (s >= -0.2785).all() and s.min() < -0.2784                    # the global minimum, -0.27846...
    assert abs(g[np.argmin(s)] + 1.2785) < 0.03                          # ... at x = -1.2785
    assert np.allclose(s[g > 25], g[g > 25], rtol=1e-10)                 # -> x
    assert (np.abs(s[g < -25]) < 1e-9).all()                             # -> 0 from below
    big = oracle.silu(np.array([-800.0, 800.0]))
    assert big[0] == 0.0 and big[1] == 800.0 and np.isfinite(big).all()  # no overflow on either side


def one_hot_layer(n, k, picks, values):
    """W[n, k] with W[r, picks[r]] = values[r] (values representable in E2M1 at scale 1), zero elsewhere."""
    w = np.zeros((n, k), np.float32)
    for r in range(n):
        w[r, picks[r]] = values[r]
    return oracle.quantize(bf16_bits(w))[:2]


def test_swiglu_pairs_rows_as_gate_then_up():
    k, f = 64, 4
    x = np.zeros((1, k), np.float32)
    x[0, :8] = [1.0, -2.0, 0.5, 3.0, 4.0, -1.0, 2.0, 0.25]
    # gate row i picks x[i], up row i picks x[4 + i] with weight 2
    picks = [0, 4, 1, 5, 2, 6, 3, 7]
    values = [1.0, 2.0] * f
    codes, scales = one_hot_layer(2 * f, k, picks, values)
    out, g, u, ag, au = oracle.linear_swiglu(bf16_bits(x), codes, scales)
    assert g[0].tolist() == [1.0, -2.0, 0.5, 3.0] and u[0].tolist() == [8.0, -2.0, 4.0, 0.5]
    assert ag[0].tolist() == [1.0, 2.0, 0.5, 3.0] and au[0].tolist() == [8.0, 2.0, 4.0, 0.5]
    want = [gi / (1.0 + math.exp(-gi)) * ui for gi, ui in zip([1.0, -2.0, 0.5, 3.0], [8.0, -2.0, 4.0, 0.5])]
    assert np.allclose(out[0], want, rtol=1e-15, atol=0)
    assert abs(out[0, 0] - 5.8484686) < 1e-6  # silu(1) * 8; with gate and up swapped it would be silu(8) * 1 = 7.9973
    sub = oracle.linear_swiglu(bf16_bits(x), codes, scales, rows=[3, 0])
    assert np.array_equal(sub[0], out[:, [3, 0]]) and np.array_equal(sub[1], g[:, [3, 0]])


def test_swiglu_is_the_composition_of_two_plain_layers():
    rng = np.random.default_rng(11)
    m, f, k = 3, 6, 96
    w = rng.standard_normal((2 * f, k)).astype(np.float32) * 0.02
    x = rng.standard_normal((m, k)).astype(np.float32)
    codes, scales = oracle.quantize(bf16_bits(w))[:2]
    out, g, u, ag, au = oracle.linear_swiglu(bf16_bits(x), codes, scales)
    y, a = oracle.linear(bf16_bits(x), codes, scales)
    assert np.array_equal(g, y[:, 0::2]) and np.array_equal(u, y[:, 1::2])
    assert np.array_equal(ag, a[:, 0::2]) and np.array_equal(au, a[:, 1::2])
    for i in range(m):
        for j in range(f):
            assert abs(out[i, j] - y[i, 2 * j] / (1.0 + math.exp(-y[i, 2 * j])) * y[i, 2 * j + 1]) <= 1e-15 * abs(out[i, j]) + 1e-300


def test_residual_is_added_once_with_its_sign():
    k, n = 32, 3
    x = np.zeros((2, k), np.float32)
    x[0, 0], x[1, 0] = 3.0, -1.0
    codes, scales = one_hot_layer(n, k, [0, 0, 0], [1.0, -2.0, 0.5])
    res = np.array([[10.0, 20.0, -30.0], [0.5, 0.0, 1.0]])
    out, a = oracle.linear_residual(bf16_bits(x), codes, scales, res)
    assert out.tolist() == [[13.0, 14.0, -28.5], [-0.5, 2.0, 0.5]]
    assert a.tolist() == [[3.0, 6.0, 1.5], [1.0, 2.0, 0.5]]
    zero, _ = oracle.linear_residual(bf16_bits(x), codes, scales, np.zeros((2, n)))
    assert np.array_equal(zero, oracle.linear(bf16_bits(x), codes, scales)[0])
    sub, _ = oracle.linear_residual(bf16_bits(x), codes, scales, res[:, [2, 1]], rows=[2, 1])
    assert sub.tolist() == [[-28.5, 14.0], [0.5, 2.0]]
