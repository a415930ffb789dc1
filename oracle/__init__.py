"""ctypes/numpy front end of the CPU oracle (``mxq_oracle.c``).

TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.  Only ``tests/``, the smoke
check and the benchmark's ``cpu_baseline`` / ``--impl reference`` legs may
import this package.  It imports nothing from the CUDA package and the CUDA
package imports nothing from here.

All tensors cross this boundary as numpy arrays: BF16 data as ``uint16`` bit
patterns, codes and scales as ``uint8``, results as ``float64`` / ``int32``.
The arithmetic is all in the C file; this module only compiles it on first
use, marshals arguments and allocates outputs (exceptions, written with numpy here: ``linear_bf16``, the unquantised
comparison layer, is the textbook matrix product; ``silu``, ``linear_residual`` and ``linear_swiglu`` apply an
elementwise formula to the outputs of ``linear``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mxq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over independent rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-O2", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, vp = ctypes.c_int64, ctypes.c_void_p
            lib.oq_quantize.restype = i64
            lib.oq_quantize.argtypes = [vp, i64, i64, vp, vp]
            lib.oq_dequantize.restype = None
            lib.oq_dequantize.argtypes = [vp, vp, i64, i64, vp]
            lib.oq_linear.restype = None
            lib.oq_linear.argtypes = [vp, i64, vp, vp, i64, i64, vp, vp]
            lib.oq_linear_rows.restype = None
            lib.oq_linear_rows.argtypes = [vp, i64, vp, vp, i64, i64, vp, i64, vp, vp]
            lib.oq_argmax.restype = None
            lib.oq_argmax.argtypes = [vp, ctypes.c_int, i64, i64, vp]
            lib.oq_greedy_accept_tokens.restype = None
            lib.oq_greedy_accept_tokens.argtypes = [vp, vp, i64, i64, i64, vp, vp]
            lib.oq_greedy_accept.restype = None
            lib.oq_greedy_accept.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, vp, vp, vp]
            lib.oq_threads.restype = ctypes.c_int
            lib.oq_set_threads.argtypes = [ctypes.c_int]
            _lib = lib
    return _lib


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _c(a, dtype):
    a = np.ascontiguousarray(a)
    if a.dtype != dtype:
        raise TypeError("expected %s, got %s" % (dtype, a.dtype))
    return a


def threads() -> int:
    return int(_load().oq_threads())


def set_threads(n: int) -> None:
    _load().oq_set_threads(int(n))


def quantize(w_bits: np.ndarray):
    """BF16 bits [N,K] -> (codes u8 [N,K/2], scales u8 [N,K/32], nonfinite blocks)."""
    w = _c(w_bits, np.uint16)
    n, k = w.shape
    if k % 32:
        raise ValueError("K must be a multiple of 32")
    codes = np.empty((n, k // 2), np.uint8)
    scales = np.empty((n, k // 32), np.uint8)
    bad = _load().oq_quantize(_p(w), n, k, _p(codes), _p(scales))
    return codes, scales, int(bad)


def dequantize(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """(codes, scales) -> float64 [N,K], each entry the exact represented value."""
    c = _c(codes, np.uint8)
    s = _c(scales, np.uint8)
    n, k = c.shape[0], c.shape[1] * 2
    assert s.shape == (n, k // 32)
    out = np.empty((n, k), np.float64)
    _load().oq_dequantize(_p(c), _p(s), n, k, _p(out))
    return out


def linear(x_bits: np.ndarray, codes: np.ndarray, scales: np.ndarray, rows=None):
    """y64[M,N] = X . dequant(W)^T and A[M,N] = sum_k |x w^|, float64.

    ``rows``: optional int64 list of output rows; then the results are [M,len(rows)].
    """
    x = _c(x_bits, np.uint16)
    c = _c(codes, np.uint8)
    s = _c(scales, np.uint8)
    m, k = x.shape
    n = c.shape[0]
    assert c.shape == (n, k // 2) and s.shape == (n, k // 32)
    if rows is None:
        y = np.empty((m, n), np.float64)
        a = np.empty((m, n), np.float64)
        _load().oq_linear(_p(x), m, _p(c), _p(s), n, k, _p(y), _p(a))
    else:
        r = np.ascontiguousarray(rows, dtype=np.int64)
        assert r.ndim == 1 and (r >= 0).all() and (r < n).all()
        y = np.empty((m, r.size), np.float64)
        a = np.empty((m, r.size), np.float64)
        _load().oq_linear_rows(_p(x), m, _p(c), _p(s), n, k, _p(r), r.size, _p(y), _p(a))
    return y, a


def linear_bf16(x_bits: np.ndarray, w_bits: np.ndarray, rows=None):
    """The layer with unquantised BF16 weights (the comparison point of Sec. III-D-3 / IV-D): the plain definition
    y[m, n] = sum_k x[m, k] * w[n, k] in FP64 (numpy's matmul is the one library step), and a[m, n] = sum_k |x w|.
    BF16 bit patterns in, every product exact in FP64.  ``rows``: compute only these output columns n."""
    x = (_c(x_bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    wb = _c(w_bits, np.uint16)
    if rows is not None:
        wb = wb[np.asarray(rows, dtype=np.int64)]
    w = (wb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return x @ w.T, np.abs(x) @ np.abs(w).T


def silu(g: np.ndarray) -> np.ndarray:
    """silu(g) = g * sigmoid(g) = g / (1 + e^-g), float64: the activation of the gated feed-forward block of the
    Llama-family models the paper evaluates (Sec. IV-A).  Written in the form that cannot overflow: for g < 0 the
    quotient is taken as g e^g / (1 + e^g)."""
    g = np.asarray(g, np.float64)
    e = np.exp(-np.abs(g))                       # in (0, 1]
    return np.where(g >= 0, g / (1.0 + e), g * e / (1.0 + e))


def linear_residual(x_bits: np.ndarray, codes: np.ndarray, scales: np.ndarray, residual: np.ndarray, rows=None):
    """The layer with the residual add fused into its output (Sec. III-D-2 lists the residual add among the operators
    fused into the linear layers): out[m, n] = residual[m, n] + sum_k x[m, k] w^[n, k], float64, and A as ``linear``.
    ``residual`` is [M, N] (or [M, len(rows)] with ``rows``) as float64 values."""
    y, a = linear(x_bits, codes, scales, rows)
    r = np.asarray(residual, np.float64)
    assert r.shape == y.shape
    return y + r, a


def linear_swiglu(x_bits: np.ndarray, codes: np.ndarray, scales: np.ndarray, rows=None):
    """Gate and up projections of the gated feed-forward block as ONE matrix of 2F rows, row 2i = gate row i and row
    2i + 1 = up row i: out[m, i] = silu(g[m, i]) * u[m, i] with g, u the two plain layer outputs.  Returns
    (out, g, u, a_g, a_u), all [M, F] float64 (a_* = sum_k |x w^| of the two rows, for error bounds).
    ``rows``: optional list of output columns i."""
    n = np.asarray(codes).shape[0]
    assert n % 2 == 0
    idx = np.arange(n // 2, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    g, ag = linear(x_bits, codes, scales, 2 * idx)
    u, au = linear(x_bits, codes, scales, 2 * idx + 1)
    return silu(g) * u, g, u, ag, au


def _logits_arg(logits: np.ndarray):
    lg = np.ascontiguousarray(logits)
    if lg.dtype == np.float32:
        return lg, 0
    if lg.dtype == np.uint16:
        return lg, 1
    raise TypeError("logits must be float32 or uint16 (BF16 bits)")


def argmax(logits: np.ndarray) -> np.ndarray:
    """[..., V] float32 or BF16 bits -> int32 [...]; lowest index on ties, NaN never wins."""
    lg, is_bf16 = _logits_arg(logits)
    v = lg.shape[-1]
    rows = lg.size // v if v else 0
    out = np.empty(lg.shape[:-1], np.int32)
    _load().oq_argmax(_p(lg), is_bf16, rows, v, _p(out))
    return out


def greedy_accept_tokens(draft: np.ndarray, verifier: np.ndarray):
    """draft [B,T], verifier [B,R] int32 -> (accept_len [B], next_token [B])."""
    d = _c(draft, np.int32)
    t = _c(verifier, np.int32)
    b, tt = d.shape
    r = t.shape[1]
    assert t.shape[0] == b and r in (tt, tt + 1)
    g = np.empty(b, np.int32)
    nxt = np.empty(b, np.int32)
    _load().oq_greedy_accept_tokens(_p(d), _p(t), b, tt, r, _p(g), _p(nxt))
    return g, nxt


def greedy_accept(logits: np.ndarray, draft: np.ndarray):
    """logits [B,R,V], draft [B,T] -> (accept_len [B], next_token [B])."""
    lg, is_bf16 = _logits_arg(logits)
    d = _c(draft, np.int32)
    b, r, v = lg.shape
    tt = d.shape[1]
    assert d.shape[0] == b and r in (tt, tt + 1)
    ver = np.empty((b, r), np.int32)
    g = np.empty(b, np.int32)
    nxt = np.empty(b, np.int32)
    _load().oq_greedy_accept(_p(lg), is_bf16, b, r, v, _p(d), tt, _p(ver), _p(g), _p(nxt))
    return g, nxt
