"""Thin ctypes binding of ``libmxq.so`` -- argument marshalling only.

Function names and argument order follow ``include/mxq.h``.  Tensors are torch CUDA
tensors (torch supplies device memory and streams, nothing else); every step of the
computation runs in the library's own kernels.  There is no fallback: if the shared
library is missing, or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
import threading

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MXQ_LIBRARY=checked in the environment loads the bounds-checked build instead (see mxq_debug_bounds_report in mxq.h)
LIB_PATH = os.path.join(_HERE, "libmxq_checked.so" if os.environ.get("MXQ_LIBRARY") == "checked" else "libmxq.so")

MXQ_OK = 0
MXQ_F32, MXQ_BF16 = 0, 1
MAX_M, MAX_T = 16, 64

_lib = None
_lock = threading.Lock()


class MxqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


def lib() -> ctypes.CDLL:
    """Load ``libmxq.so`` (built by ``python -m paper_2503_13565_b200.build``)."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                raise ImportError("the mxq library is not built (%s missing): run python -m paper_2503_13565_b200.build [--checked]; "
                                  "there is no CPU fallback" % LIB_PATH)
            L = ctypes.CDLL(LIB_PATH)
            vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
            L.mxq_version.restype = i32
            L.mxq_status_string.restype = ctypes.c_char_p
            L.mxq_status_string.argtypes = [i32]
            L.mxq_set_pdl.restype = i32
            L.mxq_set_pdl.argtypes = [i32]
            for f in (L.mxq_codes_bytes, L.mxq_scales_bytes):
                f.restype = sz
                f.argtypes = [i64, i64]
            L.mxq_linear_workspace_bytes.restype = sz
            L.mxq_linear_workspace_bytes.argtypes = [i32, i64, i64]
            L.mxq_accept_workspace_bytes.restype = sz
            L.mxq_accept_workspace_bytes.argtypes = [i64, i32, i64]
            L.mxq_quantize.restype = i32
            L.mxq_quantize.argtypes = [vp, i64, i64, vp, vp, vp, vp]
            L.mxq_dequantize.restype = i32
            L.mxq_dequantize.argtypes = [vp, vp, i64, i64, vp, vp]
            L.mxq_linear.restype = i32
            L.mxq_linear.argtypes = [vp, i32, vp, vp, i64, i64, vp, i32, vp, sz, vp]
            L.mxq_linear_plan_info.restype = i32
            L.mxq_linear_plan_info.argtypes = [i32, i32, i64, i64, vp]
            L.mxq_set_linear_kernel.restype = i32
            L.mxq_set_linear_kernel.argtypes = [i32]
            L.mxq_linear_device_status.restype = i32
            L.mxq_linear_device_status.argtypes = [vp]
            L.mxq_linear_host.restype = i32
            L.mxq_linear_host.argtypes = [vp, i32, vp, vp, i64, i64, vp, i32, vp, vp, vp, sz, vp]
            L.mxq_greedy_accept.restype = i32
            L.mxq_greedy_accept.argtypes = [vp, i32, i64, i32, i64, vp, i32, vp, vp, vp, sz, vp]
            L.mxq_greedy_accept_static.restype = i32
            L.mxq_greedy_accept_static.argtypes = [vp, i32, i64, i32, i64, vp, i32, vp, vp, vp]
            L.mxq_greedy_accept_static_max_bytes.restype = sz
            L.mxq_greedy_accept_static_max_bytes.argtypes = []
            L.mxq_greedy_accept_tokens.restype = i32
            L.mxq_greedy_accept_tokens.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp]
            L.mxq_linear_bf16.restype = i32
            L.mxq_linear_bf16.argtypes = [vp, i32, vp, i64, i64, vp, i32, vp]
            L.mxq_linear_fused_workspace_bytes.restype = sz
            L.mxq_linear_fused_workspace_bytes.argtypes = [i32, i64, i64]
            L.mxq_linear_residual.restype = i32
            L.mxq_linear_residual.argtypes = [vp, i32, vp, vp, i64, i64, vp, vp, i32, vp, sz, vp]
            L.mxq_linear_swiglu.restype = i32
            L.mxq_linear_swiglu.argtypes = [vp, i32, vp, vp, i64, i64, vp, i32, vp, sz, vp]
            L.mxq_lm_head_accept_workspace_bytes.restype = sz
            L.mxq_lm_head_accept_workspace_bytes.argtypes = [i32, i64, i64]
            L.mxq_lm_head_accept.restype = i32
            L.mxq_lm_head_accept.argtypes = [vp, i32, vp, vp, i64, i64, vp, i32, vp, vp, vp, vp, sz, vp]
            L.mxq_set_linear_layout.restype = i32
            L.mxq_set_linear_layout.argtypes = [i32, i32]
            L.mxq_linear_batch_workspace_bytes.restype = sz
            L.mxq_linear_batch_workspace_bytes.argtypes = [vp, i32, i32]
            L.mxq_linear_batch.restype = i32
            L.mxq_linear_batch.argtypes = [vp, i32, i32, vp, sz, vp]
            L.mxq_linear_batch_info.restype = i32
            L.mxq_linear_batch_info.argtypes = [vp, i32, i32, vp]
            L.mxq_debug_bounds_report.restype = i32
            L.mxq_debug_bounds_report.argtypes = [vp]
            L.mxq_debug_bounds_selftest.restype = i32
            L.mxq_debug_bounds_selftest.argtypes = [vp]
            L.mxq_debug_batch_fault.restype = i32
            L.mxq_debug_batch_fault.argtypes = [i32, ctypes.c_uint]
            _lib = L
    return _lib


def _check(status: int, where: str) -> None:
    if status != MXQ_OK:
        raise MxqError(status, where)


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dev(t: torch.Tensor, dtype, what: str) -> int:
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return t.data_ptr()


def _dt(dtype) -> int:
    if dtype == torch.float32:
        return MXQ_F32
    if dtype == torch.bfloat16:
        return MXQ_BF16
    raise TypeError("dtype must be torch.float32 or torch.bfloat16")


# ---- the calls of include/mxq.h ---------------------------------------------------------


def mxq_version() -> int:
    return int(lib().mxq_version())


def status_string(status: int) -> str:
    return lib().mxq_status_string(int(status)).decode()


def mxq_set_pdl(enabled: bool) -> bool:
    return bool(lib().mxq_set_pdl(1 if enabled else 0))


def mxq_codes_bytes(n: int, k: int) -> int:
    return int(lib().mxq_codes_bytes(n, k))


def mxq_scales_bytes(n: int, k: int) -> int:
    return int(lib().mxq_scales_bytes(n, k))


def mxq_linear_workspace_bytes(m: int, n: int, k: int) -> int:
    return int(lib().mxq_linear_workspace_bytes(m, n, k))


KERNELS = {"auto": -1, "generic": 0, "mma": 1, "umma": 2, "fp4": 3}
_KERNEL_NAMES = {v: k for k, v in KERNELS.items()}
_PLAN_KEYS = {
    3: ("kernel", "grid", "ring", "split", "chunk_max", "tiles", "tmem_cols", "smem_bytes", "nb", "kb", "groups", "tiles_max"),
    2: ("kernel", "grid", "ring", "split", "chunk_max", "tiles", "tmem_cols", "smem_bytes", "nb", "kb", "groups", "tiles_max"),
    1: ("kernel", "grid", "stages", "windows", "bw", "bw_last", "max_tiles", "smem_bytes", "nt8", "kb"),
    0: ("kernel", "grid"),
}


def mxq_set_linear_kernel(kernel) -> str:
    """Override mxq_linear's choice of kernel: "auto" (default: by measured speed), or "fp4" / "umma" / "mma" /
    "generic" = the first kernel not above that one that covers the call.  Returns the previous setting."""
    code = KERNELS[kernel] if isinstance(kernel, str) else int(kernel)
    return _KERNEL_NAMES[int(lib().mxq_set_linear_kernel(code))]


def mxq_linear_plan_info(m: int, n: int, k: int, kernel="auto") -> dict:
    """How a kernel would run this shape (diagnostics).  ``kernel`` is a name of KERNELS; the result's
    "kernel" is the name of the kernel described, or None if the requested one does not cover the shape."""
    info = (ctypes.c_int32 * 12)()
    code = KERNELS[kernel] if isinstance(kernel, str) else int(kernel)
    _check(lib().mxq_linear_plan_info(code, m, n, k, ctypes.cast(info, ctypes.c_void_p)), "mxq_linear_plan_info")
    vals = [int(v) for v in info]
    if vals[0] < 0:
        return {"kernel": None}
    out = dict(zip(_PLAN_KEYS[vals[0]], vals))
    out["kernel"] = _KERNEL_NAMES[vals[0]]
    return out


def mxq_linear_device_status() -> int:
    """The sticky word in which the tcgen05 kernel records a bounded wait that gave up (0 = never); cleared by the call."""
    word = ctypes.c_uint32(0)
    _check(lib().mxq_linear_device_status(ctypes.cast(ctypes.byref(word), ctypes.c_void_p)), "mxq_linear_device_status")
    return int(word.value)


def mxq_accept_workspace_bytes(b: int, r: int, v: int) -> int:
    return int(lib().mxq_accept_workspace_bytes(b, r, v))


_default_ws = {}


def _default_workspace(nbytes: int, device) -> torch.Tensor:
    """A cached, zero-initialised workspace per device for callers that pass none."""
    key = (torch.device(device).type, torch.device(device).index if torch.device(device).index is not None
           else torch.cuda.current_device())
    ws = _default_ws.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = new_workspace(nbytes, device)
        _default_ws[key] = ws
    return ws


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Zero-filled workspace of at least ``nbytes`` (the zero fill is the one-time initialisation)."""
    return torch.zeros(max(16, (int(nbytes) + 15) // 16 * 16), dtype=torch.uint8, device=device)


def mxq_quantize(w: torch.Tensor, codes: torch.Tensor = None, scales: torch.Tensor = None,
                 nonfinite_blocks: torch.Tensor = None, stream=None):
    """BF16 W[N,K] -> (codes u8 [N,K/2], scales u8 [N,K/32])."""
    n, k = w.shape
    if codes is None:
        codes = torch.empty((n, k // 2), dtype=torch.uint8, device=w.device)
    if scales is None:
        scales = torch.empty((n, k // 32), dtype=torch.uint8, device=w.device)
    cnt = 0 if nonfinite_blocks is None else _dev(nonfinite_blocks, torch.int32, "nonfinite_blocks")
    _check(lib().mxq_quantize(_dev(w, torch.bfloat16, "W"), n, k, _dev(codes, torch.uint8, "codes"),
                              _dev(scales, torch.uint8, "scales"), cnt, _stream(stream)), "mxq_quantize")
    return codes, scales


def mxq_dequantize(codes: torch.Tensor, scales: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
    n, k = codes.shape[0], codes.shape[1] * 2
    if out is None:
        out = torch.empty((n, k), dtype=torch.bfloat16, device=codes.device)
    _check(lib().mxq_dequantize(_dev(codes, torch.uint8, "codes"), _dev(scales, torch.uint8, "scales"), n, k,
                                _dev(out, torch.bfloat16, "out"), _stream(stream)), "mxq_dequantize")
    return out


def mxq_linear(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, out: torch.Tensor = None,
               out_dtype=torch.float32, workspace: torch.Tensor = None, stream=None) -> torch.Tensor:
    """Y[M,N] = X[M,K] . dequant(codes, scales)^T."""
    m, k = x.shape
    n = codes.shape[0]
    if codes.shape[1] * 2 != k or tuple(scales.shape) != (n, k // 32):
        raise ValueError("shape mismatch between X, codes and scales")
    if out is None:
        out = torch.empty((m, n), dtype=out_dtype, device=x.device)
    if workspace is None:
        need = mxq_linear_workspace_bytes(m, n, k)
        workspace = _default_workspace(need, x.device) if need else None
    ws_ptr, ws_bytes = (0, 0) if workspace is None else (_dev(workspace, torch.uint8, "workspace"), workspace.numel())
    _check(lib().mxq_linear(_dev(x, torch.bfloat16, "X"), m, _dev(codes, torch.uint8, "codes"),
                            _dev(scales, torch.uint8, "scales"), n, k, _dev(out, out.dtype, "Y"), _dt(out.dtype),
                            ws_ptr, ws_bytes, _stream(stream)), "mxq_linear")
    return out


def mxq_linear_host(x_host: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, y_host: torch.Tensor,
                    x_stage: torch.Tensor, y_stage: torch.Tensor, workspace: torch.Tensor = None, stream=None) -> None:
    """Same layer with X and Y in (pinned) host memory; staging buffers live on the device."""
    m, k = x_host.shape
    n = codes.shape[0]
    if x_host.is_cuda or y_host.is_cuda or x_host.dtype != torch.bfloat16 or not x_host.is_contiguous() \
            or not y_host.is_contiguous() or tuple(y_host.shape) != (m, n):
        raise TypeError("x_host / y_host must be contiguous host tensors (BF16 X[M,K], Y[M,N])")
    if x_stage.numel() * x_stage.element_size() < m * k * 2 or \
            y_stage.numel() * y_stage.element_size() < m * n * y_host.element_size():
        raise ValueError("staging buffers too small")
    if workspace is None:
        need = mxq_linear_workspace_bytes(m, n, k)
        workspace = _default_workspace(need, codes.device) if need else None
    ws_ptr, ws_bytes = (0, 0) if workspace is None else (_dev(workspace, torch.uint8, "workspace"), workspace.numel())
    _check(lib().mxq_linear_host(x_host.data_ptr(), m, _dev(codes, torch.uint8, "codes"),
                                 _dev(scales, torch.uint8, "scales"), n, k, y_host.data_ptr(), _dt(y_host.dtype),
                                 x_stage.data_ptr(), y_stage.data_ptr(), ws_ptr, ws_bytes, _stream(stream)),
           "mxq_linear_host")


def mxq_greedy_accept(logits: torch.Tensor, draft: torch.Tensor, workspace: torch.Tensor = None, stream=None, out=None):
    """logits [B,R,V] (fp32 or bf16), draft [B,T] int32 -> (accept_len [B], next_token [B]) int32.  ``out``: optional
    pair of int32 [B] tensors to write into (pass them when the call runs on another stream than the current one)."""
    b, r, v = logits.shape
    t = draft.shape[1]
    if workspace is None:
        workspace = new_workspace(mxq_accept_workspace_bytes(b, r, v), logits.device)
    if out is None:
        g = torch.empty(b, dtype=torch.int32, device=logits.device)
        nxt = torch.empty(b, dtype=torch.int32, device=logits.device)
    else:
        g, nxt = out
        if tuple(g.shape) != (b,) or tuple(nxt.shape) != (b,):
            raise ValueError("out must be two int32 tensors of shape [B]")
    _check(lib().mxq_greedy_accept(_dev(logits, logits.dtype, "logits"), _dt(logits.dtype), b, r, v,
                                   _dev(draft, torch.int32, "draft"), t, _dev(g, torch.int32, "accept_len"), _dev(nxt, torch.int32, "next_token"),
                                   _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
           "mxq_greedy_accept")
    return g, nxt


def mxq_greedy_accept_static_max_bytes() -> int:
    return int(lib().mxq_greedy_accept_static_max_bytes())


def mxq_greedy_accept_static(logits: torch.Tensor, draft: torch.Tensor, accept_len: torch.Tensor,
                             next_token: torch.Tensor, stream=None) -> None:
    """mxq_greedy_accept without a workspace, for callers that cannot allocate one: the scratch is an array
    built into the library (1 MiB per GPU).  The caller passes the outputs too (int32 [B] each); nothing is
    allocated on the way.  Calls on one device share that array, so calls that may overlap on the GPU race."""
    b, r, v = logits.shape
    t = draft.shape[1]
    if tuple(accept_len.shape) != (b,) or tuple(next_token.shape) != (b,):
        raise ValueError("accept_len and next_token must be int32 tensors of shape [B]")
    _check(lib().mxq_greedy_accept_static(_dev(logits, logits.dtype, "logits"), _dt(logits.dtype), b, r, v,
                                          _dev(draft, torch.int32, "draft"), t,
                                          _dev(accept_len, torch.int32, "accept_len"),
                                          _dev(next_token, torch.int32, "next_token"), _stream(stream)),
           "mxq_greedy_accept_static")


def mxq_greedy_accept_tokens(draft: torch.Tensor, verifier: torch.Tensor, stream=None):
    b, t = draft.shape
    r = verifier.shape[1]
    g = torch.empty(b, dtype=torch.int32, device=draft.device)
    nxt = torch.empty(b, dtype=torch.int32, device=draft.device)
    _check(lib().mxq_greedy_accept_tokens(_dev(draft, torch.int32, "draft"), _dev(verifier, torch.int32, "verifier"),
                                          b, t, r, g.data_ptr(), nxt.data_ptr(), _stream(stream)),
           "mxq_greedy_accept_tokens")
    return g, nxt


def mxq_lm_head_accept_workspace_bytes(r: int, v: int, k: int) -> int:
    return int(lib().mxq_lm_head_accept_workspace_bytes(r, v, k))


def mxq_lm_head_accept(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, draft: torch.Tensor = None,
                       workspace: torch.Tensor = None, stream=None):
    """Vocabulary projection + argmax of every row + walk over the draft in one launch (the logits are never written).
    x [R,K] BF16, codes/scales the MXFP4 pair of the [V,K] projection, draft [T] int32 with R == T or T + 1 (None: T = 0).
    Returns (verifier [R] int32, accept_len [1] int32, next_token [1] int32).  ``workspace``: from ``new_workspace(
    mxq_lm_head_accept_workspace_bytes(R, V, K))`` (zero-filled once; reusable; one per stream)."""
    r, k = x.shape
    v = codes.shape[0]
    t = 0 if draft is None else int(draft.numel())
    if workspace is None:
        workspace = new_workspace(mxq_lm_head_accept_workspace_bytes(r, v, k), x.device)
    verifier = torch.empty(r, dtype=torch.int32, device=x.device)
    g = torch.empty(1, dtype=torch.int32, device=x.device)
    nxt = torch.empty(1, dtype=torch.int32, device=x.device)
    _check(lib().mxq_lm_head_accept(_dev(x, torch.bfloat16, "x"), r, _dev(codes, torch.uint8, "codes"),
                                    _dev(scales, torch.uint8, "scales"), v, k,
                                    0 if draft is None else _dev(draft, torch.int32, "draft"), t,
                                    verifier.data_ptr(), g.data_ptr(), nxt.data_ptr(),
                                    _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
           "mxq_lm_head_accept")
    return verifier, g, nxt


def mxq_linear_bf16(x: torch.Tensor, w: torch.Tensor, out: torch.Tensor = None, out_dtype=torch.float32, stream=None) -> torch.Tensor:
    """Y[M,N] = X[M,K] . W[N,K]^T with W in BF16 (not quantised): the comparison point for mxq_linear."""
    m, k = x.shape
    n = w.shape[0]
    if out is None:
        out = torch.empty((m, n), dtype=out_dtype, device=x.device)
    _check(lib().mxq_linear_bf16(_dev(x, torch.bfloat16, "x"), m, _dev(w, torch.bfloat16, "w"), n, k,
                                 _dev(out, out.dtype, "out"), _dt(out.dtype), _stream(stream)), "mxq_linear_bf16")
    return out


def mxq_linear_fused_workspace_bytes(m: int, n: int, k: int) -> int:
    return int(lib().mxq_linear_fused_workspace_bytes(m, n, k))


def mxq_linear_residual(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, residual: torch.Tensor,
                        out: torch.Tensor = None, workspace: torch.Tensor = None, stream=None) -> torch.Tensor:
    """Y[M,N] = residual[M,N] + X[M,K] . dequant(W)^T in one launch.  ``residual`` is FP32 or BF16 and fixes Y's type;
    ``out`` may be ``residual`` itself (in-place add).  ``workspace``: uint8, at least
    ``mxq_linear_fused_workspace_bytes(M, N, K)`` bytes (allocated here if None: pass one in a hot loop)."""
    m, k = x.shape
    n = codes.shape[0]
    if out is None:
        out = torch.empty((m, n), dtype=residual.dtype, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(16, mxq_linear_fused_workspace_bytes(m, n, k)), dtype=torch.uint8, device=x.device)
    _check(lib().mxq_linear_residual(_dev(x, torch.bfloat16, "x"), m, _dev(codes, torch.uint8, "codes"),
                                     _dev(scales, torch.uint8, "scales"), n, k, _dev(residual, out.dtype, "residual"),
                                     _dev(out, out.dtype, "out"), _dt(out.dtype),
                                     _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
           "mxq_linear_residual")
    return out


def mxq_linear_swiglu(x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, out: torch.Tensor = None,
                      out_dtype=torch.bfloat16, workspace: torch.Tensor = None, stream=None) -> torch.Tensor:
    """Y[M,F] = silu(X . gate^T) * (X . up^T) in one launch; ``codes`` / ``scales`` are the MXFP4 pair of the [2F,K]
    matrix whose row 2i is gate row i and row 2i+1 up row i (``interleave_gate_up``)."""
    m, k = x.shape
    n = codes.shape[0]
    if out is None:
        out = torch.empty((m, n // 2), dtype=out_dtype, device=x.device)
    if workspace is None:
        workspace = torch.empty(max(16, mxq_linear_fused_workspace_bytes(m, n, k)), dtype=torch.uint8, device=x.device)
    _check(lib().mxq_linear_swiglu(_dev(x, torch.bfloat16, "x"), m, _dev(codes, torch.uint8, "codes"),
                                   _dev(scales, torch.uint8, "scales"), n, k, _dev(out, out.dtype, "out"), _dt(out.dtype),
                                   _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
           "mxq_linear_swiglu")
    return out


def interleave_gate_up(gate: torch.Tensor, up: torch.Tensor) -> torch.Tensor:
    """[F,C] gate and up arrays (BF16 weights, or their codes or scales: the cast works row by row) -> the [2F,C] array
    mxq_linear_swiglu expects: row 2i = gate[i], row 2i+1 = up[i].  A copy, no arithmetic."""
    assert gate.shape == up.shape and gate.dtype == up.dtype
    return torch.stack((gate, up), dim=1).reshape(2 * gate.shape[0], gate.shape[1]).contiguous()


# ---- several layers in one launch -------------------------------------------------------------

LAYOUT_KNOBS = {"split": 0, "ring": 1, "tiles": 2, "operand_through_ring": 3, "presplit_min_m": 4, "batch_ring": 5,
                "batch_ctas_per_sm": 6}
EPILOGUES = {"none": 0, "residual": 1, "swiglu": 2}
MAX_BATCH = 64


def mxq_set_linear_layout(what, value: int) -> None:
    """Force one layout parameter of the tcgen05 kernels (tests, comparisons); see mxq_layout_knob in mxq.h."""
    code = LAYOUT_KNOBS[what] if isinstance(what, str) else int(what)
    _check(lib().mxq_set_linear_layout(code, int(value)), "mxq_set_linear_layout")


class _LinearDesc(ctypes.Structure):
    _fields_ = [("X_bf16", ctypes.c_void_p), ("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("Y", ctypes.c_void_p), ("residual", ctypes.c_void_p), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("y_dtype", ctypes.c_int32), ("epilogue", ctypes.c_int32), ("flags", ctypes.c_int32), ("reserved", ctypes.c_int32)]


def _any_mem(t: torch.Tensor, dtype, what: str) -> int:
    """Device tensor, or a page-locked host tensor the GPU can address."""
    if not ((t.is_cuda or t.is_pinned()) and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA (or pinned host) tensor of dtype %s" % (what, dtype))
    return t.data_ptr()


class LinearBatch:
    """The descriptor array of one mxq_linear_batch call, marshalled once and reusable (the call itself is then a
    single C call).  ``layers``: dicts with x [M,K] BF16, codes, scales, out [M,N] (or [M,N/2] for "swiglu"), and
    optionally epilogue ("none" | "residual" | "swiglu"), residual, and depends=True for a layer that (with the ones after
    it) reads what the layers before it write.  The tensors are kept alive by this object."""

    def __init__(self, layers):
        if not 1 <= len(layers) <= MAX_BATCH:
            raise ValueError("1..%d layers per call" % MAX_BATCH)
        self.m = int(layers[0]["x"].shape[0])
        self.count = len(layers)
        self.array = (_LinearDesc * self.count)()
        self.keep = []
        self.device = layers[0]["codes"].device
        self.groups = 0   # groups of layers that run one after the other (1: all layers independent)
        for i, (d, lay) in enumerate(zip(self.array, layers)):
            x, codes, scales, out = lay["x"], lay["codes"], lay["scales"], lay["out"]
            epi = EPILOGUES[lay.get("epilogue", "none")]
            res = lay.get("residual")
            m, k = x.shape
            n = codes.shape[0]
            if m != self.m or codes.shape[1] * 2 != k or tuple(scales.shape) != (n, k // 32):
                raise ValueError("shape mismatch between X, codes and scales")
            if tuple(out.shape) != (m, n // 2 if epi == 2 else n):
                raise ValueError("out has the wrong shape")
            d.X_bf16 = _any_mem(x, torch.bfloat16, "x")
            d.codes = _dev(codes, torch.uint8, "codes")
            d.scales = _dev(scales, torch.uint8, "scales")
            d.Y = _any_mem(out, out.dtype, "out")
            d.residual = _any_mem(res, out.dtype, "residual") if res is not None else None
            d.N, d.K = n, k
            d.y_dtype = _dt(out.dtype)
            d.epilogue = epi
            d.flags = 1 if lay.get("depends") else 0   # MXQ_BATCH_DEPENDS: a new group, after everything before it
            self.groups += 1 if (i == 0 or d.flags) else 0
            d.reserved = 0
            self.keep.append((x, codes, scales, out, res))
        self._ptr = ctypes.cast(self.array, ctypes.c_void_p)

    def workspace_bytes(self) -> int:
        return int(lib().mxq_linear_batch_workspace_bytes(self._ptr, self.count, self.m))

    def info(self) -> dict:
        info = (ctypes.c_int32 * 8)()
        _check(lib().mxq_linear_batch_info(self._ptr, self.count, self.m, ctypes.cast(info, ctypes.c_void_p)), "mxq_linear_batch_info")
        return dict(zip(("persistent", "grid", "ring", "smem_bytes", "nb", "units", "tmem_cols", "acc_slots"), [int(v) for v in info]))

    def run(self, workspace: torch.Tensor, stream=None) -> None:
        _check(lib().mxq_linear_batch(self._ptr, self.count, self.m, _dev(workspace, torch.uint8, "workspace"),
                                      workspace.numel(), _stream(stream)), "mxq_linear_batch")


def mxq_linear_batch(layers, workspace: torch.Tensor = None, stream=None) -> LinearBatch:
    """Several independent layers in one launch (see mxq_linear_batch in mxq.h).  Returns the marshalled batch, whose
    ``run(workspace)`` repeats the call without re-marshalling.  ``workspace``: from ``new_workspace(batch.workspace_bytes())``
    (zero-filled once; reusable by calls in one stream)."""
    batch = layers if isinstance(layers, LinearBatch) else LinearBatch(layers)
    if workspace is None:
        workspace = new_workspace(batch.workspace_bytes(), batch.device)
    batch.run(workspace, stream)
    return batch


class IndependentBatches:
    """Several mxq_linear_batch calls that do not read one another's outputs, issued round-robin on ``streams`` CUDA
    streams with a workspace each (calls that may run concurrently need one each, see mxq.h) between a fork and a join on
    the caller's stream.  In one stream a call cannot touch its inputs or the workspace before the call ahead of it has
    completed to its last CTA, and the memory system idles while its early CTAs wait; on two streams a call starts in the
    SM slots the other stream's call leaves.  Only stream plumbing: every call is the library's own."""

    def __init__(self, batches, streams: int = 2):
        self.batches = [b if isinstance(b, LinearBatch) else LinearBatch(b) for b in batches]
        if not self.batches:
            raise ValueError("no calls")
        self.device = self.batches[0].device
        n = max(1, min(int(streams), len(self.batches)))
        if n > 1 and any(b.groups > 1 for b in self.batches):
            # (the CTAs of a call of several groups wait for one another and need the whole grid resident: see mxq.h)
            raise ValueError("calls with dependent groups must not share the device with calls on other streams")
        self.workspaces = [new_workspace(max(b.workspace_bytes() for b in self.batches), self.device) for _ in range(n)]
        self.streams = [torch.cuda.Stream(device=self.device) for _ in range(n)] if n > 1 else []

    def run(self, stream=None) -> None:
        cur = torch.cuda.current_stream(self.device) if stream is None else stream
        if not self.streams:
            for b in self.batches:
                b.run(self.workspaces[0], cur)
            return
        fork = torch.cuda.Event()
        fork.record(cur)
        for s in self.streams:
            s.wait_event(fork)
        n = len(self.streams)
        for i, b in enumerate(self.batches):
            b.run(self.workspaces[i % n], self.streams[i % n])
        for s in self.streams:
            join = torch.cuda.Event()
            join.record(s)
            cur.wait_event(join)


def mxq_debug_bounds_report() -> dict:
    """What the bounds-checked build has refused since the last call (see mxq.h); ``checked`` is False for the ordinary build."""
    r = (ctypes.c_uint64 * 6)()
    _check(lib().mxq_debug_bounds_report(ctypes.cast(r, ctypes.c_void_p)), "mxq_debug_bounds_report")
    files = ("mxq_linear.cu", "mxq_linear_umma.cu", "mxq_linear_fp4.cu", "mxq_linear_mma.cu", "mxq_linear_batch.cu", "mxq_linear_bf16.cu")
    out = {"checked": bool(r[0]), "refused": int(r[1])}
    if r[1]:
        out.update(file=files[int(r[2])], line=int(r[3]), offset=int(r[4]), extent=int(r[5]))
    return out


def mxq_debug_bounds_selftest(stream=None) -> None:
    """Checked build only: one store outside a 64-byte buffer must be refused and redirected (see mxq.h)."""
    _check(lib().mxq_debug_bounds_selftest(_stream(stream)), "mxq_debug_bounds_selftest")


def mxq_debug_batch_fault(unit: int, wait_us: int) -> None:
    """Test hook: the next mxq_linear_batch call leaves out one weight copy and bounds its waits (see mxq.h)."""
    _check(lib().mxq_debug_batch_fault(int(unit), int(wait_us)), "mxq_debug_batch_fault")
