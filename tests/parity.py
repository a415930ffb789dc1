"""Helpers shared by the GPU parity tests: the tolerance of the linear layer and small converters."""
import numpy as np
import torch

from paper_2503_13565_b200 import synth

REL, ABS = 2e-3, 1e-6   # |y - y64| <= REL * sum_k |x_k w^_k| + ABS


def check_linear(y_gpu: torch.Tensor, y64: np.ndarray, a64: np.ndarray, what=""):
    """Element-by-element bound; BF16 outputs are widened exactly first."""
    y = y_gpu.detach().float().cpu().numpy().astype(np.float64)
    assert y.shape == y64.shape, (y.shape, y64.shape)
    fmax = float(np.finfo(np.float32).max)
    # where the exact value (give or take the tolerance) is beyond what FP32 can hold, the FP32 result is
    # an infinity of the right sign; everywhere else the output must be finite and within the bound
    over = np.isfinite(y64) & (np.abs(y64) + REL * a64 >= fmax)
    assert (np.isinf(y[over]) & (np.sign(y[over]) == np.sign(y64[over])) | np.isfinite(y[over])).all(), what
    finite = np.isfinite(y64) & ~(over & np.isinf(y))
    assert np.isfinite(y[finite]).all(), what + ": non-finite output where the oracle is finite"
    err = np.abs(y - y64)[finite]
    tol = (REL * a64 + ABS)[finite]
    worst = float((err / tol).max()) if err.size else 0.0
    assert worst <= 1.0, "%s: error/tolerance = %.3g" % (what, worst)
    assert np.isnan(y[np.isnan(y64)]).all(), what + ": NaN expected where a scale byte is 0xFF"
    return worst


def to_np_u8(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def gpu_bf16(bits: np.ndarray) -> torch.Tensor:
    return synth.from_bits(bits, "cuda")
