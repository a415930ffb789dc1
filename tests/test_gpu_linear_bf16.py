"""GPU parity of the unquantised comparison layer (mxq_linear_bf16) against its oracle: products of BF16 numbers are
exact in FP32, so only the FP32 accumulation separates the kernel from the FP64 sum: |y - y64| <= 1e-3 * sum|x w| + 1e-6
(K * 2^-24 = 8e-4 at K = 13824)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth
from parity import gpu_bf16

pytestmark = pytest.mark.gpu


def check(m, n, k, seed, out_dtype=torch.float32, rows=None):
    w = synth.bits_of(synth.weight(3, seed, n, k))
    x = synth.bits_of(synth.activations(3, seed, m, k))
    y64, a64 = oracle.linear_bf16(x, w, rows=rows)
    y = mxq.mxq_linear_bf16(gpu_bf16(x), gpu_bf16(w), out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert mxq.mxq_linear_device_status() == 0
    if rows is not None:
        y = y[:, torch.as_tensor(rows, device="cuda")]
    got = y.float().cpu().numpy().astype(np.float64)
    tol = 1e-3 * a64 + 1e-6 + (np.abs(y64) * 2.0 ** -8 if out_dtype == torch.bfloat16 else 0)
    bad = np.abs(got - y64) > tol
    assert not bad.any(), (m, n, k, int(bad.sum()), float(np.abs(got - y64).max()))
    return y


@pytest.mark.parametrize("m", [1, 2, 5, 8, 16])
@pytest.mark.parametrize("n,k", [(203, 1408), (128, 64), (1, 128), (1000, 4096), (300, 5120)])
def test_ragged_and_small_shapes(m, n, k):
    check(m, n, k, seed=m)


@pytest.mark.parametrize("m", [1, 8])
@pytest.mark.parametrize("n,k", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_7b_layers_sampled_rows(n, k, m):
    rows = np.unique(np.concatenate([[0, n - 1], np.random.default_rng(n + k).integers(0, n, 300)])).astype(np.int64)
    check(m, n, k, seed=2, rows=rows)


@pytest.mark.parametrize("n,k", [(37, 96), (5, 2), (130, 4090)])
def test_shapes_outside_the_tensor_core_path(n, k):
    check(3, n, k, seed=9)


def test_bf16_output_and_canaries():
    y32 = check(4, 515, 2048, seed=4)
    y16 = check(4, 515, 2048, seed=4, out_dtype=torch.bfloat16)
    assert torch.equal(y16, y32.to(torch.bfloat16))
    w = gpu_bf16(synth.bits_of(synth.weight(3, 4, 515, 2048)))
    x = gpu_bf16(synth.bits_of(synth.activations(3, 4, 4, 2048)))
    buf = torch.full((4 * 515 + 64,), 777.0, dtype=torch.float32, device="cuda")
    mxq.mxq_linear_bf16(x, w, out=buf[32:32 + 4 * 515].view(4, 515))
    torch.cuda.synchronize()
    assert (buf[:32] == 777.0).all() and (buf[32 + 4 * 515:] == 777.0).all()
