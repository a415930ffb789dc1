"""Seeded synthetic inputs for the MXFP4 weight-only linear path.

This module only *draws numbers and arranges them*: it holds none of the
method's arithmetic (no quantisation, no dequantisation, no matrix product,
no argmax).  Tests and the benchmark hand the very same bits to the CPU
oracle and to the CUDA library.

Shapes follow the Llama-family models of the paper's evaluation (Sec. IV-A:
a 7B target, a 68M draft) and its 8192x8192 GEMM micro-benchmark
(Sec. IV-D); values are random because the path is data-oblivious.

Seeding rule: tensor ``i`` of config ``c`` uses seed ``1000*c + i``
(config 1, the tiny case, uses seed 0 for its weight).
"""
from __future__ import annotations

import numpy as np
import torch

MX_BLOCK = 32

# (name, N = output features, K = input features)
LAYERS_68M = [("q", 768, 768), ("k", 768, 768), ("v", 768, 768), ("o", 768, 768),
              ("gate", 3072, 768), ("up", 3072, 768), ("down", 768, 3072), ("lm_head", 32000, 768)]
LAYERS_7B = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
             ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LAYERS_13B = [("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
              ("gate", 13824, 5120), ("up", 13824, 5120), ("down", 5120, 13824)]
LM_HEADS = [("lm_head_32k", 32000, 4096), ("lm_head_128k", 128256, 4096)]
PAPER_GEMM = ("gemm_8192", 8192, 8192)


def seed_for(config: int, index: int) -> int:
    return 0 if (config == 1 and index == 0) else 1000 * config + index


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def bits_of(t: torch.Tensor) -> np.ndarray:
    """BF16 tensor -> host uint16 array holding the same bit patterns."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(bits: np.ndarray, device="cpu") -> torch.Tensor:
    """uint16 bit patterns -> BF16 tensor on ``device``."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return torch.from_numpy(b.view(np.int16)).to(device).view(torch.bfloat16)


def normal_bf16(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std^2) drawn in FP32, rounded to BF16 (nearest even)."""
    g = _gen(seed, device)
    return (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)


def student_t_bf16(shape, std: float, seed: int, nu: int = 5, device="cpu", chunk_rows: int = 2048) -> torch.Tensor:
    """Student-t(nu) scaled to standard deviation ``std`` (variance of t_nu is nu/(nu-2))."""
    n, k = shape
    g = _gen(seed, device)
    out = torch.empty((n, k), dtype=torch.bfloat16, device=device)
    scale = std / (nu / (nu - 2.0)) ** 0.5
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        z = torch.randn((r1 - r0, k), generator=g, device=device, dtype=torch.float32)
        chi2 = torch.zeros_like(z)
        for _ in range(nu):
            chi2 += torch.randn((r1 - r0, k), generator=g, device=device, dtype=torch.float32) ** 2
        out[r0:r1] = (z / torch.sqrt(chi2 / nu) * scale).to(torch.bfloat16)
    return out


def add_outliers_(w: torch.Tensor, seed: int, frac: float = 1e-3, factor: float = 20.0) -> torch.Tensor:
    """Multiply a seeded fraction of entries by ``factor`` (in place)."""
    g = _gen(seed, w.device)
    cnt = max(1, int(round(w.numel() * frac)))
    idx = torch.randint(0, w.numel(), (cnt,), generator=g, device=w.device)
    flat = w.view(-1)
    flat[idx] = (flat[idx].float() * factor).to(torch.bfloat16)
    return w


def hand_blocks_bits() -> dict:
    """BF16 bit patterns of the special blocks the direct cast must survive.

    Keys: 'clamp_low' (values straddling the smallest scale), 'subnormal'
    (BF16 subnormals), 'scale_one' (largest element just above 2^-124),
    'top' (largest finite BF16), 'zeros', 'neg_zero'.
    """
    def f2b(x: float) -> int:
        return int(np.array([x], np.float32).view(np.uint32)[0] >> 16)

    blocks = {}
    b = np.zeros(MX_BLOCK, np.uint16)
    for i, e in enumerate([-125, -126, -127, -128, -129]):
        b[i] = f2b(2.0 ** e)
    blocks["clamp_low"] = b
    b = np.zeros(MX_BLOCK, np.uint16)
    b[0], b[1], b[2], b[3] = f2b(2.0 ** -130), f2b(2.0 ** -128), f2b(-(2.0 ** -129)), f2b(3 * 2.0 ** -128)
    blocks["subnormal"] = b
    b = np.zeros(MX_BLOCK, np.uint16)
    b[0], b[1] = f2b(1.75 * 2.0 ** -124), f2b(2.0 ** -126)
    blocks["scale_one"] = b
    b = np.zeros(MX_BLOCK, np.uint16)
    b[0], b[1], b[2] = 0x7F7F, 0xFEFF, 0x7E7F  # max, -max/2, max/4
    blocks["top"] = b
    blocks["zeros"] = np.zeros(MX_BLOCK, np.uint16)
    b = np.zeros(MX_BLOCK, np.uint16)
    b[5] = 0x8000
    blocks["neg_zero"] = b
    return blocks


def inject_edge_blocks_(w: torch.Tensor, seed: int, frac_zero: float = 1e-3, frac_tiny: float = 1e-3) -> torch.Tensor:
    """Zero a seeded fraction of 32-blocks, push another fraction down by 2^-125
    (into the BF16 subnormal range) and plant the hand blocks (in place)."""
    n, k = w.shape
    nblk = n * k // MX_BLOCK
    g = _gen(seed, w.device)
    blocks = w.view(nblk, MX_BLOCK)
    nz = max(1, int(round(nblk * frac_zero)))
    nt = max(1, int(round(nblk * frac_tiny)))
    zi = torch.randint(0, nblk, (nz,), generator=g, device=w.device)
    ti = torch.randint(0, nblk, (nt,), generator=g, device=w.device)
    blocks[zi] = 0
    blocks[ti] = (blocks[ti].float() * (2.0 ** -125)).to(torch.bfloat16)
    planted = torch.randint(0, nblk, (8,), generator=g, device=w.device).tolist()
    for pos, (_, bits) in zip(planted, sorted(hand_blocks_bits().items())):
        blocks[pos] = from_bits(bits, w.device)
    return w


def weight(config: int, index: int, n: int, k: int, device="cpu") -> torch.Tensor:
    """The BF16 weight matrix [n,k] of tensor ``index`` of benchmark config ``config``."""
    seed = seed_for(config, index)
    if config in (1, 4):
        return normal_bf16((n, k), 0.02, seed, device)
    if config == 2:
        w = normal_bf16((n, k), 0.02, seed, device)
        return add_outliers_(w, seed + 500)
    if config == 3:
        return student_t_bf16((n, k), 0.02, seed, device=device)
    if config == 5:
        w = student_t_bf16((n, k), 0.02, seed, device=device)
        return inject_edge_blocks_(w, seed + 500)
    raise ValueError("config must be 1..5")


def activations(config: int, index: int, m: int, k: int, device="cpu") -> torch.Tensor:
    """BF16 X[m,k] ~ N(0,1)."""
    return normal_bf16((m, k), 1.0, seed_for(config, 100 + index), device)


def accept_trials(b: int, t: int, r: int, v: int, seed: int, dtype=torch.float32, device="cpu", n_ties: int = 4):
    """Speculated sequences with a planted verifier choice.

    logits[b,r,:] ~ N(0,1) except one planted entry per row raised to 12.0
    (far above the largest of ``v`` standard normal draws), so the verifier's
    greedy token of every row is known by construction without computing an
    argmax here.  The draft agrees with it before a uniformly drawn mismatch
    position p in {0..t}, differs at p, and afterwards agrees with probability
    1/2 (agreement after the first mismatch must not count).  In the first
    ``n_ties`` sequences row 0 gets a second entry with exactly the planted
    value at a *higher* index, so the lowest index must win the tie.

    Returns (logits [b,r,v], draft int32 [b,t], planted int32 [b,r], p int32 [b]).
    """
    g = _gen(seed, device)
    logits = torch.randn((b, r, v), generator=g, device=device, dtype=torch.float32)
    planted = torch.randint(0, v, (b, r), generator=g, device=device)
    logits.scatter_(2, planted.unsqueeze(-1), 12.0)
    for i in range(min(n_ties, b)):
        lo = int(planted[i, 0])
        if lo + 1 < v:
            logits[i, 0, lo + 1 + (i * 7919) % (v - lo - 1)] = 12.0
    p = torch.randint(0, t + 1, (b,), generator=g, device=device)
    pos = torch.arange(t, device=device).unsqueeze(0)
    agree_after = torch.rand((b, t), generator=g, device=device) < 0.5
    rand_tok = torch.randint(0, v, (b, t), generator=g, device=device)
    ver_t = planted[:, :t]
    offset = torch.randint(1, v, (b, t), generator=g, device=device)  # 1..v-1, never 0 mod v
    wrong = (ver_t + offset) % v
    draft = torch.where(pos < p.unsqueeze(1), ver_t,
                        torch.where(pos == p.unsqueeze(1), wrong, torch.where(agree_after, ver_t, rand_tok)))
    return logits.to(dtype), draft.to(torch.int32), planted.to(torch.int32), p.to(torch.int32)
