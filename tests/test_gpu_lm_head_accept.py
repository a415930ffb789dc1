"""GPU parity of the fused vocabulary projection + greedy verification (mxq_lm_head_accept) against the oracle
composed of its linear layer, its argmax and its accept walk."""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth
from parity import gpu_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def no_gave_up_waits():
    yield
    assert mxq.mxq_linear_device_status() == 0


def oracle_tokens(xbits, codes, scales):
    """Verifier tokens from the FP64 logits, and for every row the set of indices the FP32 path may legitimately pick:
    those whose FP64 logit lies within the layer's tolerance (2e-3 * sum|x w^| + 1e-6, twice: both candidates move) of
    the maximum."""
    y64, a64 = oracle.linear(xbits, codes, scales)
    tok = oracle.argmax(y64.astype(np.float32))
    allowed = []
    for r in range(y64.shape[0]):
        top = y64[r].max()
        tol = 2e-3 * a64[r] + 1e-6
        allowed.append(set(np.nonzero(y64[r] + tol >= top - tol[int(np.argmax(y64[r]))])[0].tolist()))
    return y64, tok, allowed


def run(r, v, k, t, seed, accept_upto=None, ws=None):
    w = synth.bits_of(synth.weight(4, seed, v, k))
    x = synth.bits_of(synth.activations(4, seed, r, k))
    codes, scales, _ = oracle.quantize(w)
    y64, tok, allowed = oracle_tokens(x, codes, scales)
    # a draft that agrees with the verifier up to position accept_upto (exclusive) and differs there
    draft = None
    if t > 0:
        d = tok[:t].astype(np.int32).copy()
        if accept_upto is not None and accept_upto < t:
            d[accept_upto] = (d[accept_upto] + 1 + seed) % v
        draft = torch.from_numpy(d).cuda()
    ver, g, nxt = mxq.mxq_lm_head_accept(gpu_bf16(x), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(),
                                         draft, workspace=ws)
    torch.cuda.synchronize()
    ver = ver.cpu().numpy()
    for row in range(r):
        assert int(ver[row]) in allowed[row], (row, int(ver[row]), int(tok[row]))
    # the walk over the draft is integer work on the tokens the kernel itself found: exact
    d = np.zeros((1, max(t, 1)), np.int32) if t == 0 else draft.cpu().numpy().reshape(1, t)
    if t == 0:
        assert int(g[0]) == 0 and int(nxt[0]) == int(ver[0])
    else:
        g_ref, n_ref = oracle.greedy_accept_tokens(d, ver.reshape(1, r))
        assert int(g[0]) == int(g_ref[0]) and int(nxt[0]) == int(n_ref[0])
        if all(len(a) == 1 for a in allowed):   # no near-ties: the oracle's own tokens decide
            g_o, n_o = oracle.greedy_accept_tokens(d, tok.reshape(1, r).astype(np.int32))
            assert int(g[0]) == int(g_o[0]) and int(nxt[0]) == int(n_o[0])
    return ver, int(g[0]), int(nxt[0])


@pytest.mark.parametrize("r,t", [(1, 0), (1, 1), (2, 1), (3, 3), (5, 4), (9, 8), (16, 16), (16, 15)])
@pytest.mark.parametrize("v,k", [(32000, 768), (5000, 1024), (1000, 4096)])
def test_fused_equals_composed_oracle(r, t, v, k):
    for upto in sorted({0, t // 2, t}):
        run(r, v, k, t, seed=r + t, accept_upto=upto)


@pytest.mark.parametrize("r,t,v", [(1, 0, 32000), (2, 1, 32000), (5, 4, 32000), (9, 8, 32000), (1, 0, 48000), (3, 2, 48000),
                                   (16, 15, 50304)])
def test_full_vocabulary_sizes(r, t, v):
    """The launch configurations of the vocabulary projections bench.py times (one CTA per SM walking several tiles)."""
    k = 4096
    w = synth.bits_of(synth.weight(4, 0, v, k))
    x = synth.bits_of(synth.activations(4, 0, r, k))
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    y = mxq.mxq_linear(gpu_bf16(x), gc, gs)                      # checked against the oracle in test_gpu_linear.py
    tok = torch.argmax(y, dim=1).to(torch.int32)
    draft = tok[:t].clone() if t else None
    if t:
        draft[t // 2] = (draft[t // 2] + 7) % v
    ver, g, nxt = mxq.mxq_lm_head_accept(gpu_bf16(x), gc, gs, draft)
    torch.cuda.synchronize()
    assert torch.equal(ver, tok)                                  # same FP32 sums, same argmax rule
    if t:
        assert int(g[0]) == t // 2 and int(nxt[0]) == int(tok[t // 2])
    else:
        assert int(g[0]) == 0 and int(nxt[0]) == int(tok[0])


@pytest.mark.parametrize("r,t,v", [(1, 0, 32000), (9, 8, 32000), (16, 15, 32000), (1, 0, 128256), (12, 11, 128256)])
def test_full_vocabulary_sizes_against_the_oracle(r, t, v):
    """The same launch configurations (at 12 rows on 128256 x 4096 the call runs unfused: plain layer, argmax of every
    row, walk over the draft) against the ORACLE's FP64 logits: every token the kernel picks must lie within the layer's
    tolerance of the row's FP64 maximum, and the accept length / next token must follow from those tokens exactly."""
    run(r, v, 4096, t, seed=40 + r, accept_upto=t // 2)


def test_workspace_is_left_reusable_and_ties_go_to_the_lowest_index():
    v, k, r = 384, 256, 3
    # identical weight rows: every logit of a row of X is the same number -> token 0 everywhere
    w = np.tile(synth.bits_of(synth.weight(4, 1, 1, k)), (v, 1))
    x = synth.bits_of(synth.activations(4, 1, r, k))
    gc, gs = mxq.mxq_quantize(gpu_bf16(w))
    ws = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(r, v, k))
    for _ in range(3):
        ver, g, nxt = mxq.mxq_lm_head_accept(gpu_bf16(x), gc, gs, torch.zeros(2, dtype=torch.int32, device="cuda"), workspace=ws)
        torch.cuda.synchronize()
        assert ver.tolist() == [0, 0, 0] and int(g[0]) == 2 and int(nxt[0]) == 0
    assert int(ws[:2176].to(torch.int64).sum()) == 0   # keys and ticket are zero again


@pytest.mark.parametrize("r,t", [(1, 0), (4, 3), (9, 8)])
def test_codes_that_are_only_16_byte_aligned(r, t):
    """`codes` 16 bytes into an allocation: the FP8-operand kernel (32-byte aligned bases only) is ruled out, and a
    workspace of the size the query names must still be enough whichever path the call then takes."""
    v, k = 3000, 1024
    w = synth.bits_of(synth.weight(4, 9, v, k))
    x = synth.bits_of(synth.activations(4, 9, r, k))
    codes, scales, _ = oracle.quantize(w)
    y64, tok, allowed = oracle_tokens(x, codes, scales)
    raw = torch.empty(codes.size + 64, dtype=torch.uint8, device="cuda")
    off = 16 if raw.data_ptr() % 32 == 0 else 32 - raw.data_ptr() % 32 + 16   # 16 mod 32
    gc = raw[off:off + codes.size].view(v, k // 2)
    gc.copy_(torch.from_numpy(codes))
    assert gc.data_ptr() % 32 == 16
    ws = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(r, v, k))
    draft = torch.from_numpy(tok[:t].astype(np.int32)).cuda() if t else None
    ver, g, nxt = mxq.mxq_lm_head_accept(gpu_bf16(x), gc, torch.from_numpy(scales).cuda(), draft, workspace=ws)
    torch.cuda.synchronize()
    for row in range(r):
        assert int(ver[row]) in allowed[row]


def test_nan_and_minus_inf_are_never_selected():
    v, k = 256, 128
    codes = np.zeros((v, k // 2), np.uint8)
    scales = np.full((v, k // 32), 127, np.uint8)
    codes[:, 0] = 0x02                       # every row: weight 1.0 at k = 0 -> logit = x[0]
    codes[7, 0] = 0x04                       # row 7: weight 2.0
    scales[3, 0] = 0xFF                      # row 3: NaN
    x = np.zeros((2, k), np.float32)
    x[0, 0] = 1.5                            # logits 1.5 everywhere, 3.0 at 7, NaN at 3 -> 7
    x[1, 0] = -2.0                           # logits -2 everywhere, -4 at 7, NaN at 3 -> 0
    xb = (x.view(np.uint32) >> 16).astype(np.uint16)
    ver, g, nxt = mxq.mxq_lm_head_accept(gpu_bf16(xb), torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(),
                                         torch.tensor([7], dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert ver.tolist() == [7, 0] and int(g[0]) == 1 and int(nxt[0]) == 0


@pytest.mark.parametrize("cap", ["mma", "generic"])
@pytest.mark.parametrize("r,t,v,k", [(1, 0, 3000, 96), (4, 3, 3000, 96), (3, 3, 2000, 1024)])
def test_without_a_tcgen05_kernel_the_logits_pass_through_the_workspace(cap, r, t, v, k):
    prev = mxq.mxq_set_linear_kernel(cap)
    try:
        assert mxq.mxq_linear_plan_info(r, v, k)["kernel"] in ("mma", "generic")
        run(r, v, k, t, seed=3, accept_upto=t // 2)
    finally:
        mxq.mxq_set_linear_kernel(prev)
