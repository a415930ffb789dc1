"""The speculative-decoding loop (specdec.decode; Sec. III-A, III-B, III-C) on the library's kernels, with every
acceptance taken from the kernels' own tokens, checked pass by pass against the oracle.

The model is a small stand-in with the structure the loop needs and nothing else: the next token is the argmax of
Head . h, h = the embedding of the current token plus a position vector pushed through L layers h <- h + W_l h (BF16
activations between layers).  The target runs on unquantised BF16 weights (mxq_linear_bf16, logits through
mxq_greedy_accept); the draft is its MXFP4 direct cast (mxq_linear_residual, mxq_lm_head_accept), which is the paper's
set-up: same model, quantised weights, so many proposals are accepted and some are not; a third level uses only the first
layer of the cast.  The oracle twin computes the same chain in FP64 (oracle.linear_bf16 / oracle.linear_residual /
oracle.linear), rounding the activations to BF16 where the GPU does.

Checked:
  (1) on the oracle alone, speculative decoding returns exactly the target's own greedy decoding (the defining property);
  (2) every pass the GPU loop makes is replayed on the oracle with the same input tokens: each token the kernels chose
      must lie within the layer's tolerance of the FP64 maximum of its row (the margin rule of the fused-verification
      tests; decisions are compared pass by pass, so one thin decision cannot cascade), and the accept length and next
      token must follow from the kernels' tokens exactly (integer work, checked with oracle.greedy_accept_tokens);
  (3) the stream the GPU loop returns is a greedy decoding of the target in the same sense: token i + 1 is an allowed
      argmax of the oracle's target at (token i, position i);
  (4) the tally is consistent (proposals = rounds x N, tokens = accepted + rounds) and, for two levels, satisfies Eq. 1
      at the acceptance it observed; the quantised draft is accepted sometimes and refused sometimes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import specdec, synth
from parity import gpu_bf16

pytestmark = pytest.mark.gpu

V, H, LAYERS, POSITIONS = 2000, 768, 3, 64


def bf16_bits_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v):
    """Round to nearest even (through FP32, as the GPU's FP32 sums are)."""
    u = np.asarray(v, np.float64).astype(np.float32).view(np.uint32)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


class Weights:
    def __init__(self, seed):
        self.emb = synth.bits_of(synth.normal_bf16((V, H), 1.0, seed))
        self.pos = synth.bits_of(synth.normal_bf16((POSITIONS, H), 0.5, seed + 1))
        self.layers = [synth.bits_of(synth.normal_bf16((H, H), 0.03, seed + 2 + i)) for i in range(LAYERS)]
        self.head = synth.bits_of(synth.normal_bf16((V, H), 0.02, seed + 50))
        self.q_layers = [oracle.quantize(w)[:2] for w in self.layers]
        self.q_head = oracle.quantize(self.head)[:2]

    def rows(self, toks, pos):
        """Input activations [R, H] as BF16 bits: embedding + position vector, rounded to BF16."""
        h = np.stack([bf16_bits_to_f64(self.emb[t]) + bf16_bits_to_f64(self.pos[(pos + j) % POSITIONS]) for j, t in enumerate(toks)])
        return f64_to_bf16_bits(h)


def allowed_tokens(y64, a64, rel):
    """Per row: the indices whose FP64 logit lies within the tolerance (both candidates may move) of the row's maximum."""
    out = []
    for r in range(y64.shape[0]):
        top = int(np.argmax(y64[r]))
        tol = rel * a64[r] + 1e-6
        out.append(set(np.nonzero(y64[r] + tol >= y64[r, top] - tol[top])[0].tolist()))
    return out


class OracleModel:
    def __init__(self, w, quantised, layers):
        self.w, self.quantised, self.nl = w, quantised, layers
        self.rel = 2e-3 if quantised else 1e-3

    def logits(self, toks, pos):
        h = self.w.rows(toks, pos)
        for i in range(self.nl):
            if self.quantised:
                y, _ = oracle.linear_residual(h, self.w.q_layers[i][0], self.w.q_layers[i][1], bf16_bits_to_f64(h))
            else:
                y, _ = oracle.linear_bf16(h, self.w.layers[i])
                y = y + bf16_bits_to_f64(h)
            h = f64_to_bf16_bits(y)
        return oracle.linear(h, self.w.q_head[0], self.w.q_head[1]) if self.quantised else oracle.linear_bf16(h, self.w.head)

    def tokens(self, toks, pos):
        return np.argmax(self.logits(toks, pos)[0], axis=1).astype(np.int32)

    def next(self, cur, pos):
        return int(self.tokens([cur], pos)[0])

    def verify(self, cur, pos, proposals):
        ver = self.tokens([cur] + list(proposals), pos)
        g, nxt = oracle.greedy_accept_tokens(np.asarray(proposals, np.int32).reshape(1, -1), ver.reshape(1, -1))
        return int(g[0]), int(nxt[0])


class GpuModel:
    """The same model on the library's kernels.  Only the embedding lookup (a host-side table read) and, for the BF16
    target, the residual add between its layers are done outside them."""

    def __init__(self, w, quantised, layers):
        self.w, self.quantised, self.nl = w, quantised, layers
        self.passes = []   # (input tokens, position, proposals, kernels' row tokens or None, G, next token)
        if quantised:
            self.layers = [(torch.from_numpy(c).cuda(), torch.from_numpy(s).cuda()) for c, s in w.q_layers[:layers]]
            self.head = (torch.from_numpy(w.q_head[0]).cuda(), torch.from_numpy(w.q_head[1]).cuda())
            self.ws_layer = mxq.new_workspace(max(16, mxq.mxq_linear_fused_workspace_bytes(16, H, H)))
            self.ws_head = {}
        else:
            self.layers = [gpu_bf16(x) for x in w.layers[:layers]]
            self.head = gpu_bf16(w.head)

    def hidden(self, toks, pos):
        h = gpu_bf16(self.w.rows(toks, pos))
        for i in range(self.nl):
            if self.quantised:
                h = mxq.mxq_linear_residual(h, self.layers[i][0], self.layers[i][1], h, workspace=self.ws_layer)
            else:
                h = (mxq.mxq_linear_bf16(h, self.layers[i]) + h.float()).to(torch.bfloat16)
        return h

    def run(self, toks, pos, draft):
        h = self.hidden(toks, pos)
        r = len(toks)
        d = torch.tensor(draft, dtype=torch.int32, device="cuda") if draft else None
        ver = None
        if self.quantised:
            if r not in self.ws_head:
                self.ws_head[r] = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(r, V, H))
            ver, g, nxt = mxq.mxq_lm_head_accept(h, self.head[0], self.head[1], d, workspace=self.ws_head[r])
            ver = ver.cpu().numpy()
        else:
            logits = mxq.mxq_linear_bf16(h, self.head).view(1, r, V)
            if d is None:   # a plain step: one row, one (never matching) stand-in proposal; the next token is the argmax
                g, nxt = mxq.mxq_greedy_accept(logits, torch.full((1, 1), -1, dtype=torch.int32, device="cuda"))
            else:
                g, nxt = mxq.mxq_greedy_accept(logits, d.view(1, -1))
        self.passes.append((list(toks), pos, list(draft) if draft else [], ver, int(g[0]), int(nxt[0])))
        return int(g[0]), int(nxt[0])

    def next(self, cur, pos):
        return self.run([cur], pos, None)[1]

    def verify(self, cur, pos, proposals):
        return self.run([cur] + list(proposals), pos, list(proposals))


@pytest.mark.parametrize("levels,n,tokens", [(2, [4], 96), (2, [7], 96), (3, [4, 3], 64)])
def test_decoding_with_the_kernels_own_tokens(levels, n, tokens):
    w = Weights(7000 + levels)
    depth = [LAYERS, LAYERS, 1][:levels]
    o_models = [OracleModel(w, i > 0, depth[i]) for i in range(levels)]
    g_models = [GpuModel(w, i > 0, depth[i]) for i in range(levels)]
    first = 11
    # (1) speculative decoding changes nothing about the output: the target alone produces the same tokens
    o_out, _ = specdec.decode(o_models, n, first, tokens)
    plain, _ = specdec.decode([OracleModel(w, False, LAYERS)], [], first, len(o_out))
    assert plain == o_out

    g_out, tally = specdec.decode(g_models, n, first, tokens)
    torch.cuda.synchronize()
    assert mxq.mxq_linear_device_status() == 0 and len(g_out) >= tokens
    # (2) every pass of the GPU loop against the oracle on the same inputs
    for lvl, (gm, om) in enumerate(zip(g_models, o_models)):
        assert len(gm.passes) == tally.steps[lvl]
        for toks, pos, draft, ver, g, nxt in gm.passes:
            y64, a64 = om.logits(toks, pos)
            ok = allowed_tokens(y64, a64, om.rel)
            if ver is not None:   # the fused verification reports the token of every row
                for r in range(len(toks)):
                    assert int(ver[r]) in ok[r], (lvl, toks, pos, r)
                if draft:
                    g_ref, n_ref = oracle.greedy_accept_tokens(np.asarray(draft, np.int32).reshape(1, -1), ver.reshape(1, -1).astype(np.int32))
                    assert (g, nxt) == (int(g_ref[0]), int(n_ref[0]))
                else:
                    assert g == 0 and nxt == int(ver[0])
            else:                 # logits + mxq_greedy_accept: G proposals agreed with the row's choice, the next one did not
                assert all(draft[j] in ok[j] for j in range(g)) and nxt in ok[g]
                assert g == len(draft) or nxt != draft[g]
    # (3) the returned stream is a greedy decoding of the target
    cur = first
    for i, t in enumerate(g_out):
        y64, a64 = o_models[0].logits([cur], i)
        assert t in allowed_tokens(y64, a64, o_models[0].rel)[0], i
        cur = t
    # (4) the tally
    for lvl in range(levels - 1):
        assert tally.proposed[lvl] == tally.steps[lvl] * n[lvl]
        assert 0 < tally.accepted[lvl] < tally.proposed[lvl], "the quantised draft was never accepted, or never refused"
    produced = tally.accepted[0] + tally.steps[0]
    assert produced == len(g_out)
    if levels == 2:
        alpha = tally.accepted[0] / tally.proposed[0]
        for s_ in (1.77, 3.76):   # Eq. 1 at the observed acceptance, for a measured and for the byte-count ratio of step times
            assert produced / tally.time([1.0, 1.0 / s_]) == pytest.approx(specdec.eq1_speedup(alpha, n[0], s_), rel=1e-12)
