"""A decoder's dependent chain of calls issued back to back, with no host synchronisation between them.

Every single-call kernel starts while the call before it is still running (programmatic dependent launch): it may touch
its inputs only after its dependency wait, and only through loads that the wait covers.  A layer is four calls whose
outputs feed the next call through the same buffers for every layer, so a kernel that reads an input too early, or from a
cache the wait does not cover, computes from the PREVIOUS layer's activations.  (It did, for the token rows rewritten by
the separate kernel of the 3..16-row path and of two rows on large K: its loads went through the non-coherent path.)

Checked, for 1..16 token rows and under every kernel choice:
  (1) the chain issued asynchronously gives bit for bit what the same chain gives with a device synchronisation after
      every call;
  (2) the last layer of the asynchronous run satisfies the oracle's bounds stage by stage, each stage's oracle fed with
      the GPU's own inputs of that stage -- which are the last layer's only if nothing was read early.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth
from parity import ABS, REL, gpu_bf16

pytestmark = pytest.mark.gpu


def values(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


class Chain:
    """L layers of {q/k/v as one matrix; o + residual; gate/up with SiLU(gate) * up; down + residual}, BF16 in and out,
    every layer through the same five activation buffers and one workspace."""

    def __init__(self, m, h, f, layers, seed):
        self.m, self.h, self.f = m, h, f
        self.w = []
        for li in range(layers):
            mats = []
            for j, (n, k) in enumerate([(3 * h, h), (h, h), (2 * f, h), (h, f)]):
                codes, scales, _ = oracle.quantize(synth.bits_of(synth.weight(3, seed + 4 * li + j, n, k)))
                mats.append((codes, scales, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()))
            self.w.append(mats)
        self.h0 = gpu_bf16(synth.bits_of(synth.activations(3, seed, m, h)))
        self.att = gpu_bf16(synth.bits_of(synth.activations(3, seed + 1, m, h)))
        bf = dict(dtype=torch.bfloat16, device="cuda")
        self.qkv, self.h1 = torch.empty((m, 3 * h), **bf), torch.empty((m, h), **bf)
        self.act, self.h2 = torch.empty((m, f), **bf), torch.empty((m, h), **bf)
        need = max(mxq.mxq_linear_fused_workspace_bytes(m, n, k) for n, k in [(3 * h, h), (h, h), (2 * f, h), (h, f)])
        self.ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")

    def run(self, sync):
        def step():
            if sync:
                torch.cuda.synchronize()
        for (wqkv, wo, wgu, wd) in self.w:
            mxq.mxq_linear(self.h0, wqkv[2], wqkv[3], out=self.qkv, workspace=self.ws)
            step()
            mxq.mxq_linear_residual(self.att, wo[2], wo[3], self.h0, out=self.h1, workspace=self.ws)
            step()
            mxq.mxq_linear_swiglu(self.h1, wgu[2], wgu[3], out=self.act, workspace=self.ws)
            step()
            mxq.mxq_linear_residual(self.act, wd[2], wd[3], self.h1, out=self.h2, workspace=self.ws)
            step()
        torch.cuda.synchronize()
        return [t.clone() for t in (self.qkv, self.h1, self.act, self.h2)]

    def batches(self, one_call_per_layer):
        """The same chain through mxq_linear_batch: four calls per layer (each waits for the one before it), or one call of
        three dependent groups per layer."""
        out = []
        for (wqkv, wo, wgu, wd) in self.w:
            lays = [dict(x=self.h0, codes=wqkv[2], scales=wqkv[3], out=self.qkv),
                    dict(x=self.att, codes=wo[2], scales=wo[3], out=self.h1, epilogue="residual", residual=self.h0),
                    dict(x=self.h1, codes=wgu[2], scales=wgu[3], out=self.act, epilogue="swiglu", depends=True),
                    dict(x=self.act, codes=wd[2], scales=wd[3], out=self.h2, epilogue="residual", residual=self.h1, depends=True)]
            if one_call_per_layer:
                out.append(mxq.LinearBatch(lays))
            else:
                out += [mxq.LinearBatch([dict(lay, depends=False)]) for lay in lays]
        return out

    def run_batches(self, batches, ws, sync):
        for b in batches:
            b.run(ws)
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        return [t.clone() for t in (self.qkv, self.h1, self.act, self.h2)]

    def check_last_layer(self, rows_of=lambda n: None):
        """Oracle bounds on the buffers as the last run left them (they hold the last layer's values)."""
        wqkv, wo, wgu, wd = self.w[-1]
        bf = lambda want: np.abs(want) * 2.0 ** -8
        h0, att = synth.bits_of(self.h0.cpu()), synth.bits_of(self.att.cpu())
        h1, act = synth.bits_of(self.h1.cpu()), synth.bits_of(self.act.cpu())

        def within(got, want, tol, what):
            assert np.isfinite(got).all(), what
            worst = float((np.abs(got - want) / tol).max())
            assert worst <= 1.0, "%s: error/tolerance = %.3g" % (what, worst)

        rows = rows_of(3 * self.h)
        sel = slice(None) if rows is None else rows
        y64, a64 = oracle.linear(h0, wqkv[0], wqkv[1], rows=rows)
        within(values(self.qkv)[:, sel], y64, REL * a64 + ABS + bf(y64), "q/k/v")
        rows = rows_of(self.h)
        sel = slice(None) if rows is None else rows
        want, a = oracle.linear_residual(att, wo[0], wo[1], values(self.h0)[:, sel], rows=rows)
        within(values(self.h1)[:, sel], want, REL * a + ABS + 2.0 ** -23 * np.abs(want) + bf(want), "o + residual")
        rows = rows_of(self.f)   # (output columns: each is one gate / up pair of weight rows)
        want, g, u, ag, au = oracle.linear_swiglu(h1, wgu[0], wgu[1], rows=rows)
        tg, tu = REL * ag + ABS, REL * au + ABS
        tol = 1.1 * tg * (np.abs(u) + tu) + np.abs(oracle.silu(g)) * tu + 1e-6 * np.abs(want) + 1e-30 + bf(want)
        got = values(self.act)
        within(got if rows is None else got[:, rows], want, tol, "gate/up")
        rows = rows_of(self.h)
        sel = slice(None) if rows is None else rows
        want, a = oracle.linear_residual(act, wd[0], wd[1], values(self.h1)[:, sel], rows=rows)
        within(values(self.h2)[:, sel], want, REL * a + ABS + 2.0 ** -23 * np.abs(want) + bf(want), "down + residual")


@pytest.mark.parametrize("kernel", ["auto", "umma", "mma", "generic"])
@pytest.mark.parametrize("m", [1, 2, 3, 5, 8, 16])
def test_asynchronous_chain_equals_the_synchronised_one(m, kernel):
    prev = mxq.mxq_set_linear_kernel(kernel)
    try:
        chain = Chain(m, 1024, 2816, layers=3, seed=700)
        ref = chain.run(sync=True)
        for _ in range(3):
            got = chain.run(sync=False)
            for name, a, b in zip(("q/k/v", "o", "gate/up", "down"), ref, got):
                assert torch.equal(a, b), "%s differs between the asynchronous and the synchronised chain (M=%d, %s)" % (name, m, kernel)
        chain.check_last_layer()
        assert mxq.mxq_linear_device_status() == 0
    finally:
        mxq.mxq_set_linear_kernel(prev)


@pytest.mark.parametrize("m", [2, 8])
def test_asynchronous_chain_on_the_7b_shapes(m):
    """The shapes on which the separate rewriting kernel runs at two token rows already (K = 11008)."""
    chain = Chain(m, 4096, 11008, layers=2, seed=720)
    ref = chain.run(sync=True)
    for _ in range(3):
        got = chain.run(sync=False)
        for name, a, b in zip(("q/k/v", "o", "gate/up", "down"), ref, got):
            assert torch.equal(a, b), "%s differs between the asynchronous and the synchronised chain (M=%d)" % (name, m)

    def sampled(n):
        return np.unique(np.concatenate([[0, 1, n - 2, n - 1], np.random.default_rng(n).integers(0, n, 300)])).astype(np.int64)
    chain.check_last_layer(rows_of=sampled)
    assert mxq.mxq_linear_device_status() == 0


@pytest.mark.parametrize("one_call_per_layer", [False, True])
@pytest.mark.parametrize("m", [1, 4, 8, 12])
def test_asynchronous_chain_through_the_batch_call(m, one_call_per_layer):
    """The persistent kernel starts early too, and consecutive calls share one workspace: a call per matrix (each reads what
    the call before it wrote), and a call of three dependent groups per layer (12 rows: two passes over row halves)."""
    chain = Chain(m, 1024, 2816, layers=3, seed=740)
    batches = chain.batches(one_call_per_layer)
    ws = mxq.new_workspace(max(b.workspace_bytes() for b in batches))
    ref = chain.run_batches(batches, ws, sync=True)
    for _ in range(3):
        got = chain.run_batches(batches, ws, sync=False)
        for name, a, b in zip(("q/k/v", "o", "gate/up", "down"), ref, got):
            assert torch.equal(a, b), "%s differs between the asynchronous and the synchronised chain (M=%d)" % (name, m)
    chain.check_last_layer()
    assert mxq.mxq_linear_device_status() == 0


@pytest.mark.parametrize("m", [1, 5, 9])
def test_verification_fused_into_the_projection_at_the_end_of_a_chain(m):
    """mxq_lm_head_accept reads the last layer's output the moment its own wait returns: same tokens, accept length and
    next token with and without synchronisation between the calls."""
    chain = Chain(m, 1024, 2816, layers=2, seed=760)
    codes, scales, _ = oracle.quantize(synth.bits_of(synth.weight(4, 77, 5000, 1024)))
    hc, hs = torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda()
    draft = torch.arange(m - 1, dtype=torch.int32, device="cuda") if m > 1 else None
    ws = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(m, 5000, 1024))

    def run(sync):
        for (wqkv, wo, wgu, wd) in chain.w:
            for call in (lambda: mxq.mxq_linear_residual(chain.att, wo[2], wo[3], chain.h0, out=chain.h1, workspace=chain.ws),
                         lambda: mxq.mxq_linear_swiglu(chain.h1, wgu[2], wgu[3], out=chain.act, workspace=chain.ws),
                         lambda: mxq.mxq_linear_residual(chain.act, wd[2], wd[3], chain.h1, out=chain.h2, workspace=chain.ws)):
                call()
                if sync:
                    torch.cuda.synchronize()
        ver, g, nxt = mxq.mxq_lm_head_accept(chain.h2, hc, hs, draft, workspace=ws)
        torch.cuda.synchronize()
        return ver.clone(), int(g[0]), int(nxt[0])

    ref = run(True)
    for _ in range(3):
        got = run(False)
        assert torch.equal(ref[0], got[0]) and ref[1:] == got[1:]
    # and the tokens are the argmax of the projection of what the chain left in h2 (margin rule of the fused-verification tests)
    y64, a64 = oracle.linear(synth.bits_of(chain.h2.cpu()), codes, scales)
    ver = ref[0].cpu().numpy()
    for r in range(m):
        top = int(np.argmax(y64[r]))
        tol = REL * a64[r] + ABS
        assert y64[r, ver[r]] + tol[ver[r]] >= y64[r, top] - tol[top], r


@pytest.mark.parametrize("m", [1, 2, 8])
def test_chain_replayed_from_a_cuda_graph(m):
    """The benchmark times its chains as replayed graphs (the captured launches keep their programmatic dependences):
    a replay leaves what the synchronised chain leaves."""
    chain = Chain(m, 4096, 11008, layers=2, seed=780)
    ref = chain.run(sync=True)

    def calls():
        for (wqkv, wo, wgu, wd) in chain.w:
            mxq.mxq_linear(chain.h0, wqkv[2], wqkv[3], out=chain.qkv, workspace=chain.ws)
            mxq.mxq_linear_residual(chain.att, wo[2], wo[3], chain.h0, out=chain.h1, workspace=chain.ws)
            mxq.mxq_linear_swiglu(chain.h1, wgu[2], wgu[3], out=chain.act, workspace=chain.ws)
            mxq.mxq_linear_residual(chain.act, wd[2], wd[3], chain.h1, out=chain.h2, workspace=chain.ws)

    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        calls()
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            calls()
        for _ in range(3):
            for t in (chain.qkv, chain.h1, chain.act, chain.h2):
                t.fill_(float("nan"))
            graph.replay()
            graph.replay()
            st.synchronize()
            for name, a, b in zip(("q/k/v", "o", "gate/up", "down"), ref, (chain.qkv, chain.h1, chain.act, chain.h2)):
                assert torch.equal(a, b), "%s differs after a graph replay (M=%d)" % (name, m)
    assert mxq.mxq_linear_device_status() == 0
