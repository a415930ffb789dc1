"""Random programs of library calls over a small pool of buffers, run without host synchronisation.

Every kernel of the library that carries the dependent-launch attribute is already running when the call before it
finishes; what keeps a program correct is that each kernel touches what earlier calls wrote (activations, residuals,
re-cast weights, workspaces) only after its dependency wait and through coherent loads, and writes only after it.  The
single-call tests cannot see a violation of that (they synchronise), a fixed chain sees the ones on its own edges.  Here a
seeded generator strings 40 calls together -- plain, residual and gate/up layers, the BF16-weight layer followed by a
torch cast, a re-cast of a weight matrix whose codes the following calls stream, the fused verification, the batch call --
with outputs feeding later inputs through six shared buffers, in place where the call allows it.  The program is run
with a device synchronisation after every call, then three times with none: all buffers, all re-cast weights and all
verification results must come out bit for bit the same.  (Correctness of each call against the oracle is the other
tests' business; this one is about order.)
"""
import random

import pytest
import torch

import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth

pytestmark = pytest.mark.gpu

V = 3000   # a small vocabulary for the fused verification


def same_bits(a, b):
    """Equality of the stored bytes (a NaN equals itself: long programs may overflow BF16, which is no ordering matter)."""
    return torch.equal(a.contiguous().view(torch.uint8), b.contiguous().view(torch.uint8))


class Program:
    def __init__(self, m, seed, steps=40, widths=(1024, 1408), kinds=("lin", "res", "swi", "down", "bf16", "recast", "accept", "batch")):
        """widths: the two activation widths A (hidden) and B (feed-forward), both multiples of 128.  kinds: the calls
        to draw from ("bf16" and "batch" put torch kernels, which never start early, between the library's own)."""
        self.m = m
        A, B = self.A, self.B = widths
        rng = random.Random(seed)
        dev = "cuda"
        cast = lambda w: list(mxq.mxq_quantize(w))
        # (weights a quarter of the benchmark's size, so that forty layers on top of one another stay inside BF16)
        small = lambda cfg, idx, n, k: synth.weight(cfg, idx, n, k, device=dev) * 0.25
        self.src_aa = [small(3, 800 + i, A, A) for i in range(3)]    # BF16 sources, also the BF16-weight layers
        self.w_aa = [cast(w) for w in self.src_aa]                                       # [codes, scales], re-cast in place by "recast"
        self.w_ba = [cast(small(3, 810 + i, 2 * B, A)) for i in range(2)]
        self.w_ab = [cast(small(3, 820 + i, A, B)) for i in range(2)]
        self.head = cast(synth.weight(4, 830, V, A, device=dev))
        self.h0 = [synth.normal_bf16((m, A), 1.0, 840 + i, dev) for i in range(4)]
        self.g0 = [synth.normal_bf16((m, B), 1.0, 850 + i, dev) for i in range(2)]
        self.h = [t.clone() for t in self.h0]
        self.g = [t.clone() for t in self.g0]
        self.f32 = torch.empty((m, A), dtype=torch.float32, device=dev)
        need = max(mxq.mxq_linear_fused_workspace_bytes(m, n, k) for n, k in [(A, A), (2 * B, A), (A, B)])
        self.ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        self.ws_head = mxq.new_workspace(mxq.mxq_lm_head_accept_workspace_bytes(m, V, A))
        self.draft = torch.arange(max(m - 1, 0), dtype=torch.int32, device=dev) if m > 1 else None
        self.ops = []
        for _ in range(steps):
            kind = rng.choice(kinds)
            i, j, k = rng.randrange(4), rng.randrange(4), rng.randrange(4)
            if kind in ("lin", "bf16") and i == j:
                j = (j + 1) % 4          # these two may not run in place
            if kind == "res" and i == j:
                j = (j + 1) % 4          # the output may be the residual (k), never the input
            self.ops.append((kind, i, j, k, rng.randrange(3), rng.randrange(2)))
        self.batch_ws = None
        self.batches = {}

    def reset(self):
        for t, t0 in zip(self.h + self.g, self.h0 + self.g0):
            t.copy_(t0)
        for pair, w in zip(self.w_aa, self.src_aa):
            mxq.mxq_quantize(w, codes=pair[0], scales=pair[1])
        torch.cuda.synchronize()

    def run(self, sync):
        self.reset()
        h, g, A, B = self.h, self.g, self.A, self.B
        seen = []
        for kind, i, j, k, r3, r2 in self.ops:
            if kind == "lin":
                mxq.mxq_linear(h[j], *self.w_aa[r3], out=h[i], workspace=self.ws)
            elif kind == "res":
                mxq.mxq_linear_residual(h[j], *self.w_aa[r3], h[k], out=h[i], workspace=self.ws)
            elif kind == "swi":
                mxq.mxq_linear_swiglu(h[j], *self.w_ba[r2], out=g[i % 2], workspace=self.ws)
            elif kind == "down":
                mxq.mxq_linear_residual(g[j % 2], *self.w_ab[r2], h[k], out=h[i], workspace=self.ws)
            elif kind == "bf16":
                mxq.mxq_linear_bf16(h[j], self.src_aa[r3], out=self.f32)
                h[i].copy_(self.f32.mul(0.25))      # (a foreign kernel between two of the library's)
            elif kind == "recast":
                # the weights the next calls stream are rewritten: a cast of another source (the two alternate)
                mxq.mxq_quantize(self.src_aa[(r3 + 1) % 3], codes=self.w_aa[r3][0], scales=self.w_aa[r3][1])
            elif kind == "accept":
                seen.append(mxq.mxq_lm_head_accept(h[j], *self.head, self.draft, workspace=self.ws_head))
            elif kind in ("batch_direct", "batch_groups"):
                # the batch call writing straight into the shared buffers: no torch kernel anywhere near it
                a_, b_ = (j + 1) % 4, (j + 2) % 4          # two outputs that are not the input h[j]
                if kind == "batch_direct":   # three independent layers (none reads what another writes)
                    lays = [dict(x=h[j], codes=self.w_aa[r3][0], scales=self.w_aa[r3][1], out=h[a_]),
                            dict(x=g[1 - r2], codes=self.w_ab[r2][0], scales=self.w_ab[r2][1], out=h[b_], epilogue="residual", residual=h[b_]),
                            dict(x=h[j], codes=self.w_ba[r2][0], scales=self.w_ba[r2][1], out=g[r2], epilogue="swiglu")]
                else:                        # a dependent chain in three groups: o + residual -> gate/up -> down + residual
                    lays = [dict(x=h[j], codes=self.w_aa[r3][0], scales=self.w_aa[r3][1], out=h[a_], epilogue="residual", residual=h[(j + 3) % 4]),
                            dict(x=h[a_], codes=self.w_ba[r2][0], scales=self.w_ba[r2][1], out=g[r2], epilogue="swiglu", depends=True),
                            dict(x=g[r2], codes=self.w_ab[r2][0], scales=self.w_ab[r2][1], out=h[b_], epilogue="residual", residual=h[a_], depends=True)]
                key = (kind, j, r3, r2)
                if key not in self.batches:
                    self.batches[key] = mxq.LinearBatch(lays)
                    need = self.batches[key].workspace_bytes()
                    if self.batch_ws is None or self.batch_ws.numel() < need:
                        torch.cuda.synchronize()
                        self.batch_ws = mxq.new_workspace(need)
                self.batches[key].run(self.batch_ws)
            else:   # three independent layers in one launch, reading what earlier calls left
                outs = [torch.empty((self.m, A), dtype=torch.bfloat16, device="cuda") for _ in range(2)] + \
                       [torch.empty((self.m, B), dtype=torch.bfloat16, device="cuda")]
                batch = mxq.LinearBatch([dict(x=h[j], codes=self.w_aa[r3][0], scales=self.w_aa[r3][1], out=outs[0]),
                                         dict(x=g[r2], codes=self.w_ab[r2][0], scales=self.w_ab[r2][1], out=outs[1], epilogue="residual", residual=h[k]),
                                         dict(x=h[j], codes=self.w_ba[r2][0], scales=self.w_ba[r2][1], out=outs[2], epilogue="swiglu")])
                if self.batch_ws is None:
                    self.batch_ws = mxq.new_workspace(batch.workspace_bytes())
                batch.run(self.batch_ws)
                h[i].copy_(outs[0])
                h[(i + 1) % 4].copy_(outs[1])
                g[r2].copy_(outs[2])
            if sync:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        state = [t.clone() for t in h + g] + [t.clone() for pair in self.w_aa for t in pair]
        for ver, acc, nxt in seen:
            state += [ver.clone(), acc.clone(), nxt.clone()]
        return state


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("m", [1, 3, 8, 12])
def test_a_program_of_calls_without_synchronisation(m, seed):
    prog = Program(m, 1000 * m + seed)
    ref = prog.run(sync=True)
    assert all(bool(torch.isfinite(t.float()).all()) for t in ref[:6]), "the program's values ran away: not a useful case"
    for attempt in range(3):
        got = prog.run(sync=False)
        for idx, (a, b) in enumerate(zip(ref, got)):
            assert same_bits(a, b), "M=%d seed %d: item %d of the final state differs without synchronisation (attempt %d)" % (m, seed, idx, attempt)
    assert mxq.mxq_linear_device_status() == 0


@pytest.mark.parametrize("only_own_kernels", [False, True])
@pytest.mark.parametrize("m", [2, 8])
def test_a_program_on_the_7b_widths(m, only_own_kernels):
    """The same on hidden 4096 / feed-forward 11008, where the separate rewriting kernel runs from two token rows on and a
    call's CTAs are spread over the whole GPU; once with nothing but the library's own early-starting kernels in the
    stream (every call then overlaps the one before it)."""
    kinds = ("lin", "res", "swi", "down", "accept") if only_own_kernels else ("lin", "res", "swi", "down", "bf16", "recast", "accept", "batch")
    prog = Program(m, 77 + m, steps=32, widths=(4096, 11008), kinds=kinds)
    ref = prog.run(sync=True)
    assert all(bool(torch.isfinite(t.float()).all()) for t in ref[:6])
    for attempt in range(3):
        got = prog.run(sync=False)
        for idx, (a, b) in enumerate(zip(ref, got)):
            assert same_bits(a, b), "M=%d: item %d of the final state differs without synchronisation (attempt %d)" % (m, idx, attempt)
    assert mxq.mxq_linear_device_status() == 0


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 8, 9, 16])
def test_programs_of_the_librarys_own_kernels_only(m, seed):
    """Every call overlaps the one before it: the hardest ordering case, at every kernel choice the token count selects."""
    prog = Program(m, 5000 + 10 * m + seed, steps=32, widths=(4096, 11008), kinds=("lin", "res", "swi", "down", "accept", "recast", "batch_direct", "batch_groups"))
    ref = prog.run(sync=True)
    assert all(bool(torch.isfinite(t.float()).all()) for t in ref[:6]), "the program's values ran away: not a useful case"
    for attempt in range(2):
        got = prog.run(sync=False)
        for idx, (a, b) in enumerate(zip(ref, got)):
            assert same_bits(a, b), "M=%d seed %d: item %d of the final state differs without synchronisation (attempt %d)" % (m, seed, idx, attempt)
    assert mxq.mxq_linear_device_status() == 0
