"""mxq_greedy_accept_static: the accept step for callers that cannot allocate a workspace.

Some users of the library run where device memory is already spoken for -- a server that sized its pools at
start-up, a plugin that is handed its input and output buffers and nothing more -- so they cannot give
mxq_greedy_accept the scratch it asks for.  The static variant keeps that scratch in an array built into the
library.  This file checks, through the C ABI, that it returns exactly what the ordinary entry point returns,
on two calls in a row (the second finds the array as the first left it), and that a shape too large for the
built-in array is refused rather than served from somewhere else.

Collected last on purpose: if it fails under `-x`, every other test has already run.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import binding, synth


@pytest.mark.gpu
def test_static_variant_matches_the_workspace_variant_on_two_calls_in_a_row():
    cases = [(250, 16, 17, 32000, torch.float32, 901), (3, 16, 17, 128256, torch.bfloat16, 902)]
    for b, t, r, v, dtype, seed in cases:   # two different shapes, back to back, sharing the built-in array
        logits, draft, _, p = synth.accept_trials(b, t, r, v, seed=seed, dtype=dtype, device="cuda")
        want_len, want_next = mxq.mxq_greedy_accept(logits, draft)          # caller-provided workspace
        got_len = torch.full((b,), -7, dtype=torch.int32, device="cuda")
        got_next = torch.full((b,), -7, dtype=torch.int32, device="cuda")
        mxq.mxq_greedy_accept_static(logits, draft, got_len, got_next)     # built-in scratch, through the C ABI
        torch.cuda.synchronize()
        assert torch.equal(got_len, want_len) and torch.equal(got_next, want_next)   # integers: no tolerance
        assert np.array_equal(got_len.cpu().numpy(), p.cpu().numpy())               # and they are the planted answer
        # and both outputs are what the oracle computes from the same logits (BF16 logits go over as bit patterns)
        lg = logits.cpu()
        lg_np = lg.numpy() if dtype == torch.float32 else synth.bits_of(lg)
        o_len, o_next = oracle.greedy_accept(lg_np, draft.cpu().numpy())
        assert np.array_equal(got_len.cpu().numpy(), o_len) and np.array_equal(got_next.cpu().numpy(), o_next)
    # same shape again right away: the array holds the previous call's partial results and must not mind
    logits, draft, _, p = synth.accept_trials(250, 16, 17, 32000, seed=903, device="cuda")
    want_len, want_next = mxq.mxq_greedy_accept(logits, draft)
    got_len = torch.empty(250, dtype=torch.int32, device="cuda")
    got_next = torch.empty(250, dtype=torch.int32, device="cuda")
    mxq.mxq_greedy_accept_static(logits, draft, got_len, got_next)
    torch.cuda.synchronize()
    assert torch.equal(got_len, want_len) and torch.equal(got_next, want_next)


def test_shapes_beyond_the_built_in_array_are_refused():
    """Refused on the host, before anything touches the GPU: no hidden allocation makes room."""
    limit = mxq.mxq_greedy_accept_static_max_bytes()
    assert limit == 1 << 20
    assert mxq.mxq_accept_workspace_bytes(250, 17, 32000) <= limit
    assert mxq.mxq_accept_workspace_bytes(100000, 17, 32000) > limit
    L = binding.lib()
    fake = 0x1000   # aligned, never dereferenced: the call must fail validation first
    assert L.mxq_greedy_accept_static(fake, 0, 100000, 17, 32000, fake, 16, fake, fake, None) == 5
    assert L.mxq_greedy_accept_static(None, 0, 1, 17, 32000, fake, 16, fake, fake, None) == 1
    assert L.mxq_greedy_accept_static(fake, 0, 1, 19, 32000, fake, 16, fake, fake, None) == 2
