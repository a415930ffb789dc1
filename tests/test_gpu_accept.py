"""GPU parity of mxq_greedy_accept against the oracle: accept lengths and next tokens identical."""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth

pytestmark = pytest.mark.gpu


def np_logits(lg: torch.Tensor) -> np.ndarray:
    if lg.dtype == torch.bfloat16:
        return synth.bits_of(lg)
    return lg.cpu().numpy()


DEV = "cuda"   # inputs are drawn on the device (fast) and copied to the host for the oracle: same bits


def both(lg: torch.Tensor, draft: torch.Tensor):
    og, on = oracle.greedy_accept(np_logits(lg), draft.cpu().numpy())
    g, nxt = mxq.mxq_greedy_accept(lg.cuda(), draft.cuda())
    torch.cuda.synchronize()
    assert np.array_equal(g.cpu().numpy(), og), np.argwhere(g.cpu().numpy() != og)[:5]
    assert np.array_equal(nxt.cpu().numpy(), on)
    return og, on


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_config4_trials_32k_vocab(dtype):
    """10 000 sequences of 16 speculated tokens, in batches of 250 (each batch is one call)."""
    seen = set()
    for batch in range(40):
        lg, draft, planted, p = synth.accept_trials(250, 16, 17, 32000, seed=4000 + batch, dtype=dtype, device=DEV)
        og, on = both(lg, draft)
        assert np.array_equal(og, p.cpu().numpy())           # the planted mismatch position is what comes out
        seen |= set(og.tolist())
    assert seen == set(range(17))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_large_vocab_single_sequence(dtype):
    for seed in range(6):
        lg, draft, planted, p = synth.accept_trials(1, 16, 17, 128256, seed=4100 + seed, dtype=dtype, device=DEV)
        og, _ = both(lg, draft)
        assert og[0] == int(p[0])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_natural_logits_with_many_ties(dtype):
    """No planted maximum: BF16 rounding makes the largest values tie; the draft follows the oracle's
    own greedy tokens up to a chosen position."""
    g = torch.Generator().manual_seed(4200)
    b, t, r, v = 64, 8, 9, 32000
    lg = torch.randn((b, r, v), generator=g).to(dtype)
    ver = oracle.argmax(np_logits(lg))
    draft = torch.from_numpy(ver[:, :t].copy())
    p = torch.randint(0, t + 1, (b,), generator=g)
    for i in range(b):
        if p[i] < t:
            draft[i, p[i]] = (draft[i, p[i]] + 1) % v
    og, on = both(lg, draft.to(torch.int32))
    assert np.array_equal(og, p.numpy())


@pytest.mark.parametrize("v", [1, 2, 5, 31, 1000, 2047, 2048, 2049, 4099, 50257])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_odd_vocab_sizes_and_no_bonus_row(v, dtype):
    g = torch.Generator().manual_seed(v)
    b, t = 5, 4
    for r in (t, t + 1):
        lg = torch.randn((b, r, v), generator=g).to(dtype)
        draft = torch.randint(0, v, (b, t), generator=g).to(torch.int32)
        ver = oracle.argmax(np_logits(lg))
        draft[0] = torch.from_numpy(ver[0, :t])           # one fully accepted sequence
        draft[1, :2] = torch.from_numpy(ver[1, :2])
        both(lg, draft)


def test_nan_inf_and_all_equal_rows():
    b, t, r, v = 3, 3, 4, 4096
    lg = torch.zeros((b, r, v))
    lg[0, 0, :] = float("nan")
    lg[0, 1, :] = float("-inf")
    lg[0, 2, 100] = float("inf")
    lg[0, 2, 7] = float("nan")
    lg[1, 0, 4000] = 1e-30
    lg[1, 1, :] = -1.0
    lg[1, 1, 4095] = -0.5
    lg[2, :, :] = float("nan")
    lg[2, 1, 2049] = -7.0
    draft = torch.tensor([[0, 0, 100], [4000, 4095, 0], [0, 2049, 0]], dtype=torch.int32)
    og, on = both(lg, draft)
    assert list(og) == [3, 3, 3]


def test_workspace_is_reusable_across_shapes():
    ws = mxq.new_workspace(max(mxq.mxq_accept_workspace_bytes(250, 17, 32000),
                               mxq.mxq_accept_workspace_bytes(1, 17, 128256)))
    for (b, v, seed) in [(250, 32000, 1), (1, 128256, 2), (250, 32000, 3), (7, 5000, 4)]:
        lg, draft, planted, p = synth.accept_trials(b, 16, 17, v, seed=4300 + seed)
        og, on = oracle.greedy_accept(lg.numpy(), draft.numpy())
        g, nxt = mxq.mxq_greedy_accept(lg.cuda(), draft.cuda(), workspace=ws)
        assert np.array_equal(g.cpu().numpy(), og) and np.array_equal(nxt.cpu().numpy(), on)
    assert not ws.view(torch.int32)[:1024].any()    # tickets are back to zero


def test_accept_tokens_variant():
    g = torch.Generator().manual_seed(9)
    b, t = 1000, 16
    for r in (t, t + 1):
        ver = torch.randint(0, 50, (b, r), generator=g).to(torch.int32)
        draft = ver[:, :t].clone()
        flip = torch.rand((b, t), generator=g) < 0.1
        draft[flip] += 1
        og, on = oracle.greedy_accept_tokens(draft.numpy(), ver.numpy())
        gg, nn = mxq.mxq_greedy_accept_tokens(draft.cuda(), ver.cuda())
        assert np.array_equal(gg.cpu().numpy(), og) and np.array_equal(nn.cpu().numpy(), on)


def test_one_workspace_across_differently_shaped_calls_through_the_c_abi():
    """The contract of mxq_accept_workspace_bytes: zero the first 4096 bytes once, then every call that completes leaves
    them zero, so one workspace serves later calls of other shapes.  Raw C calls (no helper re-zeroes anything)."""
    import ctypes

    from paper_2503_13565_b200 import binding
    L = binding.lib()
    shapes = [(40, 16, 17, 32000, torch.float32), (3, 8, 9, 128256, torch.bfloat16), (250, 4, 4, 5000, torch.float32),
              (40, 16, 17, 32000, torch.float32)]
    need = max(mxq.mxq_accept_workspace_bytes(b, r, v) for b, t, r, v, _ in shapes)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda").fill_(0xAB)   # scratch part deliberately dirty
    ws[:4096].zero_()                                                      # the one-time initialisation
    st = torch.cuda.current_stream().cuda_stream
    for i, (b, t, r, v, dtype) in enumerate(shapes):
        logits, draft, _, p = synth.accept_trials(b, t, r, v, seed=300 + i, dtype=dtype, device="cuda")
        g = torch.full((b,), -9, dtype=torch.int32, device="cuda")
        nxt = torch.full((b,), -9, dtype=torch.int32, device="cuda")
        rc = L.mxq_greedy_accept(logits.data_ptr(), 0 if dtype == torch.float32 else 1, b, r, v, draft.data_ptr(), t,
                                 g.data_ptr(), nxt.data_ptr(), ws.data_ptr(), ws.numel(), ctypes.c_void_p(st))
        assert rc == 0
        torch.cuda.synchronize()
        lg = logits.cpu()
        og, on = oracle.greedy_accept(lg.numpy() if dtype == torch.float32 else synth.bits_of(lg), draft.cpu().numpy())
        assert np.array_equal(g.cpu().numpy(), og) and np.array_equal(nxt.cpu().numpy(), on)
        assert int(ws[:4096].to(torch.int64).sum()) == 0, "the counters were not left at zero"
