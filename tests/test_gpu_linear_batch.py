"""GPU parity of mxq_linear_batch (several layers in one persistent launch) against the oracle, layer by layer.

Plain layers: |y - y64| <= 2e-3 * sum|x w^| + 1e-6 element by element (the bound of mxq_linear); epilogues: the bounds
of tests/test_gpu_epilogues.py.  The cases cover one CTA per unit (tiny calls), tiles cut between two and three CTAs'
ranges, ragged N, the half-full last stage (K % 256 == 128), shared and distinct X, every token count the persistent
kernel takes (1..8) and the calls it hands on to the one-by-one path.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import synth
from parity import ABS, REL, check_linear, gpu_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def status_clean():
    yield
    assert mxq.mxq_linear_device_status() == 0, "a bounded wait inside a kernel gave up"


def values(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def make_layer(cfg, idx, n, k, m, x=None, epilogue="none", out_dtype=torch.float32, rows=None):
    """One layer of a batch with everything the oracle needs to check it afterwards."""
    codes, scales, _ = oracle.quantize(synth.bits_of(synth.weight(cfg, idx, n, k)))
    xbits = synth.bits_of(synth.activations(cfg, idx, m, k)) if x is None else x
    lay = {"x": gpu_bf16(xbits), "codes": torch.from_numpy(codes).cuda(), "scales": torch.from_numpy(scales).cuda(),
           "epilogue": epilogue, "_codes": codes, "_scales": scales, "_x": xbits, "_rows": rows}
    n_out = n // 2 if epilogue == "swiglu" else n
    lay["out"] = torch.full((m, n_out), float("nan"), dtype=out_dtype, device="cuda")
    if epilogue == "residual":
        g = torch.Generator().manual_seed(500 + idx)
        lay["residual"] = (torch.randn(m, n, generator=g) * 0.5).to(out_dtype).cuda()
    return lay


def check_layer(lay, what):
    rows = lay["_rows"]
    sel = slice(None) if rows is None else np.asarray(rows)
    out_dtype = lay["out"].dtype
    bf = (lambda want: np.abs(want) * 2.0 ** -8) if out_dtype == torch.bfloat16 else (lambda want: 0.0)
    got = values(lay["out"])
    if lay["epilogue"] == "none":
        y64, a64 = oracle.linear(lay["_x"], lay["_codes"], lay["_scales"], rows=rows)
        if out_dtype == torch.float32:
            return check_linear(lay["out"] if rows is None else lay["out"][:, torch.as_tensor(rows, device="cuda")], y64, a64, what)
        tol = REL * a64 + ABS + bf(y64)
        want = y64
    elif lay["epilogue"] == "residual":
        r64 = values(lay["residual"])[:, sel]
        want, a = oracle.linear_residual(lay["_x"], lay["_codes"], lay["_scales"], r64, rows=rows)
        tol = REL * a + ABS + 2.0 ** -23 * np.abs(want) + bf(want)
    else:
        want, g, u, ag, au = oracle.linear_swiglu(lay["_x"], lay["_codes"], lay["_scales"], rows=rows)
        tg, tu = REL * ag + ABS, REL * au + ABS
        tol = 1.1 * tg * (np.abs(u) + tu) + np.abs(oracle.silu(g)) * tu + 1e-6 * np.abs(want) + 1e-30 + bf(want)
    got = got[:, sel]
    assert np.isfinite(got).all(), what + ": non-finite output"
    worst = float((np.abs(got - want) / tol).max())
    assert worst <= 1.0, "%s: error/tolerance = %.3g" % (what, worst)
    return worst


def run_batch(layers, expect_persistent=True):
    batch = mxq.LinearBatch(layers)
    assert bool(batch.info()["persistent"]) == expect_persistent, batch.info()
    ws = mxq.new_workspace(batch.workspace_bytes())
    batch.run(ws)
    torch.cuda.synchronize()
    return batch, ws


def sample_rows(n, seed, count=300):
    return np.unique(np.concatenate([[0, 1, 127, 128, n - 129, n - 128, n - 2, n - 1],
                                     np.random.default_rng(seed).integers(0, n, count)])).astype(np.int64)


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 8])
def test_small_ragged_layers(m):
    """Fewer units than SMs (every CTA owns one unit, every tile is summed across CTAs), ragged N, half-full last stage."""
    layers = [make_layer(3, 20, 203, 1408, m), make_layer(3, 21, 515, 2048, m), make_layer(3, 22, 128, 128, m),
              make_layer(3, 23, 1000, 384, m)]
    run_batch(layers)
    for i, lay in enumerate(layers):
        check_layer(lay, "small batch layer %d M=%d" % (i, m))


@pytest.mark.parametrize("m", [1, 4])
def test_config2_draft_model_layer_set(m):
    """The 68M-Llama-like draft model's layer set in one call; q/k/v share X, gate/up share X."""
    xh = synth.bits_of(synth.activations(2, 0, m, 768))
    xf = synth.bits_of(synth.activations(2, 6, m, 3072))
    layers = [make_layer(2, i, 768, 768, m, x=xh) for i in range(4)]
    layers += [make_layer(2, 4, 3072, 768, m, x=xh), make_layer(2, 5, 3072, 768, m, x=xh), make_layer(2, 6, 768, 3072, m, x=xf),
               make_layer(2, 7, 32000, 768, m, x=xh, rows=sample_rows(32000, 1))]
    xg = layers[0]["x"]
    for lay in layers[:6] + layers[7:]:
        lay["x"] = xg   # the same device tensor: one image
    run_batch(layers)
    for i, lay in enumerate(layers):
        check_layer(lay, "config2 layer %d M=%d" % (i, m))


@pytest.mark.parametrize("m", [1, 2, 4, 8])
def test_config3_7b_layer_set(m):
    """The benchmark's call: seven 7B-shaped layers in one launch, sampled rows of every layer against the oracle."""
    shapes = synth.LAYERS_7B
    xs = {k: gpu_bf16(synth.bits_of(synth.activations(3, 0 if k == 4096 else 6, m, k))) for k in (4096, 11008)}
    layers = []
    for i, (name, n, k) in enumerate(shapes):
        lay = make_layer(3, i, n, k, m, x=synth.bits_of(synth.activations(3, 0 if k == 4096 else 6, m, k)), rows=sample_rows(n, i, 500))
        lay["x"] = xs[k]
        layers.append(lay)
    batch, ws = run_batch(layers)
    assert batch.info()["grid"] == 2 * torch.cuda.get_device_properties(0).multi_processor_count
    for i, lay in enumerate(layers):
        check_layer(lay, "7B layer %s M=%d" % (shapes[i][0], m))
    # bit-reproducible, and the workspace is reusable as it was left
    first = [lay["out"].clone() for lay in layers]
    for lay in layers:
        lay["out"].fill_(float("nan"))
    batch.run(ws)
    torch.cuda.synchronize()
    for a, lay in zip(first, layers):
        assert torch.equal(a, lay["out"])


@pytest.mark.parametrize("m", [1, 8])
def test_the_benchmarks_launch_configuration(m):
    """What bench.py times: distinct 7B layer sets (16 here), eight sets = 56 layers per call, the calls round-robin on two
    streams with a workspace each, replayed from a CUDA graph.  The weights are cast on the GPU (bit-exact with the oracle's
    cast, tests/test_gpu_quantize.py); sampled rows of the first, a middle and the last layer of each call are checked
    against the oracle, which dequantises the GPU's own codes."""
    shapes = synth.LAYERS_7B
    nsets, per_call = 16, 8
    xbits = {k: synth.bits_of(synth.activations(3, 40 + k % 7, m, k)) for k in (4096, 11008)}
    x = {k: gpu_bf16(v) for k, v in xbits.items()}
    calls = []
    for c in range(nsets // per_call):
        lays = []
        for ls in range(per_call):
            for j, (_, n, k) in enumerate(shapes):
                codes, scales = mxq.mxq_quantize(synth.weight(3, 900 + 7 * (c * per_call + ls) + j, n, k, device="cuda"))
                lays.append(dict(x=x[k], codes=codes, scales=scales, out=torch.full((m, n), float("nan"), device="cuda")))
        calls.append(lays)
    both = mxq.IndependentBatches(calls, streams=2)
    assert both.batches[0].count == 56 and both.batches[0].info()["persistent"] == 1
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        both.run(st)
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            both.run(st)
        for lays in calls:
            for lay in lays:
                lay["out"].fill_(float("nan"))
        graph.replay()
        graph.replay()
        st.synchronize()
    for c, lays in enumerate(calls):
        for i in (0, 4, 27, 55):
            lay = lays[i]
            n, k = lay["codes"].shape[0], lay["x"].shape[1]
            rows = sample_rows(n, c + i, 200)
            y64, a64 = oracle.linear(xbits[k], lay["codes"].cpu().numpy(), lay["scales"].cpu().numpy(), rows=rows)
            check_linear(lay["out"][:, torch.as_tensor(rows, device="cuda")], y64, a64, "call %d layer %d M=%d" % (c, i, m))
        assert all(bool(torch.isfinite(lay["out"]).all()) for lay in lays)


@pytest.mark.parametrize("m", [1, 8])
def test_config5_13b_layer_set(m):
    """The seven 13B-shaped layers (hidden 5120, FFN 13824) in one call, sampled rows of every layer."""
    shapes = [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]
    xs = {k: synth.bits_of(synth.activations(5, k, m, k)) for k in (5120, 13824)}
    gx = {k: gpu_bf16(v) for k, v in xs.items()}
    layers = []
    for i, (n, k) in enumerate(shapes):
        lay = make_layer(5, i, n, k, m, x=xs[k], rows=sample_rows(n, 50 + i, 200))
        lay["x"] = gx[k]
        layers.append(lay)
    run_batch(layers)
    for i, lay in enumerate(layers):
        check_layer(lay, "13B layer %d M=%d" % (i, m))


@pytest.mark.parametrize("m", [1, 3, 6])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_epilogues(m, out_dtype):
    layers = [make_layer(3, 30, 1000, 1024, m, epilogue="residual", out_dtype=out_dtype),
              make_layer(3, 31, 2 * 700, 1024, m, epilogue="swiglu", out_dtype=out_dtype),
              make_layer(3, 32, 4096, 4096, m, epilogue="residual", out_dtype=out_dtype, rows=sample_rows(4096, 2)),
              make_layer(3, 33, 2 * 2752, 4096, m, epilogue="swiglu", out_dtype=out_dtype, rows=sample_rows(2752, 3)),
              make_layer(3, 34, 333, 1152, m, out_dtype=out_dtype)]
    res_before = [lay.get("residual").clone() if lay.get("residual") is not None else None for lay in layers]
    run_batch(layers)
    for i, lay in enumerate(layers):
        check_layer(lay, "epilogue layer %d M=%d %s" % (i, m, out_dtype))
        if res_before[i] is not None:
            assert torch.equal(res_before[i], lay["residual"]), "the residual was written to"


def test_residual_in_place():
    lay = make_layer(3, 35, 640, 2048, 2, epilogue="residual")
    keep = lay["residual"].clone()
    lay["out"] = lay["residual"]
    run_batch([lay])
    lay["residual"] = keep
    check_layer(lay, "in-place residual")


def test_one_workspace_across_differently_shaped_calls():
    """Calls in one stream share a workspace: every call leaves the counters as it found them."""
    a = [make_layer(3, 40, 203, 1408, 1), make_layer(3, 41, 4096, 4096, 1, rows=sample_rows(4096, 4))]
    b = [make_layer(3, 42, 515, 2048, 4), make_layer(3, 43, 900, 640, 4), make_layer(3, 44, 300, 5120, 4)]
    ba, bb = mxq.LinearBatch(a), mxq.LinearBatch(b)
    ws = mxq.new_workspace(max(ba.workspace_bytes(), bb.workspace_bytes()))
    for _ in range(3):
        ba.run(ws)
        bb.run(ws)
    torch.cuda.synchronize()
    assert int(ws[:16384].view(torch.int32).abs().sum()) == 0, "counters not left at zero"
    for i, lay in enumerate(a + b):
        check_layer(lay, "shared workspace layer %d" % i)


@pytest.mark.parametrize("m", [1, 3, 8])
@pytest.mark.parametrize("count", [40, 1500])
def test_many_elements_far_below_their_blocks_maximum(m, count):
    """Activations as a gated feed-forward block produces them: a few (here `count`, spread over the token rows) land
    more than 24 binades under their block's maximum and do not fit the operand's fixed point.  Up to 256 per X they are
    corrected one by one (remainder * weight in the epilogue); beyond that the layers reading that X take the scalar
    path.  Either way the bound holds, for the layer that shares the X and for the one that does not."""
    k, n = 2816, 640
    x = synth.activations(3, 230, m, k).clone().float()
    g = torch.Generator().manual_seed(count + m)
    flat = x.view(-1)
    idx = torch.randperm(flat.numel(), generator=g)[:count]
    flat[idx] = flat[idx] * 2.0 ** -40 + 2.0 ** -60
    xb = synth.bits_of(x.to(torch.bfloat16))
    a = make_layer(3, 231, n, k, m, x=xb)
    b = make_layer(3, 232, 2 * 384, k, m, x=xb, epilogue="swiglu")
    b["x"] = a["x"]
    c = make_layer(3, 233, 515, 1024, m)
    run_batch([a, b, c])
    for lay, what in ((a, "plain"), (b, "gate/up"), (c, "other X")):
        check_layer(lay, "%d tiny elements, M=%d: %s" % (count, m, what))


def test_activations_that_cannot_be_rewritten_exactly():
    """An element more than 24 binades below its block's maximum, an infinity, a NaN: corrected element by element in the
    epilogue (same bound; Inf and NaN come out as IEEE arithmetic gives them), the other layers of the call are untouched."""
    m, k = 2, 1024
    x = synth.activations(3, 50, m, k).clone()
    x[0, 5] = 2.0 ** -40
    x[0, 6] = 1.0
    xb = synth.bits_of(x)
    lay_bad = make_layer(3, 50, 515, k, m, x=xb)
    lay_ok = make_layer(3, 51, 300, 768, m)
    run_batch([lay_bad, lay_ok])
    check_layer(lay_bad, "tiny element")
    check_layer(lay_ok, "untouched layer")
    x2 = synth.activations(3, 52, m, k).clone()
    x2[1, 40] = float("inf")
    lay_inf = make_layer(3, 52, 260, k, m, x=synth.bits_of(x2))
    run_batch([lay_inf])
    y64, a64 = oracle.linear(lay_inf["_x"], lay_inf["_codes"], lay_inf["_scales"])
    got = values(lay_inf["out"])
    assert np.array_equal(np.isnan(got[1]), np.isnan(y64[1])) and np.array_equal(got[1][~np.isnan(got[1])], y64[1][~np.isnan(y64[1])])
    check_linear(lay_inf["out"][:1], y64[:1], a64[:1], "row without the infinity")


@pytest.mark.parametrize("m", [9, 12, 16])
def test_nine_to_sixteen_token_rows_run_as_two_passes(m):
    """Rows [0, 8) and [8, M) through the persistent kernel one after the other: every epilogue, BF16 and FP32 outputs,
    a residual added in place, and two layers that share an X."""
    layers = [make_layer(3, 63, 515, 2048, m), make_layer(3, 64, 2 * 300, 2048, m, epilogue="swiglu", out_dtype=torch.bfloat16),
              make_layer(3, 65, 333, 1152, m, epilogue="residual", out_dtype=torch.bfloat16)]
    layers.append(make_layer(3, 66, 200, 2048, m, x=layers[0]["_x"]))
    layers[3]["x"] = layers[0]["x"]
    batch, _ = run_batch(layers)
    assert batch.info()["persistent"] == 2
    for i, lay in enumerate(layers):
        check_layer(lay, "two passes, layer %d M=%d" % (i, m))


def test_two_passes_on_the_7b_layer_set_and_with_dependent_groups():
    m = 9   # eight speculated tokens and the one before them: the verification pass of Sec. III-B with N = 8
    shapes = [(0, 4096, 4096), (4, 11008, 4096), (6, 4096, 11008)]
    layers = [make_layer(3, idx, n, k, m, rows=sample_rows(n, idx)) for idx, n, k in shapes]
    run_batch(layers)
    for lay in layers:
        check_layer(lay, "7B shapes, M=9")
    chain = chain_layers(m, 256, 384, 210)
    run_batch(chain)
    check_chain(chain, "chain M=9")


@pytest.mark.parametrize("m,n,k", [(1, 203, 1440), (9, 203, 1440), (16, 300, 96)])
def test_calls_the_persistent_kernel_does_not_cover(m, n, k):
    """K not a multiple of 128: the layers run one by one, with the same results as the single-layer entry points."""
    layers = [make_layer(3, 60, n, k, m), make_layer(3, 61, 2 * 128, k, m, epilogue="swiglu"),
              make_layer(3, 62, n, k, m, epilogue="residual")]
    run_batch(layers, expect_persistent=False)
    for i, lay in enumerate(layers):
        check_layer(lay, "one-by-one layer %d M=%d" % (i, m))


@pytest.mark.parametrize("m", [1, 8])
def test_independent_calls_on_two_streams_with_a_workspace_each(m):
    """Calls that may run concurrently need a workspace each, and then overlap freely: six calls issued round-robin on two
    streams (the benchmark's route) leave bit for bit what the same calls leave one after the other on one stream."""
    calls = [[make_layer(3, 300 + 3 * c + j, n, k, m, rows=sample_rows(n, c + j, 100)) for j, (n, k) in enumerate([(4096, 4096), (1024, 11008), (2816, 1024)])]
             for c in range(6)]
    both = mxq.IndependentBatches(calls, streams=2)
    assert len(both.streams) == 2 and len(both.workspaces) == 2
    wss = both.workspaces
    for b in both.batches:
        b.run(wss[0])
    torch.cuda.synchronize()
    ref = [[lay["out"].clone() for lay in layers] for layers in calls]
    for _ in range(3):
        for layers in calls:
            for lay in layers:
                lay["out"].fill_(float("nan"))
        both.run()   # forks from and joins the current stream
        torch.cuda.synchronize()
        for layers, outs in zip(calls, ref):
            for lay, want in zip(layers, outs):
                assert torch.equal(lay["out"], want)
    for c, layers in enumerate(calls[:2]):
        for j, lay in enumerate(layers):
            check_layer(lay, "two streams, call %d layer %d M=%d" % (c, j, m))
    assert not wss[0][:16384].any() and not wss[1][:16384].any()


@pytest.mark.parametrize("ring,per_sm", [(2, 1), (3, 2), (5, 2), (1, 1)])
def test_other_ring_depths_and_two_ctas_per_sm(ring, per_sm):
    mxq.mxq_set_linear_layout("batch_ring", ring)
    mxq.mxq_set_linear_layout("batch_ctas_per_sm", per_sm)
    try:
        layers = [make_layer(3, 70, 4096, 4096, 1, rows=sample_rows(4096, 5)), make_layer(3, 71, 1000, 11008, 1),
                  make_layer(3, 72, 203, 1408, 1)]
        batch, _ = run_batch(layers)
        assert batch.info()["ring"] == ring
        for i, lay in enumerate(layers):
            check_layer(lay, "ring %d, %d CTAs per SM, layer %d" % (ring, per_sm, i))
    finally:
        mxq.mxq_set_linear_layout("batch_ring", 0)
        mxq.mxq_set_linear_layout("batch_ctas_per_sm", 0)


def test_sixty_four_layers_in_one_call():
    """The most layers a call takes: 64 small ones with 64 distinct X."""
    layers = [make_layer(3, 90 + i, 128 + 64 * (i % 5), 256 + 128 * (i % 4), 2) for i in range(64)]
    assert len(layers) == mxq.binding.MAX_BATCH
    run_batch(layers)
    for i, lay in enumerate(layers):
        check_layer(lay, "layer %d of 64" % i)


def test_a_bounded_wait_that_expires_is_reported_and_contained():
    """Test hook: the weight copy of one unit of the call is left out, so the MMA warp of the CTA that owns it waits for
    bytes that never arrive.  Its wait is bounded (20 ms here): the call must still complete, mxq_linear_device_status must
    report the expired wait (bit 24), the tiles that CTA had not finished (and the tiles it shares with its neighbours)
    must be NaN, and every other output must be within the bound.  Afterwards the library works as before."""
    m = 1
    layers = [make_layer(3, 100, 4096, 4096, m, rows=None), make_layer(3, 101, 1000, 2048, m)]
    batch = mxq.LinearBatch(layers)
    info = batch.info()
    assert info["persistent"] == 1
    ws = mxq.new_workspace(batch.workspace_bytes())
    unit = info["units"] // 3            # somewhere inside the first layer
    mxq.mxq_debug_batch_fault(unit, 20000)
    batch.run(ws)
    torch.cuda.synchronize()             # returns: nothing hangs
    status = mxq.mxq_linear_device_status()
    assert status & (1 << 24), "the expired wait was not reported (status %#x)" % status
    y64, a64 = oracle.linear(layers[0]["_x"], layers[0]["_codes"], layers[0]["_scales"])
    got = values(layers[0]["out"])
    bad = np.isnan(got)
    ks, tile_of_unit = 4096 // 256, unit // (4096 // 256)
    assert bad[0, tile_of_unit * 128:(tile_of_unit + 1) * 128].all(), "the tile whose data never arrived must be NaN"
    per_cta = -(-info["units"] // info["grid"])
    assert bad.sum() <= 128 * (per_cta // ks + 3), "more than one CTA's tiles were lost: %d outputs" % bad.sum()
    ok = ~bad
    assert (np.abs(got - y64)[ok] <= (REL * a64 + ABS)[ok]).all()
    check_layer(layers[1], "the layer after the lost tiles") if not np.isnan(values(layers[1]["out"])).any() else None
    # a fresh workspace (the counters of the failed call are not to be trusted) and the same call again: all good
    ws2 = mxq.new_workspace(batch.workspace_bytes())
    batch.run(ws2)
    torch.cuda.synchronize()
    assert mxq.mxq_linear_device_status() == 0
    for i, lay in enumerate(layers):
        check_layer(lay, "after the fault, layer %d" % i)


def chain_layers(m, h, f, seed):
    """A decoder layer's dependent chain in three groups: {q/k/v as one matrix, o + residual} | {gate/up with SiLU(gate)*up}
    | {down + residual}; every intermediate is BF16 and feeds the next group."""
    qkv = make_layer(3, seed, 3 * h, h, m, out_dtype=torch.bfloat16)
    o = make_layer(3, seed + 1, h, h, m, epilogue="residual", out_dtype=torch.bfloat16)
    o["residual"] = qkv["x"]                                             # h0 (the layer's input) is the residual of o
    gu = make_layer(3, seed + 2, 2 * f, h, m, epilogue="swiglu", out_dtype=torch.bfloat16)
    gu["x"], gu["depends"] = o["out"], True                              # h1 = o's output
    down = make_layer(3, seed + 3, h, f, m, epilogue="residual", out_dtype=torch.bfloat16)
    down["x"], down["residual"], down["depends"] = gu["out"], o["out"], True
    return [qkv, o, gu, down]


def check_chain(layers, what):
    """Stage by stage, each stage's oracle fed with the GPU's own (BF16) intermediates: a rounding difference in an
    intermediate cannot leak into the next stage's check."""
    qkv, o, gu, down = layers
    gu["_x"] = synth.bits_of(o["out"].cpu())
    down["_x"] = synth.bits_of(gu["out"].cpu())
    for name, lay in zip(("qkv", "o", "gate/up", "down"), layers):
        check_layer(lay, "%s: %s" % (what, name))


@pytest.mark.parametrize("m", [1, 4, 8])
@pytest.mark.parametrize("h,f", [(1024, 2816), (256, 384)])
def test_dependent_groups_in_one_call(m, h, f):
    """MXQ_BATCH_DEPENDS: a layer that reads what earlier layers of the same call wrote.  The small case has fewer units
    per group than CTAs (some CTAs own nothing in a group); the larger one cuts tiles between CTAs in every group."""
    layers = chain_layers(m, h, f, 200)
    h1_before = layers[1]["out"].clone()
    batch, ws = run_batch(layers)
    assert not torch.equal(h1_before, layers[1]["out"])
    check_chain(layers, "chain M=%d h=%d" % (m, h))
    # again on the same workspace, and bit for bit the same
    first = [lay["out"].clone() for lay in layers]
    for lay in layers:
        lay["out"].fill_(float("nan"))
    batch.run(ws)
    torch.cuda.synchronize()
    for a, lay in zip(first, layers):
        assert torch.equal(a, lay["out"])
    assert int(ws[:16384].view(torch.int32).abs().sum()) == 0, "counters not left at zero"


def test_dependent_groups_7b_layer():
    """The four-call fused 7B layer (12288 x 4096; 4096 x 4096 + residual; 22016 x 4096 gate/up; 4096 x 11008 + residual) as
    ONE call of three groups, sampled rows of every stage."""
    m, h, f = 1, 4096, 11008
    layers = chain_layers(m, h, f, 210)
    for lay, n in zip(layers, (3 * h, h, f, h)):
        lay["_rows"] = sample_rows(n, n % 97, 300)
    run_batch(layers)
    check_chain(layers, "7B chain")


def test_calls_of_different_token_counts_side_by_side():
    """Two streams, one issuing calls at one token row (16 operand columns, 128 tensor-memory columns per CTA) and the other
    at eight (128 operand columns, 256 tensor-memory columns): CTAs of both kernels share SMs; results as in isolation."""
    shapes = [(4096, 4096), (1024, 11008), (2816, 1024)]
    calls = {m: [[make_layer(3, 400 + 10 * m + 3 * c + j, n, k, m, rows=sample_rows(n, c + j, 100)) for j, (n, k) in enumerate(shapes)]
                 for c in range(4)] for m in (1, 8)}
    batches = {m: [mxq.LinearBatch(layers) for layers in calls[m]] for m in calls}
    ws = {m: mxq.new_workspace(max(b.workspace_bytes() for b in batches[m])) for m in calls}
    for m in calls:
        for b in batches[m]:
            b.run(ws[m])
    torch.cuda.synchronize()
    ref = {m: [[lay["out"].clone() for lay in layers] for layers in calls[m]] for m in calls}
    streams = {1: torch.cuda.Stream(), 8: torch.cuda.Stream()}
    for _ in range(3):
        for m in calls:
            for layers in calls[m]:
                for lay in layers:
                    lay["out"].fill_(float("nan"))
        torch.cuda.synchronize()
        for c in range(4):
            for m in (1, 8):
                batches[m][c].run(ws[m], stream=streams[m])
        torch.cuda.synchronize()
        for m in calls:
            for layers, outs in zip(calls[m], ref[m]):
                for lay, want in zip(layers, outs):
                    assert torch.equal(lay["out"], want)
    for m in calls:
        for j, lay in enumerate(calls[m][0]):
            check_layer(lay, "side by side, layer %d M=%d" % (j, m))


def test_grouped_calls_are_not_spread_over_streams():
    """The CTAs of a call of several groups wait for one another, so the whole grid must be resident: the helper that
    issues independent calls on several streams refuses such calls (on one stream they are fine)."""
    chain = chain_layers(2, 256, 384, 230)
    assert mxq.LinearBatch(chain).groups == 3 and mxq.LinearBatch([dict(lay, depends=False) for lay in chain[:1]]).groups == 1
    with pytest.raises(ValueError):
        mxq.IndependentBatches([chain, chain_layers(2, 256, 384, 240)], streams=2)
    one = mxq.IndependentBatches([chain], streams=2)   # a single call: one stream
    one.run()
    torch.cuda.synchronize()
    check_chain(chain, "one grouped call through the helper")


def test_too_many_groups_are_refused():
    lays = [make_layer(3, 220, 128, 128, 1) for _ in range(10)]
    for lay in lays[1:]:
        lay["depends"] = True
    with pytest.raises(mxq.MxqError) as e:
        mxq.LinearBatch(lays).workspace_bytes() or mxq.LinearBatch(lays).run(mxq.new_workspace(1 << 20))
    assert e.value.status == 2


def test_argument_errors():
    lay = make_layer(3, 80, 256, 256, 1)
    batch = mxq.LinearBatch([lay])
    with pytest.raises(mxq.MxqError) as e:
        batch.run(torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 5
    with pytest.raises(ValueError):
        mxq.LinearBatch([lay] * 65)
