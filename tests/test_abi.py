"""The C-ABI library loads without a GPU, exports everything include/mxq.h declares, and
rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

import paper_2503_13565_b200 as mxq
from paper_2503_13565_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(mxq_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_expected_calls():
    names = declared_symbols()
    for must in ("mxq_quantize", "mxq_linear", "mxq_greedy_accept", "mxq_dequantize", "mxq_linear_host"):
        assert must in names


@pytest.mark.parametrize("name", declared_symbols())
def test_every_declared_symbol_is_exported(name):
    assert hasattr(binding.lib(), name), name


def test_version_and_status_strings():
    assert mxq.mxq_version() == 100
    texts = {mxq.status_string(s) for s in range(7)}
    assert len(texts) == 7 and "ok" in texts
    assert mxq.status_string(99) == "unknown status"


def test_size_functions():
    assert mxq.mxq_codes_bytes(4096, 4096) == 4096 * 4096 // 2
    assert mxq.mxq_scales_bytes(4096, 4096) == 4096 * 4096 // 32
    assert (mxq.mxq_codes_bytes(4096, 11008) + mxq.mxq_scales_bytes(4096, 11008)) * 8 == 4096 * 11008 * 4.25
    assert mxq.mxq_codes_bytes(4096, 100) == 0 and mxq.mxq_scales_bytes(0, 64) == 0
    assert mxq.mxq_linear_workspace_bytes(17, 64, 64) == 0
    assert mxq.mxq_accept_workspace_bytes(1, 17, 128256) > 0
    assert mxq.mxq_accept_workspace_bytes(250, 17, 32000) >= 250 * 4 + 250 * 17 * 8


def test_argument_errors_are_caught_before_any_launch():
    L = binding.lib()
    a = 0x1000  # fake, aligned, never dereferenced: every call below must fail validation first
    assert L.mxq_quantize(None, 8, 64, a, a, None, None) == 1
    assert L.mxq_quantize(a, 8, 48, a, a, None, None) == 2
    assert L.mxq_quantize(a, 0, 64, a, a, None, None) == 2
    assert L.mxq_quantize(a + 2, 8, 64, a, a, None, None) == 3
    assert L.mxq_dequantize(a, None, 8, 64, a, None) == 1
    assert L.mxq_dequantize(a, a, 8, 31, a, None) == 2
    assert L.mxq_linear(a, 0, a, a, 8, 64, a, 0, None, 0, None) == 2
    assert L.mxq_linear(a, 17, a, a, 8, 64, a, 0, None, 0, None) == 2
    assert L.mxq_linear(a, 1, a, a, 8, 65, a, 0, None, 0, None) == 2
    assert L.mxq_linear(a, 1, a, a, 8, 64, a, 7, None, 0, None) == 4
    assert L.mxq_linear(a, 1, a + 8, a, 8, 64, a, 0, None, 0, None) == 3
    assert L.mxq_linear(None, 1, a, a, 8, 64, a, 0, None, 0, None) == 1
    assert L.mxq_linear_host(None, 1, a, a, 8, 64, a, 0, a, a, None, 0, None) == 1
    assert L.mxq_greedy_accept(a, 0, 1, 5, 100, a, 4, a, a, None, 0, None) == 5
    assert L.mxq_greedy_accept(a, 0, 1, 7, 100, a, 4, a, a, a, 1 << 20, None) == 2   # R not T or T+1
    assert L.mxq_greedy_accept(a, 0, 1, 66, 100, a, 65, a, a, a, 1 << 20, None) == 2  # T > 64
    assert L.mxq_greedy_accept(a, 3, 1, 5, 100, a, 4, a, a, a, 1 << 20, None) == 4
    assert L.mxq_greedy_accept_tokens(a, a, 1, 4, 6, a, a, None) == 2
    assert L.mxq_greedy_accept_tokens(None, a, 1, 4, 5, a, a, None) == 1
    # fused vocabulary projection + verification: R must be T or T + 1 and at most 16; a workspace is mandatory
    assert L.mxq_lm_head_accept(a, 3, a, a, 1024, 128, a, 1, None, a, a, a, 1 << 20, None) == 2
    assert L.mxq_lm_head_accept(a, 17, a, a, 1024, 128, a, 16, None, a, a, a, 1 << 20, None) == 2
    assert L.mxq_lm_head_accept(a, 2, a, a, 1024, 128, a, 1, None, a, a, None, 0, None) == 1
    assert L.mxq_lm_head_accept(a, 2, a, a, 1024, 128, a, 1, None, a, a, a, 16, None) == 5


def test_batch_argument_errors_are_caught_before_any_launch():
    L = binding.lib()
    a = 0x1000
    descs = (binding._LinearDesc * 2)()
    for d in descs:
        d.X_bf16, d.codes, d.scales, d.Y, d.residual = a, a, a, a, None
        d.N, d.K, d.y_dtype, d.epilogue = 256, 256, 0, 0
    p = ctypes.cast(descs, ctypes.c_void_p)
    assert L.mxq_linear_batch(None, 1, 1, a, 1 << 30, None) == 1
    assert L.mxq_linear_batch(p, 0, 1, a, 1 << 30, None) == 2
    assert L.mxq_linear_batch(p, 65, 1, a, 1 << 30, None) == 2
    assert L.mxq_linear_batch(p, 2, 17, a, 1 << 30, None) == 2
    assert L.mxq_linear_batch(p, 2, 1, None, 0, None) == 1
    assert L.mxq_linear_batch(p, 2, 1, a + 16, 1 << 30, None) == 3     # workspace not 256-byte aligned
    assert L.mxq_linear_batch(p, 2, 1, a, 64, None) == 5
    assert L.mxq_linear_batch_workspace_bytes(p, 2, 1) >= 16384
    descs[1].epilogue = 1                                              # residual epilogue without a residual
    assert L.mxq_linear_batch(p, 2, 1, a, 1 << 30, None) == 1
    descs[1].epilogue = 2
    descs[1].N = 255                                                   # gate / up pairing needs an even N
    assert L.mxq_linear_batch(p, 2, 1, a, 1 << 30, None) == 2
    descs[1].epilogue, descs[1].N, descs[1].K = 0, 256, 100
    assert L.mxq_linear_batch(p, 2, 1, a, 1 << 30, None) == 2
    descs[1].K, descs[1].y_dtype = 256, 9
    assert L.mxq_linear_batch(p, 2, 1, a, 1 << 30, None) == 4
    descs[1].y_dtype, descs[1].codes = 0, a + 4
    assert L.mxq_linear_batch(p, 2, 1, a, 1 << 30, None) == 3
    assert L.mxq_linear_batch_workspace_bytes(p, 2, 1) == 0
    assert L.mxq_set_linear_layout(99, 1) == 2 and L.mxq_set_linear_layout(5, 0) == 0


def test_linear_host_checks_every_argument_before_staging():
    """A bad codes / scales / Y pointer must be refused before the staging copy of X is enqueued (a fake X pointer
    would otherwise be handed to the copy engine)."""
    L = binding.lib()
    a = 0x1000
    assert L.mxq_linear_host(a, 1, None, a, 8, 64, a, 0, a, a, None, 0, None) == 1
    assert L.mxq_linear_host(a, 1, a, None, 8, 64, a, 0, a, a, None, 0, None) == 1
    assert L.mxq_linear_host(a, 1, a + 4, a, 8, 64, a, 0, a, a, None, 0, None) == 3
    assert L.mxq_linear_host(a, 1, a, a + 4, 8, 64, a, 0, a, a, None, 0, None) == 3
    assert L.mxq_linear_host(a, 1, a, a, 8, 64, a, 0, a + 4, a, None, 0, None) == 3
    assert L.mxq_linear_host(a, 1, a, a, 8, 64, a, 0, a, a + 4, None, 0, None) == 3


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError, match="no CPU fallback"):
        binding.lib()


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2503_13565_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text and "oracle/" not in text, fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c", ".h")):
            text = open(os.path.join(ROOT, "oracle", fn)).read()
            assert "paper_2503_13565_b200" not in text and "mxq.h" not in text, fn
