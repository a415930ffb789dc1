"""The bounds-checked build of the library (compiled with -DMXQ_DEBUG_BOUNDS into libmxq_checked.so): the stand-in for a
memory checker.  In it every plain global load and store of the linear kernels tests its address against the buffer it
belongs to; an access outside is counted, recorded and redirected, never performed.

The library is chosen when the binding is first loaded (MXQ_LIBRARY=checked), so both tests run child processes:
  (1) the self-test: a store 100 bytes into a 64-byte buffer (inside a larger array of the library's own, so nothing can
      fault) is refused and reported with its offset and the buffer's size, the store next to it goes through;
  (2) the ragged, tiny and multi-tile parity tests of every linear entry point, under every kernel choice they force, run
      again on the checked library: same results (they compare with the oracle as always) and, after every single test,
      an empty report (the fixture in conftest.py).
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_checked(args, timeout):
    env = dict(os.environ, MXQ_LIBRARY="checked")
    return subprocess.run([sys.executable] + args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


SELFTEST = r"""
import torch
import paper_2503_13565_b200 as mxq
assert mxq.binding.LIB_PATH.endswith("libmxq_checked.so")
first = mxq.mxq_debug_bounds_report()
assert first["checked"] and first["refused"] == 0, first
mxq.mxq_debug_bounds_selftest()
r = mxq.mxq_debug_bounds_report()
assert r["refused"] == 1 and r["file"] == "mxq_linear.cu" and r["offset"] == 100 and r["extent"] == 64, r
assert mxq.mxq_debug_bounds_report()["refused"] == 0          # reading clears the record
# an ordinary call leaves it empty
w = torch.randint(0, 256, (203, 704), dtype=torch.uint8, device="cuda")
s = torch.randint(120, 130, (203, 44), dtype=torch.uint8, device="cuda")
x = torch.randn(3, 1408, device="cuda").to(torch.bfloat16)
y = mxq.mxq_linear(x, w, s)
torch.cuda.synchronize()
assert mxq.mxq_debug_bounds_report()["refused"] == 0 and mxq.mxq_linear_device_status() == 0
print("selftest ok")
"""


def test_an_access_outside_its_buffer_is_refused_and_reported():
    r = run_checked(["-c", SELFTEST], 600)
    assert r.returncode == 0 and "selftest ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_the_ordinary_build_says_so():
    import paper_2503_13565_b200 as mxq
    if os.environ.get("MXQ_LIBRARY") == "checked":
        pytest.skip("this process runs the checked build itself")
    assert mxq.mxq_debug_bounds_report() == {"checked": False, "refused": 0}
    with pytest.raises(mxq.MxqError):
        mxq.mxq_debug_bounds_selftest()


SELECTION = ("ragged or small or windows or token_operand or workspace or config1 or config2 or wide_range or many_tiles "
             "or in_place or composed or aligned or without_a_tcgen05 or epilogues or far_below or cannot_be_rewritten "
             "or does_not_cover or ring_depths or sixty_four or dependent_groups_in_one_call or outside_the_tensor_core or two_passes "
             "or chain or program")
FILES = ["tests/test_gpu_linear.py", "tests/test_gpu_epilogues.py", "tests/test_gpu_lm_head_accept.py", "tests/test_gpu_linear_batch.py",
         "tests/test_gpu_linear_bf16.py", "tests/test_gpu_chain.py", "tests/test_gpu_async_programs.py"]


def test_ragged_and_tiny_shapes_touch_nothing_outside_their_buffers():
    if os.environ.get("MXQ_LIBRARY") == "checked":
        pytest.skip("already inside the checked run")
    r = run_checked(["-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", "-k", SELECTION] + FILES, 3000)
    tail = r.stdout[-3000:] + r.stderr[-2000:]
    assert r.returncode == 0, tail
    assert " passed" in r.stdout and "no tests ran" not in r.stdout, tail
