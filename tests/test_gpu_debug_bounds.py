"""Parity cases run once more on the library's debug build, in which every index a kernel takes from the step's inputs
(token ids, positions, page ids of the append and of the attention loads, leaf counts, tree parents, unit tables) is
compared with its range on the device before it is used.  A failed check makes the step return TS_ERR_DEVICE_BOUNDS,
which the binding raises: the cases pass only if no check fires and the results still match the oracle.  (The memory
checker tools are not available on every machine; this is the stand-in.)  The debug library is loaded in a child
process: a process holds one copy of the library."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r}); sys.path.insert(0, {tests!r})
from paper_2604_13519_b200 import build, binding
build.build(debug_bounds=True)
binding.use_debug_library()
import test_gpu_parity as P, test_gpu_tree as T
P.test_c1_decode_loop_parity(1)
P.test_synthetic_kv_single("8b-2l", 700, 64, 1)
P.test_ragged_batch()
P.test_row_counts_around_the_projection_kernels_switch("8b-2l", [33, 64, 64, 64, 64, 11])
P.test_row_counts_around_the_projection_kernels_switch("1b-2l", [40, 33, 30])
for name in dir(T):
    if name.startswith("test_") and getattr(T, name).__code__.co_argcount == 0:
        getattr(T, name)()
assert binding.LIB_PATH.endswith("libtoolspec_dbg.so")
print("debug-bounds cases ok")
"""


def test_parity_cases_on_the_debug_build():
    code = CHILD.format(root=ROOT, tests=os.path.join(ROOT, "tests"))
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "debug-bounds cases ok" in r.stdout
