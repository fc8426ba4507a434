"""The -DSPECV_DEBUG build of the library: every row index, split number, segment number and token
id the streaming kernels compute is range-checked before use.  A batch of awkward shapes runs
through it in a child process; the answers must match the oracle as usual and no check may have
fired."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

CHILD = r"""
import sys
sys.path.insert(0, "tests")
import numpy as np
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W
from gpu_utils import DeviceBatch, assert_parity
assert binding.LIB_PATH.endswith("libspecverify_debug.so")
binding.set_path(binding.PATH_STREAMING)
assert binding.debug_violation() == 0
for cfg, B, V in ((1, 3, 4099), (5, 40, 1500), (2, 8, 32000), (5, 24, 31), (5, 300, 257)):
    w = W.make_config(cfg, B=B, V=V)
    assert_parity(w, DeviceBatch(w, ld_pad=3, elem_offset=1).run(), max_excused_frac=0.1)
# data errors must be caught by the ordinary checks, not by the range checks
w = W.make_config(5, B=8, V=900)
k = w.k_per_row.copy(); k[7] += 2
dev = DeviceBatch(w)
import torch
dev.k = torch.from_numpy(k).cuda()
st = dev.run()[2]
assert st[7] == 1
assert binding.debug_violation() == 0, binding.debug_violation()
print("debug build clean")
"""


def test_no_range_check_fires_in_the_debug_build():
    from paper_2411_00853_b200 import build
    lib = build.build(variant="debug")
    env = dict(os.environ, SPECV_LIB=lib, PYTHONPATH=ROOT)
    res = subprocess.run([sys.executable, "-c", CHILD], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "debug build clean" in res.stdout, (res.stdout + res.stderr)[-3000:]


def test_the_release_build_has_no_range_checks():
    from paper_2411_00853_b200 import binding
    assert binding.debug_violation() == -1
