"""The C oracle and the host side of the CUDA library (argument validation, workspace and arena
layout) under AddressSanitizer and UndefinedBehaviorSanitizer.  Both are built with
-fsanitize=address,undefined and exercised in a child process that has libasan preloaded; any
report makes the child exit non-zero.  No GPU is involved: the library's entry points are called
only as far as their host-side checks go."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _asan_runtime():
    path = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    return path if os.path.isabs(path) and os.path.exists(path) else None


def _child_env(**extra):
    env = dict(os.environ)
    env.update(LD_PRELOAD=_asan_runtime(), PYTHONPATH=ROOT,
               ASAN_OPTIONS="detect_leaks=0:halt_on_error=1:protect_shadow_gap=0:abort_on_error=0",
               UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1", CUDA_VISIBLE_DEVICES="")
    env.update(extra)
    return env


pytestmark = pytest.mark.skipif(_asan_runtime() is None, reason="gcc's libasan runtime not found")


def test_oracle_under_address_and_undefined_behaviour_sanitizers():
    import oracle
    oracle.build(sanitize=True)
    res = subprocess.run(
        [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "tests/test_oracle_hand_cases.py",
         "tests/test_oracle_greedy.py", "tests/test_oracle_tree.py", "tests/test_oracle_properties.py",
         "-k", "not second_formulation and not fp16_logits_decode"],
        cwd=ROOT, env=_child_env(ORACLE_SANITIZE="1"), capture_output=True, text=True, timeout=900)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0, tail
    assert "passed" in res.stdout and "ERROR: AddressSanitizer" not in tail and "runtime error" not in tail


HOST_SIDE = r"""
import ctypes, itertools
from paper_2411_00853_b200 import binding
lib = binding.load()
assert binding.LIB_PATH.endswith("libspecverify_san.so")
# layout functions over many shapes, valid and not
for B, D, V in itertools.product((0, 1, 7, 512, 4095, 4096, 100000), (0, 1, 40, 4400, 1 << 20), (0, 1, 8, 4099, 128256, 1 << 22, (1 << 22) + 1)):
    w = binding.workspace_bytes(B, D, V)
    t = binding.tree_workspace_bytes(B, D, V)
    g = binding.greedy_workspace_bytes(B, D)
    for code in (0, 1, 2, 9):
        binding.host_arena_bytes(code, B, D, V)
    assert (w == 0) == (B < 1 or V < 1 or V > (1 << 22)) or D + B > 2**31 - 2
for code in range(-2, 14):
    assert binding.strerror(code)
# every argument check of the entry points, with pointers that are never dereferenced on the host
buf = (ctypes.c_char * 4096)()
p = ctypes.addressof(buf) & ~255
def call(**o):
    a = dict(tl=p, dl=p, dtype=1, V=64, ldt=64, ldd=64, tok=p, k=p, B=2, ku=0, D=10, T=p, per=0, u=p, acc=p, em=p, ws=p, wsb=1 << 20, flags=0)
    a.update(o)
    return lib.spec_verify_ex(a["tl"], a["dl"], a["dtype"], a["V"], a["ldt"], a["ldd"], a["tok"], a["k"], a["B"], a["ku"], a["D"],
                              a["T"], a["per"], a["u"], a["acc"], a["em"], None, None, None, a["ws"], a["wsb"], None, a["flags"], 0, 0, None)
assert call(tl=None) == 1 and call(V=0) == 2 and call(dtype=5) == 3 and call(ws=p + 8) == 4 and call(wsb=8) == 5
assert call(flags=3) == 9 and call(flags=64) == 9 and call(k=None, ku=3) == 2
assert call() in (6, 7)        # no device here: the call gets as far as asking for one
out = (ctypes.c_int64 * 4)()
assert lib.spec_verify_selftest_bounded_wait(0, out, None) == 2
assert lib.spec_verify_next_lookahead(p, 0, p, 0, 0, 4, p, None) == 2
assert lib.spec_verify_greedy(p, 7, 64, 64, p, p, 2, 0, 10, p, p, None, None, p, 1 << 20, None, 0) == 3
assert lib.spec_verify_tree(p, p, 1, 64, 64, 64, p, None, p, 2, 0, 10, p, 0, p, p, p, None, None, None, None, p, 1 << 20, None, 0) == 1
assert lib.spec_verify_noalloc(p, p, 1, 8, 8, 8, p, p, 30000, 0, 300000, p, 0, p, p, p, None, None, None, None) == 8
print("host side clean")
"""


def test_library_host_side_under_address_and_undefined_behaviour_sanitizers():
    from paper_2411_00853_b200 import build
    lib = build.build(variant="sanitize")
    res = subprocess.run([sys.executable, "-c", HOST_SIDE], cwd=ROOT, env=_child_env(SPECV_LIB=lib),
                         capture_output=True, text=True, timeout=600)
    tail = (res.stdout + res.stderr)[-3000:]
    assert res.returncode == 0 and "host side clean" in res.stdout, tail
    assert "ERROR: AddressSanitizer" not in tail and "runtime error" not in tail
