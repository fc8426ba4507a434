"""Builds libspecverify.so (sm_100a) in-tree with nvcc.  `python -m paper_2411_00853_b200.build`.

Variants: --debug      libspecverify_debug.so, compiled with -DSPECV_DEBUG (range checks in the
                       streaming kernels, see spec_verify_debug_violation in the header)
          --sanitize   libspecverify_san.so, host code under AddressSanitizer and
                       UndefinedBehaviorSanitizer (load it with libasan preloaded)
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libspecverify.so")
LIB_DEBUG = os.path.join(HERE, "libspecverify_debug.so")
LIB_SANITIZE = os.path.join(HERE, "libspecverify_san.so")
SOURCES = ["spec_verify.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xptxas", "-v", "-Xcompiler", "-fPIC", "-shared"]
VARIANTS = {
    "release": (LIB, []),
    "debug": (LIB_DEBUG, ["-DSPECV_DEBUG"]),
    "sanitize": (LIB_SANITIZE, ["-Xcompiler", "-fsanitize=address", "-Xcompiler", "-fsanitize=undefined",
                                "-Xcompiler", "-fno-omit-frame-pointer", "-Xptxas", "-O1"]),
}


def _inputs():
    out = []
    for root, _, files in os.walk(CSRC):
        out += [os.path.join(root, f) for f in files if f.endswith((".cu", ".cuh", ".h"))]
    out.append(os.path.join(os.path.dirname(HERE), "include", "spec_verify.h"))
    return out


def build(force: bool = False, verbose: bool = False, variant: str = "release") -> str:
    lib, extra = VARIANTS[variant]
    newest = max(os.path.getmtime(p) for p in _inputs())
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [nvcc, *NVCC_FLAGS, *extra, "-o", tmp, *[os.path.join(CSRC, s) for s in SOURCES]]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed: " + " ".join(cmd))
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    which = [v for v in ("debug", "sanitize") if "--" + v in sys.argv[1:]] or ["release"]
    for v in which:
        print(build(force=True, verbose=True, variant=v))
