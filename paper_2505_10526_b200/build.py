"""Compile the CUDA sources into ``libmassv.so`` for sm_100a with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(os.path.dirname(PKG), "include")
LIB = os.path.join(PKG, "libmassv.so")
SOURCES = ["api.cu", "attn.cu", "attn_umma.cu", "lm_head.cu", "accept.cu", "accept_static.cu", "tensor_map.cu", "tvd.cu", "top_p.cu"]


TEST_LIB = os.path.join(PKG, "libmassv_testhooks.so")


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "massv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(out, extra, verbose=False):
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC] + extra + \
          ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or _stale()):
        return LIB
    return _compile(LIB, [], verbose)


def build_test_hooks(force: bool = False) -> str:
    """The same sources with the test hooks compiled in and a short limit on device-side waits: only
    the tests load it (to make a bounded wait run out on purpose, on a tiny problem)."""
    if not (force or _stale(TEST_LIB)):
        return TEST_LIB
    return _compile(TEST_LIB, ["-DMASSV_TEST_HOOKS", "-DMASSV_SPIN_LIMIT=65536u"])


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
