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
DEBUG_LIB = os.path.join(PKG, "libmassv_debug.so")


def _stale(lib=LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "massv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def _command(out, extra, verbose=False):
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC] + extra + \
          ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES] + ["-ldl"]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    return cmd


def _compile(out, extra, verbose=False):
    subprocess.run(_command(out, extra, verbose), check=True)
    return out


VARIANTS = {LIB: [], TEST_LIB: ["-DMASSV_TEST_HOOKS", "-DMASSV_SPIN_LIMIT=65536u"], DEBUG_LIB: ["-DMASSV_DEBUG"]}


def build_all(force: bool = False):
    """The library and its two test variants, the stale ones compiled side by side."""
    procs = [(lib, subprocess.Popen(_command(lib, extra))) for lib, extra in VARIANTS.items() if force or _stale(lib)]
    for lib, proc in procs:
        if proc.wait() != 0:
            raise subprocess.CalledProcessError(proc.returncode, "nvcc -o " + lib)
    return list(VARIANTS)


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


def build_debug(force: bool = False) -> str:
    """The same sources with -DMASSV_DEBUG: index checks on the device that record MASSV_ERR_BOUNDS in the status
    word and skip the access.  The binding loads it instead of the ordinary library when MASSV_DEBUG=1 is set."""
    if not (force or _stale(DEBUG_LIB)):
        return DEBUG_LIB
    return _compile(DEBUG_LIB, VARIANTS[DEBUG_LIB])


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
