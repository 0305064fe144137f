"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libattn_fwd.so")
# The same sources with the test hooks compiled in (bounded waits of 1 ms instead of 1 s, and an extra
# entry that makes the producer leave out one K/V load): used by one GPU test to make a wait run out
# and check the time-out status.  Never loaded by the package.
WAIT_TEST_LIB_PATH = os.path.join(_HERE, "libattn_fwd_waittest.so")
WAIT_TEST_FLAGS = ["-DATTN_TEST_HOOKS", "-DATTN_TEST_WAIT_LIMIT_NS=1000000ull"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cuh"))
                  + glob.glob(os.path.join(_HERE, "..", "include", "*.h")))


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(s) > t for s in _sources())


def _compile(path: str, extra, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = path + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + [
        "-o", tmp, os.path.join(CSRC, "attn_api.cu")]
    subprocess.check_call(cmd)
    os.replace(tmp, path)
    return path


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/attn_api.cu (which includes every kernel header) into libattn_fwd.so."""
    if not force and not is_stale():
        return LIB_PATH
    return _compile(LIB_PATH, [], verbose)


def build_wait_test(force: bool = False) -> str:
    """Compile the test-hook variant of the library (see WAIT_TEST_LIB_PATH)."""
    if not force and not is_stale(WAIT_TEST_LIB_PATH):
        return WAIT_TEST_LIB_PATH
    return _compile(WAIT_TEST_LIB_PATH, WAIT_TEST_FLAGS, False)


if __name__ == "__main__":
    print(build(force=True, verbose=True))
