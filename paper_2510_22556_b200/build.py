"""Builds libsablock.so in-tree with nvcc for sm_100a (no JIT, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsablock.so")
SOURCES = ["sablock.cu"]
HEADERS = ["common.cuh", "stages.cuh", "score_simt.cuh", "score_tc.cuh", "score_fused.cuh", "decode.cuh"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "sablock.h"))
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def _compile(out: str, defines=(), verbose: bool = False) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"] + [f"-D{d}" for d in defines] + \
          ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    _compile(LIB, verbose=verbose)
    return LIB


HOOKS_LIB = os.path.join(HERE, "libsablock_hooks.so")


def build_test_hooks(force: bool = False, wait_limit_cycles: int = 2_000_000) -> str:
    """A second library for the tests of the give-up paths: the same sources with the bounded
    waits shortened to about a millisecond and with the hooks compiled in that let a test make
    one producer withhold its post.  The product library is not touched."""
    if not force and not _stale(HOOKS_LIB):
        return HOOKS_LIB
    _compile(HOOKS_LIB, defines=("SABLOCK_TEST_HOOKS", f"SABLOCK_WAIT_LIMIT_CYCLES={int(wait_limit_cycles)}LL"))
    return HOOKS_LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
