"""Builds the C-ABI shared library ``liblvlm.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "liblvlm.so")
TEST_LIB = os.path.join(PKG, "liblvlm_test.so")      # the same sources with -DLVLM_TEST_HOOKS, for the tests only
SOURCES = ["lvlm.cu", "select.cu", "compact.cu", "merge_compact.cu", "kv_compress.cu",
           "decode.cu", "score.cu", "score_tc.cu", "nearest_kept.cu", "prefill_attn.cu"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "lvlm.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def _compile(lib: str, defines, verbose: bool) -> str:
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    cmd += ["-D" + d for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    return _compile(LIB, [], verbose)


def build_test(force: bool = False) -> str:
    """The library with its test hooks compiled in (switching programmatic dependent launch off)."""
    if not force and not needs_build(TEST_LIB):
        return TEST_LIB
    return _compile(TEST_LIB, ["LVLM_TEST_HOOKS"], False)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
