"""Builds libet.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python paper_2312_14227_b200/build.py [--force] [--verbose] [--debug-hooks]

Rebuilds only when a source is newer than the library (--force: always).  --debug-hooks compiles the
development switches in (forced tile shapes from the environment); the library built without it
reads nothing from the environment.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libet.so")
SOURCES = ["et_lib.cu", "et_noalloc.cu", "select.cpp"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "et.h")]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug_hooks: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [
        nvcc, "-shared", "-o", LIB, "-std=c++17", "-O3", "-lineinfo",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=default",
        "-I", os.path.join(ROOT, "include"), "-I", CSRC,
        "-cudart", "static", "-Xcompiler", "-pthread",
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug_hooks:
        cmd += ["-DET_DEBUG_HOOKS"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv or "--debug-hooks" in sys.argv, verbose="--verbose" in sys.argv,
                debug_hooks="--debug-hooks" in sys.argv))
