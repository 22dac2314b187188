"""Builds the CUDA library in-tree: paper_2605_14513_b200/libheart.so (sm_100a only).

`build()` makes the product library.  `build_test_hooks()` makes a second, test-only library
(libheart_testhooks.so) from the same sources with HEART_TEST_HOOKS defined and a short bounded-wait
limit: in it a reserved flag bit makes the attention kernel's V producer leave out one copy, so that
the kernel's time-out / abort / drain path can be exercised by a test without faulting or hanging
anything.  The product library does not contain that hook.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libheart.so")
LIB_TEST_HOOKS = os.path.join(HERE, "libheart_testhooks.so")
TEST_HOOK_DEFINES = ("HEART_TEST_HOOKS", "HEART_WAIT_LIMIT_CYCLES=2000000LL")
SOURCES = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cuh"))) + [os.path.join(ROOT, "include", "heart.h")]


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS + [os.path.abspath(__file__)])


def _compile(lib: str, defines=(), verbose: bool = False) -> str:
    """One nvcc process per source file (in parallel), then one link."""
    objdir = os.path.join(HERE, "build", os.path.splitext(os.path.basename(lib))[0])
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include")] + [f"-D{d}" for d in defines]
    if verbose:
        flags.append("-Xptxas=-v")

    def one(src):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        subprocess.check_call([nvcc()] + flags + ["-c", src, "-o", obj])
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(SOURCES))) as pool:
        objs = list(pool.map(one, SOURCES))
    subprocess.check_call([nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib] + objs)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale(LIB):
        _compile(LIB, verbose=verbose)
    return LIB


def build_test_hooks(force: bool = False) -> str:
    if force or stale(LIB_TEST_HOOKS):
        _compile(LIB_TEST_HOOKS, defines=TEST_HOOK_DEFINES)
    return LIB_TEST_HOOKS


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--test-hooks" in sys.argv:
        print(build_test_hooks(force="--force" in sys.argv))
