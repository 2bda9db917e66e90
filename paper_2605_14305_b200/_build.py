"""Compile the CUDA library in-tree for sm_100a with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(HERE, "libfef.so")
SOURCES = ["fef_verify.cu", "fef_remask.cu", "fef_draft.cu", "fef_loop.cu", "fef_lmhead.cu", "fef_synth.cu"]
HEADERS = [os.path.join(CSRC, h) for h in ("fef_common.cuh", "fef_device_math.cuh", "fef_verify_params.cuh",
                                            "fef_residual.cuh")] + [os.path.join(INCLUDE, "fef.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; cannot build libfef.so")


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """nvcc -gencode arch=compute_100a,code=sm_100a ... -> paper_2605_14305_b200/libfef.so"""
    if not force and not needs_build():
        return LIB_PATH
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [
        nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-I", INCLUDE, "-I", CSRC, "-shared", "-Xcompiler", "-fPIC", "-o", tmp,
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


TEST_HOOKS_LIB_PATH = os.path.join(HERE, "libfef_testhooks.so")


def build_test_hooks(force: bool = False) -> str:
    """The library compiled with -DFEF_TEST_HOOKS (adds fef_test_withhold_stage_once, which lets a test
    make one bounded wait of the streaming kernel run out).  Used by the GPU tests only."""
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    if not force and os.path.exists(TEST_HOOKS_LIB_PATH) and \
            all(os.path.getmtime(d) <= os.path.getmtime(TEST_HOOKS_LIB_PATH) for d in deps):
        return TEST_HOOKS_LIB_PATH
    tmp = TEST_HOOKS_LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-DFEF_TEST_HOOKS",
           "-I", INCLUDE, "-I", CSRC, "-shared", "-Xcompiler", "-fPIC", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, TEST_HOOKS_LIB_PATH)
    return TEST_HOOKS_LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
