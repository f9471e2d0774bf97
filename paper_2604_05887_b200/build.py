"""Builds libhkv.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libhkv.so")
SOURCES = ["hkv_api.cu", "hkv_classify.cu", "hkv_compress.cu", "hkv_decode.cu", "hkv_noalloc.cu", "hkv_policy.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "hkv.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compile every .cu under csrc/ into one shared library; returns its path.

    extra_flags / out: a second build of the same sources beside the product library (the checked build
    with -DHKV_CHECKED, the profiling build with -DHKV_PROFILE); such a build is always recompiled when
    its sources are newer than it."""
    lib_path = out or LIB_PATH
    if not force and not needs_build(lib_path):
        return lib_path
    cmd = [_nvcc(), "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib_path] + list(extra_flags) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib_path)}")
    return lib_path


# Second builds of the same sources, kept beside the product library.
CHECKED_LIB_PATH = os.path.join(PKG_DIR, "libhkv_checked.so")    # index validation + short wait limit + wait self-test
PROFILE_LIB_PATH = os.path.join(PKG_DIR, "libhkv_profile.so")    # phase time stamps of the decode kernel


def build_checked(force: bool = False) -> str:
    return build_library(force, extra_flags=["-DHKV_CHECKED", "-DHKV_WAIT_CYCLES=400000000ll"], out=CHECKED_LIB_PATH)


def build_profile(force: bool = False) -> str:
    return build_library(force, extra_flags=["-DHKV_PROFILE"], out=PROFILE_LIB_PATH)


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
