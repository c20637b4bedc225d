"""Builds `libbranchattn.so` (sm_100a only) next to this file with nvcc."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libbranchattn.so")
TAP_LIB_PATH = os.path.join(_HERE, "libtapchannel.so")     # TapChannel: a separate, small library

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def sources():
    return sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = sources() + glob.glob(os.path.join(_HERE, "csrc", "*.cuh")) + \
        glob.glob(os.path.join(_ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build_tap(force: bool = False) -> str:
    src = os.path.join(_HERE, "tap", "tap_channel.cu")
    deps = [src, os.path.join(_ROOT, "include", "tap_channel.h")]
    if force or not os.path.exists(TAP_LIB_PATH) or any(os.path.getmtime(d) > os.path.getmtime(TAP_LIB_PATH) for d in deps):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, *NVCC_FLAGS, "-I", os.path.join(_ROOT, "include"), "-o", TAP_LIB_PATH, src,
                               "-lrt", "-lpthread"])
    return TAP_LIB_PATH


def build(force: bool = False, verbose: bool = False) -> str:
    build_tap(force)
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(_ROOT, "include"),
               "-I", os.path.join(_HERE, "csrc"), "-o", LIB_PATH, *sources()]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.check_call(cmd)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
