"""Builds the CUDA library in-tree: paper_2006_08173_b200/liblgn.so (sm_100a)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "liblgn.so")
SOURCES = [os.path.join(_CSRC, "lgn.cu"), os.path.join(_CSRC, "lgn_prefix.cu"),
           os.path.join(_CSRC, "lgn_dequant.cu"), os.path.join(_CSRC, "lgn_quantile.cu"),
           os.path.join(_CSRC, "lgn_host.cu")]
_DEPS = SOURCES + [os.path.join(_CSRC, "lgn_device.cuh"), os.path.join(_CSRC, "lgn_closed_form.cuh"),
                   os.path.join(_ROOT, "include", "lgn.h")]


def nvcc_command(extra=()):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
            "--threads", "0", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"), "-I", _CSRC,
            *extra, "-o", LIB_PATH, *SOURCES]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        cmd = nvcc_command(("-Xptxas", "-v") if verbose else ())
        subprocess.check_call(cmd)
    return LIB_PATH


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB_PATH)
