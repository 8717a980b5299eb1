"""Builds the CUDA library in-tree: paper_2006_08173_b200/liblgn.so (sm_100a).

Every source file is compiled to an object of its own, all of them at the same time (the
kernel instances are spread over lgn_inst_*.cu for that purpose), then linked."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_PKG, "_build")
LIB_PATH = os.path.join(_PKG, "liblgn.so")
SOURCES = [os.path.join(_CSRC, f) for f in (
    "lgn.cu", "lgn_inst_f32.cu", "lgn_inst_bf16.cu", "lgn_inst_bf16_big.cu", "lgn_inst_f32_small.cu", "lgn_inst_bf16_small.cu", "lgn_inst_misc.cu",
    "lgn_prefix.cu", "lgn_dequant.cu", "lgn_quantile.cu", "lgn_host.cu")]
_HEADERS = [os.path.join(_CSRC, "lgn_kernels.cuh"), os.path.join(_CSRC, "lgn_device.cuh"),
            os.path.join(_CSRC, "lgn_closed_form.cuh"), os.path.join(_ROOT, "include", "lgn.h")]
_DEPS = SOURCES + _HEADERS


def _nvcc():
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def compile_command(src: str, obj: str, extra=()):
    return [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
            "-Xcompiler", "-fPIC", "-I", os.path.join(_ROOT, "include"), "-I", _CSRC, *extra, "-c", src, "-o", obj]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or needs_build()):
        return LIB_PATH
    os.makedirs(_OBJ, exist_ok=True)
    extra = ("-Xptxas", "-v") if verbose else ()
    objs = [os.path.join(_OBJ, os.path.basename(s)[:-3] + ".o") for s in SOURCES]

    def one(pair):
        src, obj = pair
        r = subprocess.run(compile_command(src, obj, extra), capture_output=True, text=True)
        return src, r
    with ThreadPoolExecutor(len(SOURCES)) as ex:
        results = list(ex.map(one, zip(SOURCES, objs)))
    for src, r in results:
        if verbose or r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode != 0:
            raise subprocess.CalledProcessError(r.returncode, "nvcc -c " + src)
    subprocess.check_call([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB_PATH, *objs])
    return LIB_PATH


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB_PATH)
