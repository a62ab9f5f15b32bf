"""Builds the CUDA library (libdquant.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_INC = os.path.join(os.path.dirname(_PKG), "include")
LIB_PATH = os.path.join(_PKG, "libdquant.so")

# Extra nvcc flags for every translation unit can be given in the environment variable
# DQ_NVCC_EXTRA (e.g. "-Xptxas -v" variants while tuning).
# (source, extra flags).  The encoder is compiled without FMA contraction: its records must be
# reproducible bit for bit, every rounding is written out explicitly.
_SOURCES = [
    ("dq_tables.cu", []),
    ("dq_api.cu", []),
    ("dq_decode_tokens.cu", []),
    ("dq_attention.cu", []),
    ("dq_attention_wide.cu", []),
    ("dq_microbench.cu", []),
    ("dq_encode.cu", ["-fmad=false"]),
]
_COMMON = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-I", _INC, "-I", _CSRC]


def _newer(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "nvcc")
    obj_dir = os.path.join(_PKG, "build")
    os.makedirs(obj_dir, exist_ok=True)
    headers = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(_INC, "dq.h"))
    objs = []
    for src, extra in _SOURCES:
        s = os.path.join(_CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        if force or _newer(o, [s] + headers):
            cmd = [nvcc] + _COMMON + extra + os.environ.get("DQ_NVCC_EXTRA", "").split() + \
                  (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            subprocess.run(cmd, check=True)
        objs.append(o)
    if force or _newer(LIB_PATH, objs):
        tmp = LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.run([nvcc] + _COMMON[:2] + ["-shared", "-o", tmp] + objs, check=True)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
