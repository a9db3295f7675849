"""Build the CUDA libraries in-tree for sm_100a with plain nvcc (cross-compiles without a GPU).

    libcocod.so         the engine (C boundary of include/cocod.h)
    libcocod_inputs.so  the device build of the synthetic-input generator (not part of the path)
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC]

TARGETS = {
    "libcocod.so": ["cocod_engine.cu", "cocod_mlp.cu"],
    "libcocod_inputs.so": ["inputs_gen.cu"],
}


def _stale(out: str, srcs: list[str]) -> bool:
    if not os.path.exists(out):
        return True
    deps = list(srcs) + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    deps += [os.path.join(ROOT, "include", f) for f in os.listdir(os.path.join(ROOT, "include"))]
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> list[str]:
    nvcc = os.environ.get("NVCC", "nvcc")
    outs = []
    for name, files in TARGETS.items():
        out = os.path.join(HERE, name)
        srcs = [os.path.join(CSRC, f) for f in files]
        if force or _stale(out, srcs):
            tmp = out + f".tmp{os.getpid()}"
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + srcs + ["-o", tmp]
            subprocess.check_call(cmd)
            os.replace(tmp, out)
        outs.append(out)
    return outs


if __name__ == "__main__":
    print("\n".join(build(force="--force" in sys.argv, verbose="-v" in sys.argv)))
