"""Build libpie.so (the C-ABI library) and libpie_synth.so (input generator kernels) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
         "--use_fast_math"]

LIBS = {
    "libpie.so": ["pie_table.cpp", "pie_kernels.cu", "pie_prefill.cu", "pie_pool.cu", "pie_noalloc.cu"],
    "libpie_synth.so": ["pie_synth.cu"],
}


def _stale(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    deps = list(sources) + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".h")]
    deps.append(os.path.join(HERE, "..", "include", "pie.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> None:
    for lib, names in LIBS.items():
        target = os.path.join(HERE, lib)
        sources = [os.path.join(CSRC, n) for n in names]
        if not force and not _stale(target, sources):
            continue
        tmp = target + f".{os.getpid()}.tmp"
        cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-shared", "-o", tmp] + sources
        subprocess.check_call(cmd)
        os.replace(tmp, target)


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
