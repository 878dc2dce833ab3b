"""In-tree build of the CUDA library for sm_100a (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OUT = os.path.join(_HERE, "libaed_dec.so")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(OUT):
        return True
    built = os.path.getmtime(OUT)
    deps = _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(_HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(p) > built for p in deps)


def build_trace() -> str:
    """Debug build with device-side start-time stamps in every step kernel (libaed_dec_trace.so)."""
    out = os.path.join(_HERE, "libaed_dec_trace.so")
    src = os.path.join(CSRC, "debug", "trace_exports.cu")
    subprocess.run([os.environ.get("NVCC", "nvcc")] + NVCC_FLAGS + ["-DAED_TRACE", "-o", out, src], check=True)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libaed_dec.so next to this file; returns its path."""
    if not force and not _stale():
        return OUT
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = OUT + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + _sources()
    subprocess.run(cmd, check=True)
    os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
