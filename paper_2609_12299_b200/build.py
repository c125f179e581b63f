"""In-tree build of the CUDA library and the trace generators (nvcc / g++, sm_100a only)."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _stale(out: str, deps: list[str]) -> bool:
    return not os.path.exists(out) or os.path.getmtime(out) < max(os.path.getmtime(d) for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    csrc = os.path.join(_HERE, "csrc")
    srcs = sorted(glob.glob(os.path.join(csrc, "*.cu")))
    deps = srcs + glob.glob(os.path.join(csrc, "*.cuh")) + [os.path.join(_ROOT, "include", "argus.h")]
    out = os.path.join(_HERE, "libargus.so")
    if force or _stale(out, deps):
        cmd = [NVCC, *ARCH, "-O3", "-lineinfo", "-std=c++17", "-I", os.path.join(_ROOT, "include"), "-shared",
               "-Xcompiler", "-fPIC", "-o", out, *srcs]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.check_call(cmd)
    return out


def build_tracegen(force: bool = False) -> list[str]:
    d = os.path.join(_HERE, "tracegen")
    hdr = os.path.join(d, "tracegen.h")
    host_src, cuda_src = os.path.join(d, "tracegen_host.cpp"), os.path.join(d, "tracegen_cuda.cu")
    host_out, cuda_out = os.path.join(d, "libtracegen_host.so"), os.path.join(d, "libtracegen_cuda.so")
    if force or _stale(host_out, [host_src, hdr]):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-pthread", "-o", host_out, host_src])
    if force or _stale(cuda_out, [cuda_src, hdr]):
        subprocess.check_call([NVCC, *ARCH, "-O3", "-fmad=false", "-lineinfo", "-shared", "-Xcompiler", "-fPIC", "-o",
                               cuda_out, cuda_src])
    return [host_out, cuda_out]


def build_all(force: bool = False) -> None:
    build_library(force)
    build_tracegen(force)


if __name__ == "__main__":
    build_all(force=True)
