"""Compile the CUDA library in-tree for sm_100a with nvcc (works without a GPU)."""
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libgproj_attn.so")
SOURCES = [os.path.join(CSRC, "gproj_attn.cu")]
HEADERS = [os.path.join(CSRC, f) for f in ("sm100_primitives.cuh", "attn_fwd.cuh", "attn_bwd.cuh", "attn_bwd_w128.cuh", "key_smoothing.cuh", "attn_fp32.cuh")] + \
          [os.path.join(ROOT, "include", "gproj_attn.h")]


def nvcc_command(verbose: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", LIB] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    deps = SOURCES + HEADERS
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(p) for p in deps):
        return LIB
    res = subprocess.run(nvcc_command(verbose), capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
