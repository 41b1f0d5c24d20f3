"""Builds the CUDA library in-tree: nvcc -> paper_2605_03884_b200/libqkvshare.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libqkvshare.so")
SOURCES = ["qkvshare.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-shared", "-cudart", "static",
]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES]


def _deps():
    out = _sources() + [os.path.join(ROOT, "include", "qkvshare.h")]
    out += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    return out


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _deps())


def build(force: bool = False, verbose: bool = False, ptxas_info: bool = False,
          defines: dict | None = None, out_path: str | None = None) -> str:
    """Compile the library.  `defines` overrides tuning constants of the kernels (stages per
    warp, warps per CTA, CTAs per SM) and `out_path` writes the result somewhere else than the
    in-tree default; both exist for tuning sweeps."""
    out = out_path or LIB_PATH
    if not force and out_path is None and not is_stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + ["-I", os.path.join(ROOT, "include"), "-I", CSRC]
    for k, v in (defines or {}).items():
        cmd.append(f"-D{k}={v}")
    if ptxas_info:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", tmp] + _sources()
    if verbose:
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas-info" in sys.argv)
    print(LIB_PATH)
