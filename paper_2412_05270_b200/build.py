"""Builds libapollo.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libapollo.so"
LIB_DEBUG = PKG / "libapollo_debug.so"      # the same sources with -DAPOLLO_DEBUG: index checks inside the kernels
SOURCES = ["apollo_api.cu", "kernels_basic.cu", "kernels_tensor.cu", "apollo_static.cu", "kernels_adamw.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def _stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    built = lib.stat().st_mtime
    deps = list(CSRC.glob("*")) + [PKG.parent / "include" / "apollo.h", Path(__file__)]
    return any(p.stat().st_mtime > built for p in deps)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> Path:
    """Compiles the library in-tree.  debug=True builds libapollo_debug.so: every kernel checks the index
    range of its global loads and stores and reports a violation through the context's status word
    (apollo_status returns APOLLO_ERR_INTERNAL) instead of making the access."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objs = []
    obj_dir = PKG / ("_build/debug" if debug else "_build")
    obj_dir.mkdir(parents=True, exist_ok=True)
    flags = NVCC_FLAGS + (["-DAPOLLO_DEBUG"] if debug else [])
    procs = []
    for src in SOURCES:
        obj = obj_dir / (src + ".o")
        cmd = [nvcc, *flags, "-c", str(CSRC / src), "-o", str(obj)]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(str(obj))
    for src, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            print(out)
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
    tmp = lib.with_suffix(f".{os.getpid()}.tmp")
    subprocess.run([nvcc, "-shared", "-o", str(tmp), *objs, "-Xcompiler", "-fvisibility=hidden"], check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
