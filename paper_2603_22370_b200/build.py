"""Builds libfaar.so (sm_100a) in-tree with nvcc.  `python -m paper_2603_22370_b200.build`."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfaar.so")
LIB_DEBUG = os.path.join(HERE, "libfaar_debug.so")     # -DFAAR_DEBUG: epilogue stores checked against tensor extents
SOURCES = ["faar_api.cu", "faar_elementwise.cu", "faar_gemm.cu", "faar_static_scratch.cu", "faar_align.cu", "faar_glue.cu", "faar_fp4_gemm.cu", "faar_attention.cu", "faar_attention_tc.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "faar.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles the library in-tree.  debug=True builds libfaar_debug.so with -DFAAR_DEBUG instead: the same
    entry points, every store of the tensor-core kernels' epilogues checked against the extent of the tensor it
    writes (a store that would leave it is skipped and reported through the workspace status word).  The
    binding loads it when FAAR_LIB names it."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(lib):
        return lib
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug:
        cmd += ["-DFAAR_DEBUG"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
