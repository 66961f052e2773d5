"""Build libcartpole.so in-tree with nvcc for sm_100a.

Run as ``python -m paper_2301_13062_b200.build``. nvcc cross-compiles without a GPU.
No fast-math; separate multiply/add are never contracted (``--fmad=false`` on top
of the explicit round-to-nearest intrinsics in the kernels).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcartpole.so")
SOURCES = ["capi.cu", "step_kernel.cu", "ladder_kernels.cu", "rollout_kernel.cu", "ladder_noalloc.cu"]
HEADERS = ["cartpole_device.cuh", "cartpole_internal.h", os.path.join("..", "..", "include", "cartpole.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--fmad=false",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(target: str, deps: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra: list[str] | None = None, out: str | None = None) -> str:
    """Compile and link. `extra` adds nvcc flags (e.g. -DCP_ROLLOUT_MIN_CTAS=5) and `out` names
    another output file; both are for tuning experiments and force a full rebuild."""
    if extra or out:
        return _build_variant(extra or [], out or LIB, verbose)
    hdrs = [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS] + [os.path.abspath(__file__)]
    objs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src.replace(".cu", ".o"))
        if force or _stale(o, [s] + hdrs):
            cmd = [_nvcc(), *NVCC_FLAGS, "-c", s, "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
                print(" ".join(cmd), flush=True)
            subprocess.run(cmd, check=True)
        objs.append(o)
    if force or _stale(LIB, objs):
        cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB, *objs]
        subprocess.run(cmd, check=True)
    return LIB


def _build_variant(extra: list[str], out: str, verbose: bool) -> str:
    import tempfile
    with tempfile.TemporaryDirectory() as tmp:
        objs = []
        for src in SOURCES:
            o = os.path.join(tmp, src.replace(".cu", ".o"))
            cmd = [_nvcc(), *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            subprocess.run(cmd, check=True)
            objs.append(o)
        subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", out, *objs], check=True)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
