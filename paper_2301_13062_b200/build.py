"""Build libcartpole.so in-tree with nvcc for sm_100a.

Run as ``python -m paper_2301_13062_b200.build``. nvcc cross-compiles without a GPU.
No fast-math; separate multiply/add are never contracted (``--fmad=false`` on top
of the explicit round-to-nearest intrinsics in the kernels).

The library is rebuilt when the hash of the sources and flags differs from the one
recorded beside it at the last build (file times are not used: a copy of the tree keeps
a valid library valid).
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcartpole.so")
STAMP = os.path.join(HERE, "libcartpole.so.stamp")
SOURCES = ["rollout_networks.cu", "rollout_networks_contracted.cu", "rollout_kernel.cu", "rollout_contracted.cu",
           "rollout_assisted.cu", "rollout_deferred.cu", "rollout_deferred_networks.cu", "rollout_deferred_mlp64.cu", "capi.cu", "step_kernel.cu", "ladder_kernels.cu", "ladder_noalloc.cu"]
HEADERS = ["cartpole_device.cuh", "cartpole_internal.h", "rollout_kernel.cuh", "rollout_deferred.cuh", os.path.join("..", "..", "include", "cartpole.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--fmad=false",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def source_hash() -> str:
    h = hashlib.sha256()
    for name in SOURCES + HEADERS:
        with open(os.path.normpath(os.path.join(CSRC, name)), "rb") as f:
            h.update(name.encode() + b"\0" + f.read() + b"\0")
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def kernel_hash() -> str:
    """Hash of the files and flags that determine the instruction streams of the rollout and step
    kernels (bench.py records it beside the per-env-step instruction counts it was given)."""
    h = hashlib.sha256()
    for name in ("cartpole_device.cuh", "rollout_kernel.cuh", "rollout_deferred.cuh", "rollout_deferred.cu", "step_kernel.cu"):
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read() + b"\0")
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()[:16]


def _compile_and_link(out: str, verbose: bool) -> None:
    with tempfile.TemporaryDirectory() as tmp:
        def compile_one(src: str) -> str:
            o = os.path.join(tmp, src.replace(".cu", ".o"))
            cmd = [_nvcc(), *NVCC_FLAGS, "-c", os.path.join(CSRC, src), "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
                print(" ".join(cmd), flush=True)
            subprocess.run(cmd, check=True)
            return o

        with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
            objs = list(pool.map(compile_one, SOURCES))
        tmp_out = out + ".tmp"
        subprocess.run([_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp_out, *objs],
                       check=True)
        os.replace(tmp_out, out)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile and link if the library is missing or older than its sources (by hash)."""
    want = source_hash()
    have = open(STAMP).read().strip() if os.path.exists(STAMP) else ""
    if force or not os.path.exists(LIB) or have != want:
        _compile_and_link(LIB, verbose)
        with open(STAMP, "w") as f:
            f.write(want + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
