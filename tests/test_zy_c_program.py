"""The C ABI used from a plain C program (no Python in the product path): compile
tests/c_abi_program.c against include/cartpole.h with the host C compiler, link it with the in-tree
library, run it on the GPU and compare what it prints with the CPU oracle."""
import os
import subprocess

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def test_c_program_against_oracle(oracle, tmp_path):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import build
    lib = build.build()
    libdir = os.path.dirname(lib)
    exe = tmp_path / "c_abi_program"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-O1", os.path.join(ROOT, "tests", "c_abi_program.c"),
                    "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
                    "-L", libdir, "-l:libcartpole.so", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
                    f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{os.path.join(CUDA, 'lib64')}", "-o", str(exe)], check=True)
    n, T, seed = 5000, 120, 4
    res = subprocess.run([str(exe), str(n), str(T), str(seed)], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stderr
    out = dict(line.split(" ", 1) for line in res.stdout.strip().splitlines())
    assert "sm_100a" in out["version"] and out["t"] == "3"
    # per-step path: done counts of the first three steps
    r3 = oracle.rollout(n, 3, seed, done_bits=True)
    want_counts = [int(np.unpackbits(np.ascontiguousarray(r3["done_bits"][k]).view(np.uint8)).sum()) for k in range(3)]
    got_counts = [int(v) for v in out["done_counts"].split()]
    assert all(abs(g - w) <= 1 for g, w in zip(got_counts, want_counts)), (got_counts, want_counts)
    # rollout path
    o = oracle.rollout(n, T, seed)
    got_tot = [int(v) for v in out["totals"].split()]
    assert abs(got_tot[0] - int(o["totals"][0])) <= 1e-3 * int(o["totals"][0])
    assert abs(got_tot[1] - int(o["totals"][1])) <= 1e-3 * int(o["totals"][1]) + 1
    got_ret = np.array([float(v) for v in out["returns"].split()], np.float32)
    assert (got_ret == o["ep_return_sum"][:16]).mean() >= 0.9
    # the refused call
    code, text = out["bad_call"].split(" ", 1)
    assert int(code) == -1 and "T must be" in text
