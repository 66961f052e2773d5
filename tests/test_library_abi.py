"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every
symbol the header declares, and rejects bad arguments on the host before any
CUDA work is attempted."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "cartpole.h")


@pytest.fixture(scope="module")
def cp():
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(cp):
    names = _declared()
    assert len(names) >= 20
    assert sorted(cp.EXPORTS) == names
    L = C.CDLL(cp.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n


def test_version_and_counters(cp):
    assert "sm_100a" in cp.cp_version()
    assert cp.cp_launch_count() >= 0


def test_host_side_argument_errors(cp):
    L = cp.lib()
    assert L.cp_tune(b"no_such_key", 1) == cp.CP_EINVAL
    assert b"unknown tuning key" in L.cp_last_error()
    assert L.cp_tune(b"rollout_block", 100) == cp.CP_EINVAL
    assert L.cp_tune(b"rollout_ept", 3) == cp.CP_EINVAL
    assert L.cp_tune(b"rollout_coop", 6) == cp.CP_EINVAL
    assert L.cp_tune(b"rollout_defer", 5) == cp.CP_EINVAL
    assert L.cp_tune(b"rollout_coop", 0) == cp.CP_OK
    assert L.cp_tune(b"rollout_block", 256) == cp.CP_OK
    assert L.cp_tune(b"rollout_block", 0) == cp.CP_OK
    r = cp.cp_returns()
    assert L.cp_rollout(0, 10, 0, None, C.byref(r)) == cp.CP_EINVAL
    assert L.cp_rollout(16, 0, 0, None, C.byref(r)) == cp.CP_EINVAL
    assert L.cp_rollout(16, (1 << 30) + 1, 0, None, C.byref(r)) == cp.CP_EINVAL
    assert L.cp_rollout(16, 10, 0, None, None) == cp.CP_EINVAL
    bad = cp.cp_policy(7, None)
    assert L.cp_rollout(16, 10, 0, C.byref(bad), C.byref(r)) == cp.CP_EINVAL
    noweights = cp.cp_policy(cp.CP_POLICY_MLP, None)
    assert L.cp_rollout(16, 10, 0, C.byref(noweights), C.byref(r)) == cp.CP_EINVAL
    assert L.cp_rollout_shard(0xFFFFFFFF, 16, 10, 0, None, C.byref(r)) == cp.CP_EINVAL
    assert not L.cp_wrap(None, 16, 16, 0, 0, 0)
    assert not L.cp_reset(0, 0)
    assert not L.cp_reset(-5, 0)
    assert L.cp_step(None, None, None, None, None) == cp.CP_EINVAL
    assert L.cp_step_unfused(None, None, None, None, None, None, 0) == cp.CP_EINVAL
    assert L.cp_actions(0, 0, 0, 0, None) == cp.CP_EINVAL
    assert L.cp_rollout_host(8, 10, 0, None, None, None, None) == cp.CP_EINVAL
    assert L.cp_step_host(8, 0, 0, None, None, None, None, None) == cp.CP_EINVAL
    assert L.cp_selftest_sincos(5, 1, None) == cp.CP_EINVAL
    L.cp_free(None)
    assert L.cp_unfused_workspace_bytes(0) == 0
    assert L.cp_unfused_workspace_bytes(1024) >= 1024 * (33 * 4 + 7)


def test_binding_structs_have_the_layout_the_header_declares(cp, tmp_path):
    """Compile the header with the host C compiler, print sizeof/offsetof of every struct member,
    and compare with the ctypes mirror in the binding."""
    import subprocess
    structs = {"cp_policy": cp.cp_policy, "cp_returns": cp.cp_returns, "cp_rollout_args": cp.cp_rollout_args}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "cartpole.h"', 'int main(void) {']
    for name, cls in structs.items():
        lines.append(f'printf("{name} %zu\\n", sizeof({name}));')
        for field, _ in cls._fields_:
            lines.append(f'printf("{name}.{field} %zu\\n", offsetof({name}, {field}));')
    lines += ['return 0; }']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for name, cls in structs.items():
        assert int(got[name]) == C.sizeof(cls), name
        for field, _ in cls._fields_:
            assert int(got[f"{name}.{field}"]) == getattr(cls, field).offset, f"{name}.{field}"
    # and every member the header declares is mirrored (count the members of each struct body)
    text = re.sub(r"/\*.*?\*/", "", open(HEADER).read(), flags=re.S)
    for name, cls in structs.items():
        body = re.search(r"typedef struct %s \{(.*?)\} %s;" % (name, name), text, flags=re.S).group(1)
        members = [m for decl in body.split(";") for m in decl.split(",") if m.strip()]
        assert len(members) == len(cls._fields_), (name, members)


def test_misaligned_rollout_outputs_are_refused_before_any_launch(cp):
    """Every cp_returns member is stored in 4-byte units (totals in 8-byte units): an odd pointer
    must come back as CP_EINVAL from the host-side checks, never reach a kernel (no GPU is needed
    for this test, and none must be touched)."""
    L = cp.lib()
    before = L.cp_launch_count()
    base = 0x7000_0000_0000
    for field in ("ep_return_sum", "ep_count", "reward_stream", "done_bits", "action_bits", "final_state",
                  "trajectory", "totals"):
        for odd in (1, 2, 3) if field != "totals" else (4,):
            r = cp.cp_returns()
            setattr(r, field, base + odd)
            assert L.cp_rollout(64, 10, 0, None, C.byref(r)) == cp.CP_EINVAL, field
            assert field.encode() in L.cp_last_error() or b"aligned" in L.cp_last_error()
    a = cp.cp_rollout_args()
    a.struct_size = C.sizeof(cp.cp_rollout_args)
    r = cp.cp_returns()
    a.n_envs, a.T, a.returns = 64, 10, C.pointer(r)
    a.ep_len = base + 2
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    assert L.cp_launch_count() == before


def test_general_rollout_rejects_bad_arguments_on_the_host(cp):
    L = cp.lib()
    r = cp.cp_returns()
    a = cp.cp_rollout_args()
    a.n_envs, a.T, a.returns = 16, 10, C.pointer(r)
    a.struct_size = C.sizeof(cp.cp_rollout_args) - 8
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    assert b"struct_size" in L.cp_last_error()
    a.struct_size = C.sizeof(cp.cp_rollout_args)
    a.arithmetic = 2
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    assert b"arithmetic" in L.cp_last_error()
    a.arithmetic = cp.CP_ARITH_CONTRACTED
    a.T = 0
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    a.T = 10
    a.returns = None
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    assert L.cp_rollout_ex(None) == cp.CP_EINVAL


def test_allocator_hooks_are_called_and_paired(cp):
    """cp_reset takes its batch from the installed allocator and gives it back through the paired
    release function: checked with a fake allocator (on a machine without a GPU the start-state
    launch fails, and the batch must come back through release before cp_reset returns NULL)."""
    import torch
    L = cp.lib()
    assert L.cp_set_allocator(cp.ALLOC_FN(lambda n: 0), cp.RELEASE_FN(0)) == cp.CP_EINVAL
    if torch.cuda.is_available():
        pytest.skip("the fake device pointer must never reach a real launch")
    calls = []

    def alloc(nbytes):
        calls.append(("alloc", nbytes))
        return 0x7000_0000_0000 if nbytes < (1 << 30) else 0

    def release(ptr):
        calls.append(("release", ptr))

    cp.cp_set_allocator(alloc, release)
    try:
        assert not L.cp_reset(1001, 3)                     # no device: launch error
        assert calls == [("alloc", 1004 * 16), ("release", 0x7000_0000_0000)]
        calls.clear()
        assert not L.cp_reset(1 << 27, 3)                  # allocator says no
        assert calls == [("alloc", (1 << 27) * 16)] and b"allocator returned NULL" in L.cp_last_error()
    finally:
        cp.cp_set_allocator(None, None)
    calls.clear()
    assert not L.cp_reset(8, 0)                            # default allocator again: hooks untouched
    assert calls == []


def test_wrap_bookkeeping_needs_no_gpu(cp):
    L = cp.lib()
    fake = C.c_void_p(0x7000_0000_0100)  # never dereferenced on the host
    h = L.cp_wrap(fake, 100, 128, 9, 5, 1000)
    assert h
    st = cp.State(h)
    info = st.info()
    assert info == {"n_envs": 100, "plane_stride": 128, "seed": 9, "t": 5, "env_offset": 1000,
                    "planes": 0x7000_0000_0100}
    cp.cp_set_time(st, 77)
    assert st.info()["t"] == 77
    assert not L.cp_wrap(fake, 100, 64, 0, 0, 0)  # stride < n
    st.close()


def test_missing_library_fails_loudly(cp, monkeypatch):
    monkeypatch.setattr(cp, "_lib", None)
    monkeypatch.setattr(cp, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(ImportError):
        cp.lib()
