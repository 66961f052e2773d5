"""The allocation-free per-op step (cp_step_unfused_noalloc), collected last.

Some users of the library may not allocate device memory at the point where they step
their environments — for instance a control loop that cannot afford the device-wide stall
an allocation may cause, or a plugin whose host application owns all device memory. For
them the per-op step keeps its intermediate planes in an array that is part of the
library. This test calls that entry point through the C ABI twice in a row and checks
both results against the ordinary cp_step_unfused (caller-supplied workspace) bit for
bit, which is the tolerance the ladder tests use; the second call runs over the first
call's leftovers in the shared array.
"""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()  # no-op when the in-tree library matches the sources
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def _planes(n, z=None):
    p = torch.zeros(4, (n + 3) // 4 * 4, dtype=torch.float32, device="cuda")
    if z is not None:
        p[:, :n] = torch.from_numpy(z).cuda()
    return p


def _run(cp, fn, z, seed, t, action, off):
    n = z.shape[1]
    pin, pout = _planes(n, z), _planes(n)
    s_in, s_out = cp.cp_wrap(pin, n, seed, t, off), cp.cp_wrap(pout, n, 0)
    reward = torch.full((n,), -3.0, dtype=torch.float32, device="cuda")
    done = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    act = torch.from_numpy(action).cuda() if action is not None else None
    fn(s_in, act, s_out, reward, done)
    torch.cuda.synchronize()
    info = s_out.info()
    assert (info["t"], info["seed"], info["env_offset"]) == (t + 1, seed, off)
    return pout[:, :n].cpu().numpy(), reward.cpu().numpy(), done.cpu().numpy()


def test_noalloc_step_equals_workspace_step_twice_in_a_row(cp):
    # two different batches back to back: a ragged size first, then the maximum size
    cases = [(50001, "edge", None, 11, 5), (cp.CP_NOALLOC_MAX_ENVS, "live", inputs.random_actions(cp.CP_NOALLOC_MAX_ENVS, 4), 3, 0)]
    for n, spread, action, t, off in cases:
        z = inputs.random_states(n, seed=n % 97, spread=spread)
        ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        want = _run(cp, lambda a, b, c, d, e: cp.cp_step_unfused(a, b, c, d, e, ws), z, 7, t, action, off)
        del ws
        got = _run(cp, cp.cp_step_unfused_noalloc, z, 7, t, action, off)
        for w, g in zip(want, got):
            assert np.array_equal(w.view(np.uint8), g.view(np.uint8))
        assert want[2].any() and not want[2].all()


def test_noalloc_step_rejects_oversized_batches(cp):
    n = cp.CP_NOALLOC_MAX_ENVS + 1
    pin, pout = _planes(n), _planes(n)
    s_in, s_out = cp.cp_wrap(pin, n, 0), cp.cp_wrap(pout, n, 0)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    before = cp.cp_launch_count()
    with pytest.raises(cp.CartpoleError) as e:
        cp.cp_step_unfused_noalloc(s_in, None, s_out, reward, done)
    assert e.value.code == cp.CP_EINVAL and "CP_NOALLOC_MAX_ENVS" in str(e.value)
    assert cp.cp_launch_count() == before and s_out.info()["t"] == 0


def test_noalloc_step_refuses_in_place_use_and_takes_no_device_memory(cp):
    n = 4096
    z = inputs.random_states(n, seed=1, spread="live")
    pin, pout = _planes(n, z), _planes(n)
    s_in, s_out = cp.cp_wrap(pin, n, 0), cp.cp_wrap(pout, n, 0)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    # in place (a size the call accepts otherwise): refused on the host, nothing launched
    before = cp.cp_launch_count()
    with pytest.raises(cp.CartpoleError) as e:
        cp.cp_step_unfused_noalloc(s_in, None, s_in, reward, done)
    assert e.value.code == cp.CP_EINVAL and "in place" in str(e.value)
    assert cp.cp_launch_count() == before and s_in.info()["t"] == 0
    # a call after the first one on this device (which may have loaded the module that holds the
    # array) leaves the device's free memory exactly as it found it
    cp.cp_step_unfused_noalloc(s_in, None, s_out, reward, done)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    cp.cp_set_time(s_in, 0)
    cp.cp_step_unfused_noalloc(s_in, None, s_out, reward, done)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert cp.cp_launch_count() - before == 2 * 46
