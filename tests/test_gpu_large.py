"""Maximum-size cases: batches whose arrays pass 2^31 and 2^32 bytes, so that any 32-bit index or
byte-offset arithmetic in the kernels would show. Compared with the oracle on env ranges at the
start, around the 2^29-th env and at the ragged end (the oracle computes any env range directly
from the global env ids)."""
import numpy as np
import pytest

from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

N_BIG = (1 << 29) + 37          # 536,870,949 envs: 2.1 GB per float plane
RANGES = [(0, 96), ((1 << 29) - 60, 96), (N_BIG - 70, 70)]


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    if torch.cuda.get_device_properties(0).total_memory < 60e9:
        pytest.skip("needs a GPU with 60 GB")
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def bits_of_range(words, lo, m):
    """[T, W] uint32 words of a done/action stream -> [T, m] bits of envs lo .. lo+m-1."""
    w0 = lo // 32
    chunk = words[:, w0:(lo + m + 31) // 32].cpu().numpy()
    return H.unpack_bits(chunk, (lo - 32 * w0) + m)[:, lo - 32 * w0:]


def test_rollout_beyond_4_gib(cp, oracle):
    n, seed = N_BIG, 5
    words = (n + 31) // 32
    ret = torch.full((n,), -1.0, device="cuda")
    cnt = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    tot = torch.zeros(2, dtype=torch.int64, device="cuda")
    # (a) 40 steps with the done bit stream (the general stream kernel): restarts happen
    T = 40
    done = torch.zeros(T, words, dtype=torch.int32, device="cuda")
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, ep_return_sum=ret, ep_count=cnt, totals=tot, done_bits=done)
    torch.cuda.synchronize()
    assert int(tot[1]) == int(cnt.sum(dtype=torch.int64)) and int(tot[0]) == int(ret.sum(dtype=torch.float64))
    assert 0.5 * n < int(tot[1]) < 3 * n
    for lo, m in RANGES:
        o = oracle.rollout(m, T, seed, env_offset=lo, done_bits=True)
        assert np.array_equal(ret[lo:lo + m].cpu().numpy(), o["ep_return_sum"]), lo
        assert np.array_equal(cnt[lo:lo + m].cpu().numpy().view(np.uint32), o["ep_count"]), lo
        assert np.array_equal(bits_of_range(done, lo, m), H.unpack_bits(o["done_bits"], m)), lo
    assert not bool((done[:, -1].cpu().numpy().view(np.uint32) >> (n % 32)).any())   # padding bits stay zero
    del done
    # (b) 3 steps from global time 18 with the reward plane (6.4 GB: row offsets pass 2^32 bytes)
    # and the done bits: the kernel with one running pointer per stream
    T, t0 = 3, 18
    reward = torch.zeros(T, n, device="cuda")
    done = torch.zeros(T, words, dtype=torch.int32, device="cuda")
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, t0=t0, ep_return_sum=ret, ep_count=cnt, reward_stream=reward,
                     done_bits=done)
    torch.cuda.synchronize()
    assert bool((reward == 1.0).all())
    for lo, m in RANGES:
        o = oracle.rollout(m, T, seed, env_offset=lo, t0=t0, done_bits=True)
        assert np.array_equal(ret[lo:lo + m].cpu().numpy(), o["ep_return_sum"]), lo
        assert np.array_equal(bits_of_range(done, lo, m), H.unpack_bits(o["done_bits"], m)), lo
    del reward, done, ret, cnt
    torch.cuda.empty_cache()


def test_last_environment_ids(cp, oracle):
    """The top of the 32-bit env-id space: the range that ends at id 2^32 - 1 is accepted and
    matches the oracle, one id further is refused on the host."""
    n, T, seed = 1000, 60, 2
    off = (1 << 32) - n
    ret = torch.empty(n, device="cuda")
    cnt = torch.empty(n, dtype=torch.int32, device="cuda")
    done = torch.zeros(T, (n + 31) // 32, dtype=torch.int32, device="cuda")
    cp.cp_rollout_shard(off, n, T, seed, None, ep_return_sum=ret, ep_count=cnt, done_bits=done)
    torch.cuda.synchronize()
    o = oracle.rollout(n, T, seed, env_offset=off, done_bits=True)
    assert np.array_equal(ret.cpu().numpy(), o["ep_return_sum"])
    assert np.array_equal(H.unpack_bits(done.cpu().numpy(), n), H.unpack_bits(o["done_bits"], n))
    with pytest.raises(cp.CartpoleError):
        cp.cp_rollout_shard(off + 1, n, T, seed, None, ep_return_sum=ret, ep_count=cnt)


def test_fused_step_beyond_4_gib(cp, oracle):
    n, seed = N_BIG, 5
    stride = (n + 3) // 4 * 4
    a = torch.empty(4, stride, device="cuda")                      # 8.6 GB: plane offsets pass 2^32 bytes
    b = torch.empty(4, stride, device="cuda")
    sa, sb = cp.cp_wrap(a, n, seed, 7), cp.cp_wrap(b, n, seed)
    cp.cp_fill_start(sa)
    reward = torch.zeros(n, device="cuda")
    done = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    cp.cp_step(sa, None, sb, reward, done)
    torch.cuda.synchronize()
    assert sb.info()["t"] == 8 and bool((reward == 1.0).all()) and int(done.max()) <= 1
    for lo, m in RANGES:
        z0 = oracle.initial_state(m, seed, 7, lo)
        assert np.array_equal(a[:, lo:lo + m].cpu().numpy().view(np.uint32), z0.view(np.uint32)), lo
        want = oracle.step(z0, seed=seed, t=7, env_offset=lo, want_pre_reset=True)
        H.assert_step_matches(want, z0, b[:, lo:lo + m].cpu().numpy(), reward[lo:lo + m].cpu().numpy(),
                              done[lo:lo + m].cpu().numpy())
    del a, b, reward, done
    torch.cuda.empty_cache()
