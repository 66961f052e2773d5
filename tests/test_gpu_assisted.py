"""The producer-assisted rollout kernel (very small batches: a helper warp hashes actions and start
states ahead of each stepping warp). It must give the same bits as the general kernel, which the
other files pin to the oracle, and it is compared with the oracle directly as well. Cases: ragged
batch sizes, horizons around the 16- and 32-step hand-overs, both CTA forms with an odd number of warp
tasks, a caller's initial state with angles outside the polynomial range, carried episode lengths
and the step limit."""
import contextlib

import numpy as np
import pytest

from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

ASSISTED, PER_LANE = 4, 2


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    torch.cuda.set_device(0)
    return binding


@contextlib.contextmanager
def kernel(cp, coop, block=0):
    cp.cp_tune("rollout_block", block)
    try:
        with H.rollout_shape(cp, 1, coop):
            yield
    finally:
        cp.cp_tune("rollout_block", 0)


def rollout(cp, coop, n, T, seed, block=0, streams=(), **kw):
    words = (n + 31) // 32
    out = {"ep_return_sum": torch.full((n,), -1.0, device="cuda"),
           "ep_count": torch.full((n,), -1, dtype=torch.int32, device="cuda"),
           "totals": torch.zeros(2, dtype=torch.int64, device="cuda"),
           "final_state": torch.zeros(4, n, device="cuda")}
    shapes = {"done_bits": ((T, words), torch.int32), "action_bits": ((T, words), torch.int32),
              "reward_stream": ((T, n), torch.float32), "trajectory": ((T, 4, n), torch.float32)}
    for name in streams:
        out[name] = torch.full(shapes[name][0], 7, dtype=shapes[name][1], device="cuda")
    with kernel(cp, coop, block):
        cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, **kw, **out)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def assert_same_bits(a, b):
    for k in a:
        assert np.array_equal(a[k].view(np.uint32) if a[k].dtype == np.float32 else a[k],
                              b[k].view(np.uint32) if b[k].dtype == np.float32 else b[k]), k


@pytest.mark.parametrize("n", [1, 33, 1000, 4737])
@pytest.mark.parametrize("T", [1, 15, 16, 17, 32, 33, 100])
def test_same_bits_as_general_kernel_and_oracle(cp, oracle, n, T):
    seed, t0, off = 12, 5, 77
    general = rollout(cp, PER_LANE, n, T, seed, t0=t0, env_offset=off)
    for block in (64, 128):                      # one pair and two pairs per CTA (4737 envs: 149 tasks, odd)
        got = rollout(cp, ASSISTED, n, T, seed, block, t0=t0, env_offset=off)
        assert_same_bits(got, general)
    auto = rollout(cp, 0, n, T, seed, t0=t0, env_offset=off)      # what a caller gets
    assert_same_bits(auto, general)
    o = oracle.rollout(n, T, seed, env_offset=off, t0=t0, min_gap=True)
    H.assert_returns_match(auto["ep_return_sum"], auto["ep_count"].view(np.uint32), o["ep_return_sum"],
                           o["ep_count"], excuse=o["min_gap"] < 1e-5,
                           min_identical=0.999 if n >= 1000 else 0.0)
    assert int(auto["totals"][1]) == int(auto["ep_count"].astype(np.int64).sum())


@pytest.mark.parametrize("limit", [0, 30])
def test_contracted_arithmetic_same_bits_as_general_kernel(cp, oracle, limit):
    n, T, seed = 3001, 150, 5
    kw = {"arithmetic": cp.CP_ARITH_CONTRACTED, "max_episode_steps": limit, "t0": 3}
    general = rollout(cp, PER_LANE, n, T, seed, **kw)
    for block in (64, 128):
        assert_same_bits(rollout(cp, ASSISTED, n, T, seed, block, **kw), general)
    auto = rollout(cp, 0, n, T, seed, **kw)
    assert_same_bits(auto, general)
    canonical = rollout(cp, 0, n, T, seed, max_episode_steps=limit, t0=3)
    assert not np.array_equal(auto["final_state"], canonical["final_state"])    # the variant really ran
    o = oracle.rollout(n, T, seed, t0=3, max_episode_steps=limit)
    H.assert_returns_match(auto["ep_return_sum"], auto["ep_count"].view(np.uint32), o["ep_return_sum"], o["ep_count"])


@pytest.mark.parametrize("streams", [("done_bits",), ("reward_stream", "done_bits"),
                                     ("done_bits", "action_bits", "reward_stream", "trajectory")])
@pytest.mark.parametrize("supplied", [False, True])
def test_streams_and_supplied_actions(cp, oracle, streams, supplied):
    n, T, seed, limit = 2101, 70, 8, 40
    words = (n + 31) // 32
    kw, ora_kw = {"t0": 2, "env_offset": 9, "max_episode_steps": limit}, {}
    if supplied:
        rng = np.random.default_rng(5)
        bits = rng.integers(0, 1 << 32, (T, words), dtype=np.uint64).astype(np.uint32)
        kw["action_bits_in"] = torch.from_numpy(bits.view(np.int32)).cuda()
        ora_kw["action_bits_in"] = bits
    general = rollout(cp, PER_LANE, n, T, seed, streams=streams, **kw)
    for block in (64, 128):
        assert_same_bits(rollout(cp, ASSISTED, n, T, seed, block, streams=streams, **kw), general)
    auto = rollout(cp, 0, n, T, seed, streams=streams, **kw)
    assert_same_bits(auto, general)
    o = oracle.rollout(n, T, seed, t0=2, env_offset=9, max_episode_steps=limit, done_bits=True, action_bits=True,
                       min_gap=True, **ora_kw)
    same = (auto["ep_return_sum"] == o["ep_return_sum"]) & (auto["ep_count"].view(np.uint32) == o["ep_count"])
    assert (same | (o["min_gap"] < 1e-5)).mean() >= 0.999
    gd, od = H.unpack_bits(auto["done_bits"], n), H.unpack_bits(o["done_bits"], n)
    assert np.array_equal(gd[:, same], od[:, same])
    if "action_bits" in streams:
        assert np.array_equal(H.unpack_bits(auto["action_bits"], n), H.unpack_bits(o["action_bits"], n))
    if "reward_stream" in streams:
        assert np.all(auto["reward_stream"] == 1.0)
    if "trajectory" in streams:
        assert np.array_equal(auto["trajectory"][-1], auto["final_state"])


def test_forced_on_a_large_batch_and_at_the_end_of_time(cp, oracle):
    """Far more pairs than fit on the chip at once (CTAs in waves), and the last steps the
    32-bit step counter allows (the counter 4 * (t + 1) of the last start state wraps to 0 on
    both sides)."""
    n, T, seed = 300007, 20, 3
    general = rollout(cp, PER_LANE, n, T, seed)
    assert_same_bits(rollout(cp, ASSISTED, n, T, seed), general)
    n, T = 5000, 45
    t0 = (1 << 30) - T
    general = rollout(cp, PER_LANE, n, T, seed, t0=t0, streams=("done_bits",))
    got = rollout(cp, 0, n, T, seed, t0=t0, streams=("done_bits",))
    assert_same_bits(got, general)
    o = oracle.rollout(n, T, seed, t0=t0, done_bits=True, final_state=True)
    H.assert_returns_match(got["ep_return_sum"], got["ep_count"].view(np.uint32), o["ep_return_sum"], o["ep_count"])
    last_done = H.unpack_bits(o["done_bits"], n)[-1].astype(bool)
    assert last_done.sum() > 50     # envs that restart at time 2^30 itself
    assert np.array_equal(got["final_state"][:, last_done], o["final_state"][:, last_done])
    with pytest.raises(cp.CartpoleError):
        rollout(cp, 0, n, T + 1, seed, t0=t0)


def test_callers_state_with_large_angles(cp, oracle):
    """Angles beyond the polynomial range in the initial state (some survive the first step): the
    first hand-over chunk must take the full-range sine and cosine."""
    n, seed, T = 2000, 4, 40
    rng = np.random.default_rng(3)
    z0 = np.stack([rng.uniform(-2, 2, n), rng.uniform(-1, 1, n), rng.uniform(-0.3, 0.3, n),
                   rng.uniform(-3, 3, n)]).astype(np.float32)
    z0[2, :8] = [0.25, -0.25, 0.2201, -0.2201, 0.5, 3.0, -40.0, 0.2199]
    z0[3, :8] = [-3.0, 3.0, -1.0, 1.0, -20.0, 0.0, 0.0, 0.0]
    res = {}
    for coop in (PER_LANE, ASSISTED):
        planes = torch.zeros(4, (n + 3) // 4 * 4, device="cuda")
        planes[:, :n] = torch.from_numpy(z0).cuda()
        st = cp.cp_wrap(planes, n, seed, 9)
        ret = torch.empty(n, device="cuda")
        cnt = torch.empty(n, dtype=torch.int32, device="cuda")
        with kernel(cp, coop):
            cp.cp_rollout_from(st, T, None, None, ep_return_sum=ret, ep_count=cnt)
        torch.cuda.synchronize()
        res[coop] = {"ret": ret.cpu().numpy(), "cnt": cnt.cpu().numpy(), "z": planes[:, :n].cpu().numpy()}
    assert_same_bits(res[ASSISTED], res[PER_LANE])
    o = oracle.rollout(n, T, seed, t0=9, init_state=z0, final_state=True, min_gap=True)
    H.assert_returns_match(res[ASSISTED]["ret"], res[ASSISTED]["cnt"].view(np.uint32), o["ep_return_sum"],
                           o["ep_count"], excuse=o["min_gap"] < 1e-5)
    survived_wide = (np.abs(z0[2]) > 0.22) & (np.abs(z0[2] + np.float32(0.02) * z0[3]) < 0.2)
    assert survived_wide.sum() >= 2        # the case the test is about occurs


def test_step_limit_and_carried_lengths_in_chunks(cp, oracle):
    n, seed, limit = 1500, 21, 25
    whole = oracle.rollout(n, 63, seed, max_episode_steps=limit, final_state=True, min_gap=True)
    res = {}
    for coop in (PER_LANE, ASSISTED):
        st = cp.cp_reset(n, seed)
        ep_len = torch.zeros(n, dtype=torch.int32, device="cuda")
        ret, cnt = np.zeros(n, np.float32), np.zeros(n, np.uint32)
        for T in (7, 16, 40):
            rs = torch.zeros(n, device="cuda")
            ct = torch.zeros(n, dtype=torch.int32, device="cuda")
            with kernel(cp, coop):
                cp.cp_rollout_ex(T=T, state=st, ep_len=ep_len, max_episode_steps=limit, ep_return_sum=rs, ep_count=ct)
            torch.cuda.synchronize()
            ret += rs.cpu().numpy()
            cnt += ct.cpu().numpy().view(np.uint32)
        res[coop] = {"ret": ret, "cnt": cnt, "len": ep_len.cpu().numpy()}
        cp.cp_free(st)
    assert_same_bits(res[ASSISTED], res[PER_LANE])
    H.assert_returns_match(res[ASSISTED]["ret"], res[ASSISTED]["cnt"], whole["ep_return_sum"], whole["ep_count"],
                           excuse=whole["min_gap"] < 1e-5)
    assert res[ASSISTED]["len"].max() < limit
