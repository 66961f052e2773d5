"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle,
element by element on the same seeded inputs, plus GPU-internal identities
(ladder == fused step == rollout, bit for bit)."""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()  # no-op when the in-tree library matches the sources
    binding.lib()  # raises if the library is missing: there is no fallback
    torch.cuda.set_device(0)
    return binding


VEC_MIN_DEFAULT = 262144  # library default of "step_vec_min_envs"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


def alloc_planes(n, stride=None):
    stride = stride or (n + 3) // 4 * 4
    return torch.zeros(4, stride, dtype=torch.float32, device="cuda")


def gpu_step(cp, z, seed, t, action=None, env_offset=0, stride=None, in_place=False, unfused=False):
    n = z.shape[1]
    pin = alloc_planes(n, stride)
    pin[:, :n] = dev(z)
    pout = pin if in_place else alloc_planes(n, stride)
    s_in = cp.cp_wrap(pin, n, seed, t, env_offset)
    s_out = s_in if in_place else cp.cp_wrap(pout, n, seed, 0, 0)
    reward = torch.full((n,), -7.0, dtype=torch.float32, device="cuda")
    done = torch.full((n,), 9, dtype=torch.uint8, device="cuda")
    act = dev(action) if action is not None else None
    if unfused:
        ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")
        cp.cp_step_unfused(s_in, act, s_out, reward, done, ws)
    else:
        cp.cp_step(s_in, act, s_out, reward, done)
    torch.cuda.synchronize()
    info = s_out.info()
    assert info["t"] == t + 1 and info["seed"] == seed and info["env_offset"] == env_offset
    return host(pout[:, :n]), host(reward), host(done)


# ------------------------------------------------------------------ generators
@pytest.mark.parametrize("n,off,t", [(1, 0, 0), (33, 0, 0), (1025, 7, 22), (70001, 1 << 20, 499)])
def test_start_states_and_actions_bit_exact(cp, oracle, n, off, t):
    planes = alloc_planes(n)
    st = cp.cp_wrap(planes, n, seed=3, t=t, env_offset=off)
    cp.cp_fill_start(st)
    a = torch.empty(n, dtype=torch.uint8, device="cuda")
    cp.cp_actions(n, 3, t, off, a)
    torch.cuda.synchronize()
    got = host(planes[:, :n])
    m = min(n, 3000)
    want = oracle.initial_state(m, 3, t, off)
    assert np.array_equal(got[:, :m].view(np.uint32), want.view(np.uint32))
    r = oracle.rollout(n, 1, 3, t0=t, env_offset=off, action_bits=True, per_env=False)
    assert np.array_equal(host(a), H.unpack_bits(r["action_bits"], n)[0])


def test_reset_allocates_and_fills(cp, oracle):
    n = 1000
    st = cp.cp_reset(n, 5)
    info = st.info()
    assert info["n_envs"] == n and info["plane_stride"] % 4 == 0 and info["t"] == 0
    planes = alloc_planes(n)
    out = cp.cp_wrap(planes, n, 5)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    cp.cp_step(st, None, out, reward, done)
    torch.cuda.synchronize()
    z0 = oracle.initial_state(n, 5)
    want = oracle.step(z0, seed=5, t=0, want_pre_reset=True)
    H.assert_step_matches(want, z0, host(planes[:, :n]), host(reward), host(done))
    assert out.info()["t"] == 1
    cp.cp_free(st)


# ------------------------------------------------------------------ single step vs oracle
@pytest.mark.parametrize("spread", ["start", "live", "edge", "wide"])
@pytest.mark.parametrize("n", [1, 3, 5, 33, 1025, 65537])
def test_step_matches_oracle(cp, oracle, spread, n):
    z = inputs.random_states(n, seed=n + len(spread), spread=spread)
    for action, off, t in ((None, 0, 0), (None, 12345, 17), (inputs.random_actions(n, 3), 0, 5)):
        want = oracle.step(z, seed=1, t=t, action_u8=action, env_offset=off, want_pre_reset=True)
        for vec_min in (0, 1 << 30):  # four-envs-per-thread vector kernel, one-env-per-thread kernel
            cp.cp_tune("step_vec_min_envs", vec_min)
            try:
                got_state, got_reward, got_done = gpu_step(cp, z, 1, t, action, off)
            finally:
                cp.cp_tune("step_vec_min_envs", VEC_MIN_DEFAULT)
            stats = H.assert_step_matches(want, z, got_state, got_reward, got_done)
            if spread in ("start", "live") and n >= 1025:
                assert stats["bit_exact_fraction"] > 0.8


def test_step_scalar_path_and_in_place_equal_vector_path(cp):
    n = 4099
    z = inputs.random_states(n, seed=2, spread="edge")
    a = inputs.random_actions(n, 9)
    cp.cp_tune("step_vec_min_envs", 0)  # vector kernel for the aligned layout
    try:
        base = gpu_step(cp, z, 4, 3, None, 100)
        assert all(np.array_equal(b, o) for b, o in zip(base, gpu_step(cp, z, 4, 3, None, 100, in_place=True)))
    finally:
        cp.cp_tune("step_vec_min_envs", VEC_MIN_DEFAULT)
    for kwargs in ({}, {"stride": n}, {"stride": n + 1}, {"in_place": True}, {"stride": n, "in_place": True}):
        other = gpu_step(cp, z, 4, 3, None, 100, **kwargs)
        for b, o in zip(base, other):
            assert np.array_equal(b.view(np.uint8), o.view(np.uint8)), kwargs
    base = gpu_step(cp, z, 4, 3, a, 100)
    other = gpu_step(cp, z, 4, 3, a, 100, stride=n)
    for b, o in zip(base, other):
        assert np.array_equal(b.view(np.uint8), o.view(np.uint8))


def test_step_optional_outputs_and_misaligned_buffers(cp):
    n = 1000
    z = inputs.random_states(n, seed=3, spread="edge")
    want = gpu_step(cp, z, 0, 0)
    pin = alloc_planes(n)
    pin[:, :n] = dev(z)
    s = cp.cp_wrap(pin, n, 0, 0)
    pout = alloc_planes(n)
    o = cp.cp_wrap(pout, n, 0)
    cp.cp_step(s, None, o, None, None)  # reward/done not wanted
    torch.cuda.synchronize()
    assert np.array_equal(host(pout[:, :n]), want[0])
    # reward/done at odd offsets: scalar path, same bits
    rbuf = torch.zeros(n + 1, dtype=torch.float32, device="cuda")
    dbuf = torch.zeros(n + 1, dtype=torch.uint8, device="cuda")
    cp.cp_set_time(s, 0)
    cp.cp_step(s, None, o, rbuf[1:], dbuf[1:])
    torch.cuda.synchronize()
    assert np.array_equal(host(pout[:, :n]), want[0])
    assert np.array_equal(host(rbuf[1:]), want[1]) and np.array_equal(host(dbuf[1:]), want[2])
    assert float(rbuf[0]) == 0 and int(dbuf[0]) == 0


def test_mirror_antisymmetry_on_gpu(cp):
    n = 50000
    z = inputs.random_states(n, seed=6, spread="edge")
    a = inputs.random_actions(n, 6)
    pin, pout = alloc_planes(n), alloc_planes(n)
    res = []
    for zz, aa in ((z, a), (-z, (1 - a).astype(np.uint8))):
        pin[:, :n] = dev(zz)
        s, o = cp.cp_wrap(pin, n, 0, 0), cp.cp_wrap(pout, n, 0)
        done = torch.empty(n, dtype=torch.uint8, device="cuda")
        cp.cp_step(s, dev(aa), o, None, done)
        torch.cuda.synchronize()
        res.append((host(pout[:, :n]), host(done)))
    live = res[0][1] == 0
    assert np.array_equal(res[0][1], res[1][1])
    assert np.array_equal(-res[0][0][:, live], res[1][0][:, live])


def test_nan_inf_states_do_not_fault(cp):
    n = 64
    z = inputs.random_states(n, seed=1, spread="live")
    z[0, 0] = np.nan
    z[2, 1] = np.nan
    z[0, 2] = np.inf
    z[3, 3] = -np.inf
    state, reward, done = gpu_step(cp, z, 0, 0)
    assert done[0] == 0 and done[1] == 0 and done[2] == 1
    assert np.isnan(state[0, 0]) and np.isnan(state[2, 1])
    assert np.all(reward == 1.0)


# ------------------------------------------------------------------ ladder == fused step
@pytest.mark.parametrize("n", [1, 33, 1025, 50001])
def test_ladder_equals_fused_step_bitwise(cp, n):
    cp.cp_tune("step_vec_min_envs", 0 if n % 2 else VEC_MIN_DEFAULT)  # both fused kernels get compared
    before = cp.cp_launch_count()
    for spread in ("edge", "wide", "start"):
        z = inputs.random_states(n, seed=n, spread=spread)
        for action in (None, inputs.random_actions(n, 4)):
            fused = gpu_step(cp, z, 7, 11, action, 5)
            ladder = gpu_step(cp, z, 7, 11, action, 5, unfused=True)
            for f, l in zip(fused, ladder):
                assert np.array_equal(f.view(np.uint8), l.view(np.uint8))
    cp.cp_tune("step_vec_min_envs", VEC_MIN_DEFAULT)
    # 3 spreads x (46 + 45 ladder launches + 2 fused launches)
    assert cp.cp_launch_count() - before == 3 * (46 + 45 + 2)


@pytest.mark.parametrize("n", [1, 4099, 2_000_003])
def test_ladder_chain_with_and_without_dependent_launches(cp, n):
    """Twelve ladder steps back to back (46 launches each, every kernel reading the plane the
    launch before it wrote, the two batches swapping roles after every step) give the bits of
    twelve fused steps — with plain launches and with programmatic dependent launches, where a
    kernel is set up while its predecessor still runs and waits for it itself."""
    T, seed = 12, 4
    a, b = alloc_planes(n), alloc_planes(n)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    ref = alloc_planes(n)
    st = cp.cp_wrap(ref, n, seed)
    cp.cp_fill_start(st)
    cp.cp_step_repeat(st, T, reward, done)
    torch.cuda.synchronize()
    want, want_done = host(ref[:, :n]), host(done)
    try:
        for pdl in (0, 1):
            cp.cp_tune("step_pdl", pdl)
            sa, sb = cp.cp_wrap(a, n, seed), cp.cp_wrap(b, n, seed)
            cp.cp_fill_start(sa)
            done.fill_(7)
            for _ in range(T // 2):
                cp.cp_step_unfused(sa, None, sb, reward, done, ws)
                cp.cp_step_unfused(sb, None, sa, reward, done, ws)
            torch.cuda.synchronize()
            assert sa.info()["t"] == T
            assert np.array_equal(host(a[:, :n]).view(np.uint32), want.view(np.uint32)), pdl
            assert np.array_equal(host(done), want_done), pdl
    finally:
        cp.cp_tune("step_pdl", 1)


def test_ladder_argument_checks(cp):
    n = 100
    pin, pout = alloc_planes(n), alloc_planes(n)
    s, o = cp.cp_wrap(pin, n, 0, 0), cp.cp_wrap(pout, n, 0)
    r = torch.empty(n, dtype=torch.float32, device="cuda")
    d = torch.empty(n, dtype=torch.uint8, device="cuda")
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    with pytest.raises(cp.CartpoleError) as e:
        cp.cp_step_unfused(s, None, s, r, d, ws)
    assert e.value.code == cp.CP_EINVAL
    with pytest.raises(cp.CartpoleError) as e:
        cp.cp_step_unfused(s, None, o, r, d, ws[:1024])
    assert e.value.code == cp.CP_ENOMEM
    with pytest.raises(cp.CartpoleError):
        cp.cp_step_unfused(s, None, o, r, d, ws[1:])
    odd = cp.cp_wrap(torch.zeros(4, 101, device="cuda"), 100, 0, 0)
    with pytest.raises(cp.CartpoleError):
        cp.cp_step_unfused(odd, None, o, r, d, ws)


# ------------------------------------------------------------------ rollout
def run_rollout(cp, n, T, seed, kind=0, weights=None, env_offset=0, streams=False, traj=False, final=True):
    words = (n + 31) // 32
    out = {
        "ep_return_sum": torch.full((n,), -1.0, dtype=torch.float32, device="cuda"),
        "ep_count": torch.full((n,), -1, dtype=torch.int32, device="cuda"),
        "totals": torch.zeros(2, dtype=torch.int64, device="cuda"),
    }
    if final:
        out["final_state"] = torch.zeros(4, n, dtype=torch.float32, device="cuda")
    if streams:
        out["reward_stream"] = torch.zeros(T, n, dtype=torch.float32, device="cuda")
        out["done_bits"] = torch.zeros(T, words, dtype=torch.int32, device="cuda")
        if streams != "reward+done":
            out["action_bits"] = torch.zeros(T, words, dtype=torch.int32, device="cuda")
    if traj:
        out["trajectory"] = torch.zeros(T, 4, n, dtype=torch.float32, device="cuda")
    pol = cp.policy(kind, weights) if kind else None
    cp.cp_rollout_shard(env_offset, n, T, seed, pol, **out)
    torch.cuda.synchronize()
    res = {k: host(v) for k, v in out.items()}
    res["ep_count"] = res["ep_count"].view(np.uint32)
    res["totals"] = res["totals"].view(np.uint64)
    return res


@pytest.mark.parametrize("n,T", [(1, 64), (33, 64), (1025, 100), (5000, 37)])
@pytest.mark.parametrize("shape", H.SHAPES)
def test_rollout_equals_repeated_fused_steps_bitwise(cp, n, T, shape):
    seed, off = 2, 77
    with H.rollout_shape(cp, *shape):
        r = run_rollout(cp, n, T, seed, env_offset=off, streams=True, traj=True)
    planes = alloc_planes(n)
    st = cp.cp_wrap(planes, n, seed, 0, off)
    cp.cp_fill_start(st)
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    act = torch.empty(n, dtype=torch.uint8, device="cuda")
    db, ab = H.unpack_bits(r["done_bits"], n), H.unpack_bits(r["action_bits"], n)
    ep_len = np.zeros(n, np.int64)
    ret = np.zeros(n, np.int64)
    cnt = np.zeros(n, np.int64)
    for t in range(T):
        cp.cp_actions(n, seed, t, off, act)
        cp.cp_step(st, None, st, reward, done)
        torch.cuda.synchronize()
        assert np.array_equal(host(planes[:, :n]).view(np.uint32), r["trajectory"][t].view(np.uint32)), t
        d = host(done)
        assert np.array_equal(d, db[t]) and np.array_equal(host(act), ab[t])
        ep_len += 1
        m = d.astype(bool)
        ret[m] += ep_len[m]
        cnt[m] += 1
        ep_len[m] = 0
    assert np.array_equal(r["final_state"], r["trajectory"][-1])
    assert np.array_equal(r["ep_return_sum"], ret.astype(np.float32))
    assert np.array_equal(r["ep_count"], cnt.astype(np.uint32))
    assert np.all(r["reward_stream"] == 1.0)
    assert int(r["totals"][0]) == ret.sum() and int(r["totals"][1]) == cnt.sum()
    # padding bits of the last mask word stay zero
    if n % 32:
        assert not np.any(r["done_bits"].view(np.uint32)[:, -1] >> (n % 32))


def test_config1_full_trajectory_against_oracle(cp, oracle):
    """1,024 envs x 200 steps, seed 0. The oracle's own trajectory is the reference throughout
    (no oracle input ever comes from the GPU): (i) teacher-forced — at every step the GPU steps
    the oracle's state and must reproduce the oracle's next state (<= 2e-6), action, reward and
    done flag (bit-exact outside the 1e-5 threshold band); (ii) free-running — the GPU rollout's
    trajectory, action and done streams against the oracle's, and the per-env returns."""
    w = inputs.WORKLOADS["c1"]
    n, T = w.n_envs, w.T
    o = oracle.rollout(n, T, w.seed, trajectory=True, done_bits=True, action_bits=True)
    od, oa = H.unpack_bits(o["done_bits"], n), H.unpack_bits(o["action_bits"], n)
    # (i) teacher-forced on the oracle's states
    planes_in, planes_out = alloc_planes(n), alloc_planes(n)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    act = torch.empty(n, dtype=torch.uint8, device="cuda")
    z = oracle.initial_state(n, w.seed)
    flips = band = 0
    for t in range(T):
        want = oracle.step(z, seed=w.seed, t=t, want_pre_reset=True)
        assert np.array_equal(want["state"], o["trajectory"][t]) and np.array_equal(want["done"], od[t])
        planes_in[:, :n] = dev(z)
        s_in, s_out = cp.cp_wrap(planes_in, n, w.seed, t), cp.cp_wrap(planes_out, n, w.seed)
        cp.cp_step(s_in, None, s_out, reward, done)
        cp.cp_actions(n, w.seed, t, 0, act)
        torch.cuda.synchronize()
        st = H.assert_step_matches(want, z, host(planes_out[:, :n]), host(reward), host(done), host(act))
        flips += st["done_flips"]
        band += st["band"]
        z = o["trajectory"][t]
    assert flips <= band
    # (ii) free-running rollout
    r = run_rollout(cp, n, T, w.seed, streams=True, traj=True)
    gd, ga = H.unpack_bits(r["done_bits"], n), H.unpack_bits(r["action_bits"], n)
    assert np.array_equal(ga, oa)  # hashed actions do not depend on the state
    assert np.all(r["reward_stream"] == 1.0)
    same = (gd == od).all(axis=0)
    assert same.mean() >= 0.999
    # where the done streams agree the trajectories stay together (restarts re-synchronise them)
    err = np.abs(r["trajectory"][:, :, same] - o["trajectory"][:, :, same]).max()
    assert err < 1e-4, err
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"])


@pytest.mark.parametrize("name", ["c3"])
def test_full_size_random_rollout_against_oracle(cp, oracle, name):
    """1,048,576 envs x 500 steps in the benchmark's launch configuration; the oracle runs the
    whole workload on all host cores."""
    import os
    w = inputs.WORKLOADS[name]
    r = run_rollout(cp, w.n_envs, w.T, w.seed, final=False)
    o = oracle.rollout(w.n_envs, w.T, w.seed, nthreads=os.cpu_count() or 1)
    s = H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"])
    assert int(r["totals"][0]) == int(r["ep_return_sum"].astype(np.int64).sum())
    assert int(r["totals"][1]) == int(r["ep_count"].astype(np.int64).sum())
    assert 21.5 < s["mean_gpu"] < 22.5


@pytest.mark.parametrize("kind,pseed,n,T", [(1, 1, 40000, 300), (2, 2, 40000, 200), (1, 5, 3001, 150), (2, 6, 3001, 150)])
def test_policy_rollouts_against_oracle(cp, oracle, kind, pseed, n, T):
    wts = inputs.policy_weights(kind, pseed)
    r = run_rollout(cp, n, T, 0, kind, wts, streams=True)
    o = oracle.rollout(n, T, 0, kind, wts, action_bits=True, done_bits=True, min_gap=True, nthreads=4)
    excuse = o["min_gap"] < 1e-5
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"], excuse)
    # until an env's first divergence its action and done streams are identical; most never diverge
    same_env = (r["ep_return_sum"] == o["ep_return_sum"])
    ga, oa = H.unpack_bits(r["action_bits"], n), H.unpack_bits(o["action_bits"], n)
    gd, od = H.unpack_bits(r["done_bits"], n), H.unpack_bits(o["done_bits"], n)
    agree = (ga == oa).all(axis=0) & (gd == od).all(axis=0)
    assert agree.mean() >= 0.995
    assert np.array_equal(gd.sum(axis=0), r["ep_count"])


@pytest.mark.parametrize("name", ["c4", "c5"])
def test_full_size_policy_configs_against_oracle(cp, oracle, name):
    """Configs 4 (4,194,304 x 1,000, linear policy, reward plane + done bitmask) and 5
    (16,777,216 x 200, MLP policy) exactly as bench.py launches them. The oracle recomputes the
    first 1,048,576 environments for all T steps, a range in the middle and the last 4,992 (results of
    an env do not depend on its neighbours): returns identical on >= 99.9 % of the envs that stayed
    1e-5 clear of every logit tie and termination threshold, and so is the whole done bit stream."""
    import os
    w = inputs.WORKLOADS[name]
    wts = inputs.policy_weights(w.policy, w.policy_seed)
    n, T = w.n_envs, w.T
    words = (n + 31) // 32
    outs = {"ep_return_sum": torch.empty(n, dtype=torch.float32, device="cuda"),
            "ep_count": torch.empty(n, dtype=torch.int32, device="cuda"),
            "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
    if w.streams:
        outs["reward_stream"] = torch.empty(T, n, dtype=torch.float32, device="cuda")
        outs["done_bits"] = torch.empty(T, words, dtype=torch.int32, device="cuda")
    cp.cp_rollout(n, T, w.seed, cp.policy(w.policy, wts), **outs)
    torch.cuda.synchronize()
    ret, cnt = host(outs["ep_return_sum"]), host(outs["ep_count"]).view(np.uint32)
    cores = os.cpu_count() or 1
    for lo, m in ((0, 1 << 20), (n // 2 - 1024, 2048), (n - 4992, 4992)):
        o = oracle.rollout(m, T, w.seed, w.policy, wts, env_offset=lo, min_gap=True, min_margin=True,
                           done_bits=w.streams, nthreads=cores)
        excuse = (o["min_gap"] < 1e-5) | (o["min_margin"] < 1e-5)
        H.assert_returns_match(ret[lo:lo + m], cnt[lo:lo + m], o["ep_return_sum"], o["ep_count"], excuse,
                               min_identical=0.999)
        if w.streams:
            gd = host(outs["done_bits"][:, lo // 32:(lo + m) // 32]).view(np.uint32)
            # the whole done bit stream, step by step: identical on >= 99.9 % of the envs that stayed
            # clear of the bands (under a feedback policy a last-bit sine difference can grow past
            # 1e-5 within an 80-step episode; measured: 132 of 1,048,576 such envs differ somewhere)
            diff = np.bitwise_or.reduce(gd ^ o["done_bits"], axis=0)
            differs = np.unpackbits(diff.view(np.uint8), bitorder="little").astype(bool)
            assert int((differs & ~excuse).sum()) <= m // 1000
            pop = np.zeros(m, np.int64)
            for k in range(32):                                       # done bits per env == its episode count
                pop[k::32] = ((gd >> np.uint32(k)) & np.uint32(1)).sum(axis=0)
            assert np.array_equal(pop, cnt[lo:lo + m])
            assert bool((outs["reward_stream"][:, lo:lo + min(m, 65536)] == 1.0).all())
    tot = host(outs["totals"]).view(np.uint64)
    assert int(tot[1]) == int(cnt.astype(np.int64).sum())
    assert int(tot[0]) == int(ret.astype(np.float64).sum())
    if w.streams:  # every row of the reward plane was written
        assert float(outs["reward_stream"].min()) == 1.0 and float(outs["reward_stream"].max()) == 1.0
    del outs
    torch.cuda.empty_cache()


def test_config2_step_path_at_full_size(cp, oracle):
    """65,536 envs x 1,000 steps through per-step launches (state round-trips HBM every step):
    equal to the one-launch rollout bit for bit, whose returns are checked against the oracle;
    and the per-op ladder equals the fused step over 20 consecutive steps at this size."""
    import os
    w = inputs.WORKLOADS["c2"]
    n, T = w.n_envs, w.T
    roll = run_rollout(cp, n, T, w.seed)
    planes = alloc_planes(n)
    st = cp.cp_wrap(planes, n, w.seed)
    cp.cp_fill_start(st)
    reward = torch.empty(n, dtype=torch.float32, device="cuda")
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    done_count = torch.zeros(n, dtype=torch.int32, device="cuda")
    for _ in range(T // 100):
        for _ in range(100):
            cp.cp_step(st, None, st, reward, done)
            done_count += done  # torch only accumulates the library's output for the comparison
    torch.cuda.synchronize()
    assert np.array_equal(host(planes[:, :n]), roll["final_state"])
    assert np.array_equal(host(done_count).view(np.uint32), roll["ep_count"])
    o = oracle.rollout(n, T, w.seed, nthreads=os.cpu_count() or 1)
    H.assert_returns_match(roll["ep_return_sum"], roll["ep_count"], o["ep_return_sum"], o["ep_count"])
    # ladder vs fused step, 20 steps, ping-pong
    a, b, c = alloc_planes(n), alloc_planes(n), alloc_planes(n)
    sa, sb, sc = cp.cp_wrap(a, n, w.seed), cp.cp_wrap(b, n, w.seed), cp.cp_wrap(c, n, w.seed)
    cp.cp_fill_start(sa)
    c.copy_(a)
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    done2 = torch.empty_like(done)
    for k in range(10):
        cp.cp_step_unfused(sa, None, sb, reward, done, ws)
        cp.cp_step_unfused(sb, None, sa, reward, done, ws)
        cp.cp_step(sc, None, sc, reward, done2)
        cp.cp_step(sc, None, sc, reward, done2)
    torch.cuda.synchronize()
    assert torch.equal(a, c) and torch.equal(done, done2)
    assert sa.info()["t"] == 20 == sc.info()["t"]


@pytest.mark.parametrize("shape", H.SHAPES)
def test_reward_and_done_only_streams_equal_the_general_stream_kernel(cp, shape):
    """The reward-plane + done-bitmask combination has a kernel of its own."""
    with H.rollout_shape(cp, *shape):
        for n, T, kind in ((5001, 60, 0), (40000, 40, 1), (33, 20, 2)):
            w = inputs.policy_weights(kind, 3) if kind else None
            a = run_rollout(cp, n, T, 2, kind, w, env_offset=9, streams=True)
            b = run_rollout(cp, n, T, 2, kind, w, env_offset=9, streams="reward+done")
            for k in ("ep_return_sum", "ep_count", "totals", "final_state", "reward_stream", "done_bits"):
                assert np.array_equal(a[k], b[k]), (k, n, kind)
            assert np.all(b["reward_stream"] == 1.0)
            assert np.array_equal(H.unpack_bits(b["done_bits"], n).sum(axis=0), b["ep_count"])


def test_work_shapes_agree_bitwise_and_survive_mass_termination(cp):
    """The three work shapes (per-lane restarts, restarts by the warp with one or two envs per
    thread) give the same bits, including when far more environments of a warp finish in one
    step than the warp's restart list holds: with an episode limit of 1 every env restarts every
    step, with 3 all of them at once every third step."""
    n, T = 5003, 31
    for kind, limit in ((0, 0), (0, 1), (0, 3), (1, 2), (2, 0)):
        w = inputs.policy_weights(kind, 3) if kind else None
        pol = cp.policy(kind, w) if kind else None
        results = []
        for shape in H.SHAPES:
            out = {"ep_return_sum": torch.zeros(n, device="cuda"),
                   "ep_count": torch.zeros(n, dtype=torch.int32, device="cuda"),
                   "totals": torch.zeros(2, dtype=torch.int64, device="cuda"),
                   "final_state": torch.zeros(4, n, device="cuda"),
                   "done_bits": torch.zeros(T, (n + 31) // 32, dtype=torch.int32, device="cuda"),
                   "trajectory": torch.zeros(T, 4, n, device="cuda")}
            with H.rollout_shape(cp, *shape):
                cp.cp_rollout_ex(n_envs=n, T=T, seed=6, env_offset=11, policy=pol, max_episode_steps=limit, **out)
            torch.cuda.synchronize()
            results.append({k: host(v) for k, v in out.items()})
        for other in results[1:]:
            for k in results[0]:
                assert np.array_equal(results[0][k].view(np.uint32) if results[0][k].dtype == np.float32 else results[0][k],
                                      other[k].view(np.uint32) if other[k].dtype == np.float32 else other[k]), (k, kind, limit)
        if limit == 1:
            assert np.all(results[0]["ep_count"] == T) and np.all(results[0]["ep_return_sum"] == T)


def test_launch_geometry_does_not_change_results(cp):
    """Persistent grids (warps looping over several tasks, re-using their shared-memory restart
    list), small CTAs and every work shape give the bits of the default launch."""
    n, T = 70001, 45
    want = run_rollout(cp, n, T, 7, streams=True)
    try:
        for per_sm, block in ((1, 256), (2, 64), (1, 32), (0, 96)):
            cp.cp_tune("rollout_ctas_per_sm", per_sm)
            cp.cp_tune("rollout_block", block)
            for shape in H.SHAPES:
                with H.rollout_shape(cp, *shape):
                    got = run_rollout(cp, n, T, 7, streams=True)
                for k in want:
                    assert np.array_equal(want[k], got[k]), (k, per_sm, block, shape)
    finally:
        cp.cp_tune("rollout_ctas_per_sm", 0)
        cp.cp_tune("rollout_block", 0)


def test_shards_compose(cp):
    n, T = 10000, 80
    whole = run_rollout(cp, n, T, 3)
    tot = np.zeros(2, np.uint64)
    for rank in range(3):
        lo, hi = inputs.shard_range(n, rank, 3)
        part = run_rollout(cp, hi - lo, T, 3, env_offset=lo)
        assert np.array_equal(part["ep_return_sum"], whole["ep_return_sum"][lo:hi])
        assert np.array_equal(part["final_state"], whole["final_state"][:, lo:hi])
        tot += part["totals"]
    assert np.array_equal(tot, whole["totals"])


def test_chunked_rollout_from_state(cp):
    n, seed = 3000, 8
    whole = run_rollout(cp, n, 90, seed)
    st = cp.cp_reset(n, seed)
    ep_len = torch.zeros(n, dtype=torch.int32, device="cuda")
    ret = np.zeros(n, np.float32)
    cnt = np.zeros(n, np.uint32)
    tot = torch.zeros(2, dtype=torch.int64, device="cuda")
    for T in (1, 29, 60):
        rs = torch.zeros(n, dtype=torch.float32, device="cuda")
        ct = torch.zeros(n, dtype=torch.int32, device="cuda")
        cp.cp_rollout_from(st, T, ep_len, None, ep_return_sum=rs, ep_count=ct, totals=tot)
        torch.cuda.synchronize()
        ret += host(rs)
        cnt += host(ct).view(np.uint32)
    assert st.info()["t"] == 90
    assert np.array_equal(ret, whole["ep_return_sum"]) and np.array_equal(cnt, whole["ep_count"])
    assert np.array_equal(host(tot).view(np.uint64), whole["totals"])
    # the batch itself now holds the final state: one more fused step equals step 91 of a longer rollout
    longer = run_rollout(cp, n, 91, seed)
    planes = alloc_planes(n)
    o = cp.cp_wrap(planes, n, seed)
    cp.cp_step(st, None, o, None, None)
    torch.cuda.synchronize()
    assert np.array_equal(host(planes[:, :n]), longer["final_state"])


def test_step_repeat_and_graph_replay_equal_rollout(cp):
    n, T, seed = 3000, 50, 6
    ref = run_rollout(cp, n, T, seed, streams=True)
    planes = alloc_planes(n)
    st = cp.cp_wrap(planes, n, seed)
    cp.cp_fill_start(st)
    reward = torch.zeros(n, dtype=torch.float32, device="cuda")
    done = torch.zeros(n, dtype=torch.uint8, device="cuda")
    for pdl in (0, 1):  # plain launches, then programmatic dependent launches (the default)
        cp.cp_tune("step_pdl", pdl)
        cp.cp_set_time(st, 0)
        cp.cp_fill_start(st)
        cp.cp_step_repeat(st, T, reward, done)
        torch.cuda.synchronize()
        assert st.info()["t"] == T
        assert np.array_equal(host(planes[:, :n]), ref["final_state"])
        assert np.array_equal(host(done), H.unpack_bits(ref["done_bits"], n)[-1])
    # the same T launches captured in a CUDA graph and replayed from the start states
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        cp.cp_set_time(st, 0)
        cp.cp_step_repeat(st, 2, reward, done)  # warm-up outside the capture
        side.synchronize()
        cp.cp_set_time(st, 0)
        with torch.cuda.graph(g, stream=side):
            cp.cp_step_repeat(st, T, reward, done)
    cp.cp_set_time(st, 0)
    cp.cp_fill_start(st)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    assert np.array_equal(host(planes[:, :n]), ref["final_state"])
    with pytest.raises(cp.CartpoleError):
        cp.cp_step_repeat(st, -1, None, None)


def test_host_buffer_entry_points(cp, oracle):
    n, T = 5000, 60
    wts = inputs.policy_weights(1, 1)
    for kind, w in ((0, None), (1, wts)):
        ref = run_rollout(cp, n, T, 4, kind, w)
        # page-locked buffers (written by the kernel directly) and pageable ones (staged copy)
        for pin in (True, False):
            h_ret = torch.full((n,), -1.0, dtype=torch.float32)
            h_cnt = torch.full((n,), -1, dtype=torch.int32)
            h_tot = torch.full((2,), -1, dtype=torch.int64)
            if pin:
                h_ret, h_cnt, h_tot = h_ret.pin_memory(), h_cnt.pin_memory(), h_tot.pin_memory()
            cp.cp_rollout_host(n, T, 4, cp.policy(kind, w) if kind else None, h_ret, h_cnt, h_tot)
            assert np.array_equal(h_ret.numpy(), ref["ep_return_sum"])
            assert np.array_equal(h_cnt.numpy().view(np.uint32), ref["ep_count"])
            assert np.array_equal(h_tot.numpy().view(np.uint64), ref["totals"])
    z = inputs.random_states(n, seed=1, spread="edge")
    a = inputs.random_actions(n, 2)
    for action in (None, a):
        want = gpu_step(cp, z, 9, 4, action)
        out, rew, dn = np.empty_like(z), np.empty(n, np.float32), np.empty(n, np.uint8)
        cp.cp_step_host(n, 9, 4, z, action, out, rew, dn)
        assert np.array_equal(out, want[0]) and np.array_equal(rew, want[1]) and np.array_equal(dn, want[2])
    cp.cp_shutdown()


def test_fused_sincos_equals_separate_sin_and_cos(cp):
    bad = torch.zeros(1, dtype=torch.int64, device="cuda")
    f = lambda v: int(np.float32(v).view(np.uint32))
    cp.cp_selftest_sincos(0, f(0.35), bad)           # every float the episodes can reach
    cp.cp_selftest_sincos(f(0.35), f(200.0), bad)    # every float up to 200 rad
    cp.cp_selftest_sincos(f(1e5), f(1.2e5), bad)     # across the switch to the large-argument path
    cp.cp_selftest_sincos(f(1e30), f(1.0001e30), bad)
    torch.cuda.synchronize()
    assert int(bad[0]) == 0


def test_sincos_accuracy_over_every_reachable_angle(cp):
    """Every float32 in [0, 0.22] (sin is odd, cos even): error against float64 below 0.54 ulp,
    i.e. tighter than the 1-ulp bound of library sinf/cosf; beyond 0.22 the library routines."""
    f = lambda v: int(np.float32(v).view(np.uint32))
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    cp.cp_selftest_sincos_accuracy(0, f(0.22), out)
    torch.cuda.synchronize()
    max_sin, max_cos, ncr_sin, ncr_cos = (int(v) for v in out.cpu())
    total = f(0.22) + 1
    print(f"sin/cos over [0, 0.22]: max error {max_sin / 1e6:.4f} / {max_cos / 1e6:.4f} ulp, "
          f"not correctly rounded {ncr_sin / total:.5f} / {ncr_cos / total:.5f} of {total} floats")
    assert max_sin <= 540_000 and max_cos <= 540_000, (max_sin, max_cos)
    assert ncr_sin / total < 0.05 and ncr_cos / total < 0.05, (ncr_sin, ncr_cos, total)
    out.zero_()
    cp.cp_selftest_sincos_accuracy(f(0.22) + 1, f(8.0), out)
    torch.cuda.synchronize()
    assert int(out[0]) <= 1_500_000 and int(out[1]) <= 1_500_000  # library routines: about 1 ulp


def test_exact_shortcuts_equal_the_operations_they_replace(cp):
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    cp.cp_selftest_arith(out)
    torch.cuda.synchronize()
    assert [int(v) for v in out.cpu()] == [0, 0, 0, 0]


def test_packed_two_env_step_has_the_bits_of_the_scalar_step(cp):
    """2^30 pseudo-random state pairs through the packed float32 instructions and through the scalar
    step (which the ladder tests tie to the one-op kernels): no bit may differ. Guards against an
    assembler that contracts a packed multiply and add (CUDA 12.9 does where it can)."""
    out = torch.zeros(3, dtype=torch.int64, device="cuda")
    for seed in (0, 1):
        cp.cp_selftest_pair(1 << 29, seed, out)
    torch.cuda.synchronize()
    bad, pairs, bad_contracted = (int(v) for v in out.cpu())
    assert pairs == 1 << 30
    assert bad == 0 and bad_contracted == 0


def test_tame_state_division_equals_ieee_division_on_its_whole_domain(cp):
    """53,688 denominators x 33,554,432 numerators x both signs, every pair (about 2 s)."""
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    cp.cp_selftest_tame_div(1, out)
    torch.cuda.synchronize()
    bad, pairs = (int(v) for v in out.cpu())
    lo, hi = (int(np.float32(v).view(np.uint32)) for v in (0.6210, 0.6242))
    assert pairs == (hi - lo + 1) * (1 << 25)
    assert bad == 0
    # the domain really contains what a tame state produces: den at c = 1 and c = cos(0.25), |num| bounds
    m, ft = np.float32(1.1), np.float32(4.0 / 3.0)
    for c in (np.float32(1.0), np.float32(np.cos(0.25)) - np.float32(1e-6)):
        den = np.float32(0.5) * (ft - (np.float32(0.1) * (c * c)) / m)
        assert 0.6210 < float(den) < 0.6242
    # a state in the tame lane (|theta| <= 0.22) that survives its step has |theta_dot| < 21.5:
    # |t2| <= 0.05 * 21.5^2 * sin(0.22), t3 = +-10 + t2, num = 9.8 s - c t3 / 1.1
    s_max, c_min = np.sin(0.22), np.cos(0.22)
    t2 = 0.05 * 21.5 ** 2 * s_max
    assert (0.2095 + 0.22) / 0.02 < 21.5
    assert c_min * (10 - t2) / 1.1 - 9.8 * s_max > 2.0 and 9.8 * s_max + (10 + t2) / 1.1 < 32.0


def test_stream_selection(cp):
    n, T = 2000, 30
    ref = run_rollout(cp, n, T, 1)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        got = run_rollout(cp, n, T, 1)
    assert np.array_equal(ref["ep_return_sum"], got["ep_return_sum"])
