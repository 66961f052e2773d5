"""GPU parity tests of the optional behaviours of the general rollout / step calls: the
episode step limit and actions supplied as a packed bit stream, against the CPU oracle and
against the library's own basic paths."""
import ctypes as C

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
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def host(t):
    return t.cpu().numpy()


def outputs(n, T, streams=True, final=True):
    words = (n + 31) // 32
    out = {"ep_return_sum": torch.full((n,), -1.0, dtype=torch.float32, device="cuda"),
           "ep_count": torch.full((n,), -1, dtype=torch.int32, device="cuda"),
           "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
    if final:
        out["final_state"] = torch.zeros(4, n, dtype=torch.float32, device="cuda")
    if streams:
        out["done_bits"] = torch.zeros(T, words, dtype=torch.int32, device="cuda")
        out["action_bits"] = torch.zeros(T, words, dtype=torch.int32, device="cuda")
    return out


def fetch(out):
    torch.cuda.synchronize()
    r = {k: host(v) for k, v in out.items()}
    r["ep_count"] = r["ep_count"].view(np.uint32)
    r["totals"] = r["totals"].view(np.uint64)
    return r


def pack_bits(bits):
    T, n = bits.shape
    words = (n + 31) // 32
    padded = np.zeros((T, words * 32), np.uint8)
    padded[:, :n] = bits
    return np.packbits(padded, axis=1, bitorder="little").view(np.uint32).reshape(T, words)


@pytest.mark.parametrize("limit", [1, 7, 50])
@pytest.mark.parametrize("kind", [0, 1])
def test_limited_rollout_against_oracle(cp, oracle, limit, kind):
    n, T, seed, off = 5003, 120, 3, 64
    w = inputs.policy_weights(kind, 4) if kind else None
    out = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, policy=cp.policy(kind, w) if kind else None,
                     max_episode_steps=limit, **out)
    r = fetch(out)
    o = oracle.rollout(n, T, seed, kind, w, env_offset=off, max_episode_steps=limit, done_bits=True,
                       min_gap=True, nthreads=4)
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"],
                           o["min_gap"] < 1e-5)
    gd, od = H.unpack_bits(r["done_bits"], n), H.unpack_bits(o["done_bits"], n)
    same = r["ep_return_sum"] == o["ep_return_sum"]
    assert same.mean() > 0.999
    assert np.array_equal(gd[:, same], od[:, same])
    # no episode outlives the limit
    for i in range(0, n, 97):
        times = np.concatenate(([-1], np.nonzero(gd[:, i])[0]))
        assert np.diff(times).max(initial=0) <= limit and T - 1 - times[-1] < limit
    if limit == 1:
        assert np.all(r["ep_count"] == T) and np.all(r["ep_return_sum"] == T)
    assert int(r["totals"][1]) == int(r["ep_count"].astype(np.int64).sum())


def test_limit_that_is_never_reached_changes_nothing(cp):
    n, T = 4000, 80
    a, b = outputs(n, T), outputs(n, T)
    cp.cp_rollout(n, T, 5, None, **a)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=5, max_episode_steps=T + 1, **b)
    ra, rb = fetch(a), fetch(b)
    for k in ra:
        assert np.array_equal(ra[k], rb[k]), k


def test_step_ex_equals_limited_rollout_and_chunks_resume(cp, oracle):
    n, T, seed, limit = 3001, 60, 2, 9
    whole = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, max_episode_steps=limit, **whole)
    rw = fetch(whole)
    gd = H.unpack_bits(rw["done_bits"], n)
    for vec_min in (0, 1 << 30):  # vector and scalar step kernels
        cp.cp_tune("step_vec_min_envs", vec_min)
        try:
            planes = torch.zeros(4, (n + 3) // 4 * 4, device="cuda")
            st = cp.cp_wrap(planes, n, seed)
            cp.cp_fill_start(st)
            ep_len = torch.zeros(n, dtype=torch.int32, device="cuda")
            reward = torch.empty(n, device="cuda")
            done = torch.empty(n, dtype=torch.uint8, device="cuda")
            for t in range(T):
                cp.cp_step_ex(st, None, st, reward, done, ep_len, limit)
                torch.cuda.synchronize()
                assert np.array_equal(host(done), gd[t]), t
                assert int(ep_len.max()) < limit
            assert np.array_equal(host(planes[:, :n]), rw["final_state"])
        finally:
            cp.cp_tune("step_vec_min_envs", 262144)
    # the same rollout in three chunks on a batch, episode lengths carried between chunks
    st = cp.cp_reset(n, seed)
    ep_len = torch.zeros(n, dtype=torch.int32, device="cuda")
    ret = np.zeros(n, np.float32)
    cnt = np.zeros(n, np.uint32)
    for chunk in (13, 1, 46):
        o = outputs(n, chunk, streams=False, final=False)
        cp.cp_rollout_ex(T=chunk, state=st, ep_len=ep_len, max_episode_steps=limit, **o)
        r = fetch(o)
        ret += r["ep_return_sum"]
        cnt += r["ep_count"]
    assert st.info()["t"] == T
    assert np.array_equal(ret, rw["ep_return_sum"]) and np.array_equal(cnt, rw["ep_count"])
    tail = np.array([T - 1 - np.max(np.nonzero(gd[:, i])[0], initial=-1) for i in range(n)], np.uint32)
    assert np.array_equal(host(ep_len).view(np.uint32), tail)
    # one more limited step from the ORACLE's state and counters: GPU step vs oracle step
    o = oracle.rollout(n, T, seed, max_episode_steps=limit, final_state=True, ep_len=np.zeros(n, np.uint32))
    want = oracle.step_limited(o["final_state"], seed, T, o["ep_len"], limit)
    planes_in = torch.zeros(4, (n + 3) // 4 * 4, device="cuda")
    planes_in[:, :n] = torch.from_numpy(o["final_state"]).cuda()
    planes = torch.zeros_like(planes_in)
    s_in, out_state = cp.cp_wrap(planes_in, n, seed, T), cp.cp_wrap(planes, n, seed)
    d_len = torch.from_numpy(o["ep_len"].view(np.int32)).cuda()
    done = torch.empty(n, dtype=torch.uint8, device="cuda")
    cp.cp_step_ex(s_in, None, out_state, None, done, d_len, limit)
    torch.cuda.synchronize()
    agree = host(done) == want["done"]
    assert agree.mean() > 0.999
    assert np.array_equal(host(d_len).view(np.uint32)[agree], want["ep_len"][agree])
    assert np.allclose(host(planes[:, :n])[:, agree], want["state"][:, agree], rtol=0, atol=2e-6)


def test_supplied_action_stream(cp, oracle):
    n, T, seed, off = 4099, 70, 8, 32
    rng = np.random.default_rng(1)
    acts = rng.integers(0, 2, (T, n)).astype(np.uint8)
    bits = pack_bits(acts)
    bits[:, -1] |= np.uint32((0xFFFFFFFF << (n % 32)) & 0xFFFFFFFF)  # garbage in the padding bits
    d_bits = torch.from_numpy(bits.view(np.int32)).cuda()
    for shape in H.SHAPES:
        with H.rollout_shape(cp, *shape):
            out = outputs(n, T)
            cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, action_bits_in=d_bits, **out)
            r = fetch(out)
        o = oracle.rollout(n, T, seed, env_offset=off, action_bits_in=pack_bits(acts), done_bits=True, nthreads=4)
        H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"])
        assert np.array_equal(H.unpack_bits(r["action_bits"], n), acts)  # echoed, padding masked off
        same = r["ep_return_sum"] == o["ep_return_sum"]
        assert np.array_equal(H.unpack_bits(r["done_bits"], n)[:, same], H.unpack_bits(o["done_bits"], n)[:, same])
    # a supplied stream overrides a policy
    w = inputs.policy_weights(1, 1)
    out2 = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, policy=cp.policy(1, w), action_bits_in=d_bits, **out2)
    r2 = fetch(out2)
    assert np.array_equal(r2["ep_return_sum"], r["ep_return_sum"]) and np.array_equal(r2["final_state"], r["final_state"])
    # feeding the hashed actions back in reproduces the random-policy rollout bit for bit
    a = outputs(n, T)
    cp.cp_rollout_shard(off, n, T, seed, None, **a)
    ra = fetch(a)
    b = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, action_bits_in=a["action_bits"], **b)
    rb = fetch(b)
    for k in ra:
        assert np.array_equal(ra[k], rb[k]), k


def test_long_horizons_and_late_global_times(cp, oracle):
    """Few environments for very many steps, and a rollout that ends at the largest global time the
    hash counters allow (t0 + T = 2^30): the 32-bit time arithmetic agrees with the oracle's."""
    n, T = 64, 200_000
    out = outputs(n, T, streams=False)
    cp.cp_rollout(n, T, 7, None, **out)
    r = fetch(out)
    o = oracle.rollout(n, T, 7, final_state=True, nthreads=4)
    assert (r["ep_return_sum"] == o["ep_return_sum"]).mean() >= 0.95  # 64 envs x 200,000 steps: a flip or two
    assert abs(float(r["ep_return_sum"].sum()) - float(o["ep_return_sum"].sum())) <= 200
    assert r["ep_return_sum"].max() <= T and r["ep_return_sum"].min() > T - 500
    n, T = 3000, 500
    t0 = (1 << 30) - T
    out = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=9, t0=t0, max_episode_steps=40, **out)
    r = fetch(out)
    o = oracle.rollout(n, T, 9, t0=t0, max_episode_steps=40, done_bits=True, action_bits=True)
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"])
    assert np.array_equal(H.unpack_bits(r["action_bits"], n), H.unpack_bits(o["action_bits"], n))
    with pytest.raises(cp.CartpoleError):
        cp.cp_rollout_ex(n_envs=n, T=T + 1, seed=9, t0=t0, **outputs(n, T + 1, streams=False))


def test_general_call_argument_checks(cp):
    L = cp.lib()
    r = cp.cp_returns()
    a = cp.cp_rollout_args()
    a.struct_size = C.sizeof(cp.cp_rollout_args) - 8
    a.n_envs, a.T = 64, 10
    a.returns = C.pointer(r)
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL and b"struct_size" in L.cp_last_error()
    a.struct_size = C.sizeof(cp.cp_rollout_args)
    a.returns = None
    assert L.cp_rollout_ex(C.byref(a)) == cp.CP_EINVAL
    assert L.cp_rollout_ex(None) == cp.CP_EINVAL
    n = 100
    planes = torch.zeros(4, n, device="cuda")
    st = cp.cp_wrap(planes, n, 0)
    with pytest.raises(cp.CartpoleError) as e:
        cp.cp_step_ex(st, None, st, None, None, None, 5)
    assert e.value.code == cp.CP_EINVAL
    before = cp.cp_launch_count()
    with pytest.raises(cp.CartpoleError):
        cp.cp_rollout_ex(n_envs=n, T=(1 << 30), seed=0, t0=5, totals=torch.zeros(2, dtype=torch.int64, device="cuda"))
    assert cp.cp_launch_count() == before


@pytest.mark.parametrize("kind,pseed", [(inputs.POLICY_MLP32, 3), (inputs.POLICY_MLP64, 3), (inputs.POLICY_MLP_DEEP, 7),
                                        (inputs.POLICY_MLP_DEEP, 11)])
def test_wider_and_deeper_mlp_policies_against_oracle(cp, oracle, kind, pseed):
    n, T, seed = 20000, 150, 1
    w = inputs.policy_weights(kind, pseed)  # draws for which the networks use both actions
    out = outputs(n, T)
    cp.cp_rollout(n, T, seed, cp.policy(kind, w), **out)
    r = fetch(out)
    o = oracle.rollout(n, T, seed, kind, w, action_bits=True, done_bits=True, min_gap=True, nthreads=8)
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"],
                           o["min_gap"] < 1e-5)
    ga, oa = H.unpack_bits(r["action_bits"], n), H.unpack_bits(o["action_bits"], n)
    gd, od = H.unpack_bits(r["done_bits"], n), H.unpack_bits(o["done_bits"], n)
    agree = (ga == oa).all(axis=0) & (gd == od).all(axis=0)
    assert agree.mean() >= 0.99
    assert 0.02 < ga.mean() < 0.98  # the policy really decides: both actions occur


def test_per_env_linear_policies_against_oracle(cp, oracle):
    n, T, seed, off = 30001, 200, 4, 96
    wp = inputs.per_env_linear_weights(n, 11)
    d_w = torch.from_numpy(wp).cuda()
    res = []
    for shape in H.SHAPES:
        with H.rollout_shape(cp, *shape):
            out = outputs(n, T)
            cp.cp_rollout_shard(off, n, T, seed, cp.policy(cp.CP_POLICY_LINEAR_PER_ENV, d_w), **out)
            res.append(fetch(out))
    for k in res[0]:
        assert all(np.array_equal(res[0][k], other[k]) for other in res[1:]), k
    r = res[0]
    o = oracle.rollout(n, T, seed, inputs.POLICY_LINEAR_PER_ENV, wp, env_offset=off, done_bits=True,
                       action_bits=True, min_gap=True, nthreads=8)
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"], o["min_gap"] < 1e-5)
    agree = (H.unpack_bits(r["action_bits"], n) == H.unpack_bits(o["action_bits"], n)).all(axis=0)
    assert agree.mean() >= 0.995
    # identical columns reproduce the shared linear policy bit for bit
    w = inputs.policy_weights(1, 1)
    a, b = outputs(n, T), outputs(n, T)
    cp.cp_rollout(n, T, seed, cp.policy(1, w), **a)
    cp.cp_rollout(n, T, seed, cp.policy(cp.CP_POLICY_LINEAR_PER_ENV, torch.from_numpy(np.repeat(w[:, None], n, axis=1)).cuda()), **b)
    ra, rb = fetch(a), fetch(b)
    for k in ra:
        assert np.array_equal(ra[k], rb[k]), k
    # fitness differs across the population
    assert r["ep_return_sum"].std() > 1 and len(set(r["ep_count"].tolist())) > 5


def test_reset_through_the_host_program_allocator(cp, oracle):
    """cp_set_allocator: cp_reset takes its batch from torch's caching allocator (visible in torch's
    accounting, returned on cp_free) and the batch behaves like any other."""
    import gc
    n = 200_003
    gc.collect()               # tensors of earlier tests must not be freed between the readings
    gc.disable()
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    cp.use_torch_allocator(True)
    try:
        st = cp.cp_reset(n, 9)
        held = torch.cuda.memory_allocated() - before
        assert held >= 16 * n, held
        cp.use_torch_allocator(False)          # the handle keeps the release function it was made with
        # one step out of the library-owned batch into torch memory: the start states were filled
        reward = torch.empty(n, device="cuda")
        done = torch.empty(n, dtype=torch.uint8, device="cuda")
        planes = torch.zeros(4, (n + 3) // 4 * 4, device="cuda")
        out = cp.cp_wrap(planes, n, 9)
        cp.cp_step(st, None, out, reward, done)
        torch.cuda.synchronize()
        z0 = oracle.initial_state(n, 9)
        H.assert_step_matches(oracle.step(z0, seed=9, t=0, want_pre_reset=True), z0, host(planes[:, :n]),
                              host(reward), host(done))
        # and a rollout in place on it
        ret = torch.empty(n, device="cuda")
        cnt = torch.empty(n, dtype=torch.int32, device="cuda")
        cp.cp_rollout_from(st, 50, None, None, ep_return_sum=ret, ep_count=cnt)
        torch.cuda.synchronize()
        o = oracle.rollout(n, 50, 9, nthreads=4)
        H.assert_returns_match(host(ret), host(cnt).view(np.uint32), o["ep_return_sum"], o["ep_count"])
        assert st.info()["t"] == 50
        with_batch = torch.cuda.memory_allocated()
        cp.cp_free(st)
        assert torch.cuda.memory_allocated() == with_batch - held   # went back through torch
        st2 = cp.cp_reset(1000, 1)             # default allocator again: invisible to torch
        assert torch.cuda.memory_allocated() == with_batch - held
        cp.cp_free(st2)
    finally:
        gc.enable()
        cp.use_torch_allocator(False)


def test_supplied_start_states(cp, oracle):
    """Start states read from a caller's [T][4][n] array instead of the hash."""
    n, T, seed, off, t0 = 5003, 90, 3, 70, 11
    # (1) GPU-internal: the hashed start states fed back as data reproduce the hashed rollout
    pool = torch.zeros(T, 4, n, device="cuda")
    for k in range(T):
        st = cp.cp_wrap(pool[k], n, seed, t0 + k + 1, off)
        cp.cp_fill_start(st)
    a, b = outputs(n, T), outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, t0=t0, **a)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, t0=t0, start_states_in=pool, **b)
    ra, rb = fetch(a), fetch(b)
    for k in ra:
        assert np.array_equal(ra[k], rb[k]), k
    # (2) against the oracle: arbitrary start states (some at the edge: very short episodes),
    # with supplied actions (all randomness as data), the hashed actions, and a linear policy
    rng = np.random.default_rng(5)
    states = (0.05 * rng.uniform(-1, 1, (T, 4, n))).astype(np.float32)
    states[:, 2, ::3] = np.float32(0.2)
    d_states = torch.from_numpy(states).cuda()
    acts = rng.integers(0, 2, (T, n)).astype(np.uint8)
    d_bits = torch.from_numpy(pack_bits(acts).view(np.int32)).cuda()
    w = inputs.policy_weights(1, 4)
    for gpu_kw, ora_kw, kind, wts in (({"action_bits_in": d_bits}, {"action_bits_in": pack_bits(acts)}, 0, None),
                                      ({}, {}, 0, None), ({}, {}, 1, w)):
        out = outputs(n, T)
        cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, start_states_in=d_states,
                         policy=cp.policy(kind, wts) if kind else None, **gpu_kw, **out)
        r = fetch(out)
        o = oracle.rollout(n, T, seed, kind, wts, env_offset=off, start_states_in=states, done_bits=True,
                           min_gap=True, nthreads=4, **ora_kw)
        H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"],
                               o["min_gap"] < 1e-5)
        same = r["ep_return_sum"] == o["ep_return_sum"]
        assert np.array_equal(H.unpack_bits(r["done_bits"], n)[:, same], H.unpack_bits(o["done_bits"], n)[:, same])
        assert r["ep_count"].sum() > n and (kind or np.median(r["ep_count"][::3]) >= 3)
    # with an episode step limit on top (the two options meet in one kernel)
    out = outputs(n, T)
    cp.cp_rollout_ex(n_envs=n, T=T, seed=seed, env_offset=off, start_states_in=d_states, max_episode_steps=7, **out)
    r = fetch(out)
    o = oracle.rollout(n, T, seed, env_offset=off, start_states_in=states, max_episode_steps=7, done_bits=True, nthreads=4)
    H.assert_returns_match(r["ep_return_sum"], r["ep_count"], o["ep_return_sum"], o["ep_count"])
    same = r["ep_return_sum"] == o["ep_return_sum"]
    assert np.array_equal(H.unpack_bits(r["done_bits"], n)[:, same], H.unpack_bits(o["done_bits"], n)[:, same])
    # (3) the contracted arithmetic and chunked calls on a batch take the option too
    st = cp.cp_reset(n, seed)
    ret = torch.empty(n, device="cuda")
    cp.cp_rollout_ex(state=st, T=T, start_states_in=d_states, arithmetic=cp.CP_ARITH_CONTRACTED, ep_return_sum=ret)
    torch.cuda.synchronize()
    assert st.info()["t"] == T and float(ret.sum()) > 0
    with pytest.raises(AssertionError):
        cp.cp_rollout_ex(n_envs=n, T=T - 1, seed=seed, start_states_in=d_states, ep_return_sum=ret)
