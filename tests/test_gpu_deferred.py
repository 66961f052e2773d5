"""GPU tests of the deferred-restart rollout kernel (two environments per thread stepped by packed
float32 instructions, a clock per environment, restarts every K trips): it must produce the bits
of the general rollout kernel for every call it covers — every policy, any trip spacing, ragged sizes, horizons
shorter than one block of trips, global times beyond 2^16, the episode step limit, steps carried
in, caller-supplied states with angles outside the polynomial range — and the oracle's returns."""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

WIDE = (inputs.POLICY_MLP32, inputs.POLICY_MLP64, inputs.POLICY_MLP_DEEP)  # 4-32-2, 4-64-2, 4-16-16-2
GENERAL = (2, 1)   # two envs per thread, restarts by the whole warp after every step
DEFERRED = (2, 5)


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def outputs(n):
    return {"ep_return_sum": torch.full((n,), -1.0, dtype=torch.float32, device="cuda"),
            "ep_count": torch.full((n,), -1, dtype=torch.int32, device="cuda"),
            "totals": torch.zeros(2, dtype=torch.int64, device="cuda"),
            "final_state": torch.full((4, n), 9.0, dtype=torch.float32, device="cuda")}


def fetch(out):
    torch.cuda.synchronize()
    return {k: v.cpu().numpy().view(np.uint32 if v.dtype != torch.int64 else np.uint64) for k, v in out.items()}


def make_policy(cp, kind, n):
    if kind == 0:
        return None, None
    if kind in (1, 2):
        w = inputs.policy_weights(kind, kind)
        return cp.policy(kind, w), w
    if kind in WIDE:  # weight draws for which the network uses both actions
        w = inputs.policy_weights(kind, 7 if kind == inputs.POLICY_MLP_DEEP else 3)
        return cp.policy(kind, w), w
    w = inputs.per_env_linear_weights(n, 11)
    return cp.policy(cp.CP_POLICY_LINEAR_PER_ENV, torch.from_numpy(w).cuda()), w


def run(cp, shape, k, **kw):
    n = kw["n_envs"]
    with H.rollout_shape(cp, *shape):
        cp.cp_tune("rollout_defer", k)
        try:
            out = outputs(n)
            cp.cp_rollout_ex(**kw, **out)
            return fetch(out)
        finally:
            cp.cp_tune("rollout_defer", 0)


@pytest.mark.parametrize("kind", [0, 1, 2, 6])
@pytest.mark.parametrize("n,T,t0,off,limit", [
    (1, 1, 0, 0, 0), (63, 2, 0, 5, 0), (65, 5, 3, 0, 0), (4099, 61, 0, 77, 0), (4099, 61, 0, 77, 23),
    (70001, 200, 0, 0, 0), (20000, 150, 70000, 1 << 20, 0), (20000, 150, 65500, 0, 40), (3000, 700, 11, 0, 500),
])
def test_same_bits_as_the_general_kernel(cp, kind, n, T, t0, off, limit):
    pol, _ = make_policy(cp, kind, n)
    kw = dict(n_envs=n, T=T, seed=3, t0=t0, env_offset=off, policy=pol, max_episode_steps=limit)
    want = run(cp, GENERAL, 0, **kw)
    assert want["ep_count"].max() > 0 or T < 8
    for k in (2, 3, 4, 6, 8):
        got = run(cp, DEFERRED, k, **kw)
        for key in want:
            assert np.array_equal(want[key], got[key]), (key, k)
    # the contracted arithmetic: its deferred form gives the bits of its general form
    kw["arithmetic"] = cp.CP_ARITH_CONTRACTED
    want_c, got_c = run(cp, GENERAL, 0, **kw), run(cp, DEFERRED, 0, **kw)
    for key in want_c:
        assert np.array_equal(want_c[key], got_c[key]), (key, "contracted")
    assert n < 4000 or not np.array_equal(want_c["final_state"], want["final_state"])


@pytest.mark.parametrize("kind", WIDE)
@pytest.mark.parametrize("n,T,t0,off", [(1, 1, 0, 0), (63, 2, 0, 5), (4099, 61, 3, 77), (70001, 120, 0, 0),
                                        (20000, 90, 70000, 1 << 20)])
def test_wider_and_deeper_networks_same_bits_as_the_general_kernel(cp, kind, n, T, t0, off):
    """The deferred kernel covers these networks for the plain call (no step limit, no per-step
    outputs), in both arithmetics; with a limit the call must still come out right (it takes the
    general kernel)."""
    pol, _ = make_policy(cp, kind, n)
    for arith in (cp.CP_ARITH_EXACT, cp.CP_ARITH_CONTRACTED):
        for limit in (0, 17):
            kw = dict(n_envs=n, T=T, seed=8, t0=t0, env_offset=off, policy=pol, max_episode_steps=limit, arithmetic=arith)
            want = run(cp, GENERAL, 0, **kw)
            before = cp.cp_launch_count()
            got = run(cp, DEFERRED, 0, **kw)
            assert cp.cp_launch_count() - before == 1
            for key in want:
                assert np.array_equal(want[key], got[key]), (key, arith, limit)
        assert want["ep_count"].max() > 0 or T < 8


@pytest.mark.parametrize("kind", [0, 1, 2])
@pytest.mark.parametrize("limit,streams,n", [(0, False, 9001), (31, False, 9001), (0, True, 9001), (13, True, 9001),
                                             (0, True, 9028), (13, True, 9028)])
def test_chunks_from_a_callers_states(cp, kind, limit, streams, n):
    """States with angles far outside the polynomial range and running-episode lengths carried in
    and out, advanced in chunks of 1, 2, 7 and 40 steps: general and deferred kernels stay
    identical in the batch itself, the carried lengths and the per-chunk results."""
    seed = 5
    z = np.concatenate([inputs.random_states(n // 3, seed=4, spread="wide"),
                        inputs.random_states(n // 3, seed=5, spread="live"),
                        inputs.random_states(n - 2 * (n // 3), seed=6, spread="edge")], axis=1)
    pol, _ = make_policy(cp, kind, n)
    results = {}
    for name, shape in (("general", GENERAL), ("deferred", DEFERRED)):
        planes = torch.zeros(4, n + 3, dtype=torch.float32, device="cuda")
        planes[:, :n] = torch.from_numpy(z).cuda()
        st = cp.cp_wrap(planes, n, seed, 17, 64)  # plane stride n + 3: no alignment to lean on
        ep_len = torch.from_numpy(np.arange(n, dtype=np.int32) % 29).cuda()
        log = []
        with H.rollout_shape(cp, *shape):
            for T in (1, 2, 7, 40):
                out = {"ep_return_sum": torch.zeros(n, device="cuda"),
                       "ep_count": torch.zeros(n, dtype=torch.int32, device="cuda"),
                       "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
                if streams:  # the reward plane and the done bits of a chunk that starts from given states
                    out["reward_stream"] = torch.full((T, n), -2.0, device="cuda")
                    out["done_bits"] = torch.full((T, (n + 31) // 32), -1, dtype=torch.int32, device="cuda")
                cp.cp_rollout_ex(T=T, state=st, ep_len=ep_len, policy=pol, max_episode_steps=limit, **out)
                torch.cuda.synchronize()
                log.append({k: v.cpu().numpy().copy() for k, v in out.items()})
                log.append({"planes": planes.cpu().numpy().copy(), "ep_len": ep_len.cpu().numpy().copy()})
        assert st.info()["t"] == 17 + 50
        results[name] = log
    for a, b in zip(results["general"], results["deferred"]):
        for key in a:
            assert np.array_equal(a[key].view(np.uint32) if a[key].dtype == np.float32 else a[key],
                                  b[key].view(np.uint32) if b[key].dtype == np.float32 else b[key]), key
    assert sum(int(c["ep_count"].sum()) for c in results["deferred"][0::2]) > n // 4


@pytest.mark.parametrize("kind", [0, 1, 2, 6, *WIDE])
def test_returns_against_the_oracle(cp, oracle, kind):
    n, T, seed = 50001, 300, 2
    pol, w = make_policy(cp, kind, n)
    r = run(cp, DEFERRED, 0, n_envs=n, T=T, seed=seed, policy=pol)
    o = oracle.rollout(n, T, seed, inputs.POLICY_LINEAR_PER_ENV if kind == 6 else kind, w, final_state=True,
                       min_gap=True, nthreads=8)
    excuse = (o["min_gap"] < 1e-5) if kind else None
    res = H.assert_returns_match(r["ep_return_sum"].view(np.float32), r["ep_count"], o["ep_return_sum"], o["ep_count"],
                                 excuse)
    assert int(r["totals"][0]) == int(r["ep_return_sum"].view(np.float32).astype(np.float64).sum())
    assert int(r["totals"][1]) == int(r["ep_count"].astype(np.int64).sum())
    same = (r["ep_return_sum"].view(np.float32) == o["ep_return_sum"]) & (r["ep_count"] == o["ep_count"])
    err = np.abs(r["final_state"].view(np.float32)[:, same].astype(np.float64) - o["final_state"][:, same])
    assert np.quantile(err.max(axis=0), 0.99) < 1e-3 and res["identical"] > 0.99


@pytest.mark.parametrize("kind", [0, 1, 2, 6])
@pytest.mark.parametrize("n,T,t0,limit", [(1, 3, 0, 0), (33, 40, 7, 0), (4099, 61, 0, 19), (70001, 120, 0, 0),
                                          (20000, 90, 65530, 0), (4164, 1, 0, 0), (4164, 2, 5, 0), (8192, 37, 0, 7),
                                          (66564, 250, 0, 0)])
def test_reward_plane_and_done_bits_with_clocks_per_environment(cp, kind, n, T, t0, limit):
    """The deferred kernel writes the reward plane row by row and sets done bits by atomic OR from
    the restart pass: every word must equal the general kernel's, padding bits included."""
    pol, _ = make_policy(cp, kind, n)
    words = (n + 31) // 32
    res = {}
    for name, shape, k in (("general", GENERAL, 0), ("deferred4", DEFERRED, 4), ("deferred3", DEFERRED, 3)):
        out = outputs(n)
        out["reward_stream"] = torch.full((T, n), -7.0, dtype=torch.float32, device="cuda")
        out["done_bits"] = torch.full((T, words), -1, dtype=torch.int32, device="cuda")  # stale bits everywhere
        with H.rollout_shape(cp, *shape):
            cp.cp_tune("rollout_defer", k)
            try:
                cp.cp_rollout_ex(n_envs=n, T=T, seed=6, t0=t0, env_offset=9, policy=pol, max_episode_steps=limit, **out)
            finally:
                cp.cp_tune("rollout_defer", 0)
        res[name] = fetch(out)
    for name in ("deferred4", "deferred3"):
        for key in res["general"]:
            assert np.array_equal(res["general"][key], res[name][key]), (key, name)
    r = res["deferred4"]
    assert (r["reward_stream"].view(np.float32) == 1.0).all()
    done = H.unpack_bits(r["done_bits"], n)
    assert np.array_equal(done.sum(axis=0), r["ep_count"])
    if n % 32:
        assert not np.any(r["done_bits"][:, -1] >> (n % 32))
