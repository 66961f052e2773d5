"""Pins for the oracle's batched step, rollout, bookkeeping and policies (CPU only).

Brute force on tiny batches (the batch functions against per-environment scalar
calls composed in Python), structural invariants of the episode bookkeeping,
exact-rational evaluation of the policy FMA chains and stored aggregates of the
smallest benchmark configuration.
"""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs
from tests.exact_arith import fma_chain_exact


def brute_step(oracle, planes, seed, t, action=None, env_offset=0):
    n = planes.shape[1]
    out = np.empty_like(planes)
    done = np.zeros(n, np.uint8)
    act = np.zeros(n, np.uint8)
    for i in range(n):
        a = int(action[i]) if action is not None else oracle.action(seed, env_offset + i, t)
        z, d = oracle.dynamics_f32(planes[:, i], a)
        if d:
            z = oracle.reset_state(seed, env_offset + i, t + 1)
        out[:, i] = z
        done[i] = d
        act[i] = a
    return out, done, act


@pytest.mark.parametrize("n", [1, 3, 5, 33])
def test_step_matches_brute_force(oracle, n):
    z = inputs.random_states(n, seed=n, spread="edge")
    for t, off, act in ((0, 0, None), (7, 1000, None), (3, 0, inputs.random_actions(n, 5))):
        r = oracle.step(z, seed=2, t=t, action_u8=act, env_offset=off)
        out, done, a = brute_step(oracle, z, 2, t, act, off)
        assert np.array_equal(r["state"].view(np.uint32), out.view(np.uint32))
        assert np.array_equal(r["done"], done) and np.array_equal(r["action"], a)
        assert np.all(r["reward"] == 1.0)
    if n == 33:
        assert done.any() and not done.all()


def test_initial_state_is_reset_at_time_zero(oracle):
    r = oracle.rollout(5, 1, 3, trajectory=False, final_state=True)
    z0 = oracle.initial_state(5, 3)
    s = oracle.step(z0, seed=3, t=0)
    assert np.array_equal(r["final_state"].view(np.uint32), s["state"].view(np.uint32))


@pytest.mark.parametrize("n,T", [(1, 64), (33, 64), (1025, 40)])
def test_rollout_equals_repeated_steps(oracle, n, T):
    seed = 0
    r = oracle.rollout(n, T, seed, trajectory=True, done_bits=True, action_bits=True,
                       reward_stream=True, final_state=True)
    z = oracle.initial_state(n, seed)
    ep_len = np.zeros(n, np.int64)
    ret = np.zeros(n, np.int64)
    cnt = np.zeros(n, np.int64)
    for t in range(T):
        s = oracle.step(z, seed, t)
        z = s["state"]
        assert np.array_equal(r["trajectory"][t].view(np.uint32), z.view(np.uint32))
        db = np.unpackbits(r["done_bits"][t].view(np.uint8), bitorder="little")[:n]
        ab = np.unpackbits(r["action_bits"][t].view(np.uint8), bitorder="little")[:n]
        assert np.array_equal(db, s["done"]) and np.array_equal(ab, s["action"])
        ep_len += 1
        d = s["done"].astype(bool)
        ret[d] += ep_len[d]
        cnt[d] += 1
        ep_len[d] = 0
    assert np.array_equal(r["final_state"], z)
    assert np.array_equal(r["ep_return_sum"], ret.astype(np.float32))
    assert np.array_equal(r["ep_count"], cnt.astype(np.uint32))
    assert np.all(r["reward_stream"] == 1.0)
    assert int(r["totals"][0]) == ret.sum() and int(r["totals"][1]) == cnt.sum()


def test_bookkeeping_invariants(oracle):
    n, T = 512, 300
    r = oracle.rollout(n, T, 4, done_bits=True)
    db = np.unpackbits(r["done_bits"].view(np.uint8), bitorder="little", axis=1)[:, :n]
    assert np.array_equal(db.sum(axis=0), r["ep_count"])
    # the sum of completed-episode lengths is the time of the last termination + 1
    last = np.where(db.any(axis=0), T - 1 - np.argmax(db[::-1], axis=0), -1)
    assert np.array_equal(r["ep_return_sum"], (last + 1).astype(np.float32))
    assert r["ep_return_sum"].max() <= T
    assert int(r["totals"][0]) == int(r["ep_return_sum"].astype(np.int64).sum())
    assert int(r["totals"][1]) == int(r["ep_count"].sum())
    # random-policy episodes last about 22 steps
    mean_len = r["totals"][0] / r["totals"][1]
    assert 20.5 < mean_len < 23.5


def test_threads_and_shards_do_not_change_results(oracle):
    n, T = 1000, 50
    base = oracle.rollout(n, T, 9, done_bits=True, final_state=True)
    mt = oracle.rollout(n, T, 9, done_bits=True, final_state=True, nthreads=3)
    for k in ("ep_return_sum", "ep_count", "totals", "done_bits", "final_state"):
        assert np.array_equal(base[k], mt[k]), k
    tot = np.zeros(2, np.uint64)
    for rank in range(3):
        lo, hi = inputs.shard_range(n, rank, 3)
        part = oracle.rollout(hi - lo, T, 9, env_offset=lo, final_state=True)
        assert np.array_equal(part["ep_return_sum"], base["ep_return_sum"][lo:hi])
        assert np.array_equal(part["final_state"], base["final_state"][:, lo:hi])
        tot += part["totals"]
    assert np.array_equal(tot, base["totals"])


def test_chunked_rollout_resumes_exactly(oracle):
    n, T1, T2 = 200, 37, 41
    whole = oracle.rollout(n, T1 + T2, 6, final_state=True)
    a = oracle.rollout(n, T1, 6, final_state=True, ep_len=np.zeros(n, np.uint32))
    b = oracle.rollout(n, T2, 6, t0=T1, init_state=a["final_state"], ep_len=a["ep_len"], final_state=True)
    assert np.array_equal(whole["final_state"], b["final_state"])
    assert np.array_equal(whole["ep_return_sum"], a["ep_return_sum"] + b["ep_return_sum"])
    assert np.array_equal(whole["ep_count"], a["ep_count"] + b["ep_count"])


def test_config1_aggregates(oracle):
    # Stored aggregates of 1,024 envs x 200 steps, seed 0, random policy; they were
    # computed before this repository existed by an independent numpy evaluation.
    r = oracle.rollout(1024, 200, 0, done_bits=True, action_bits=True)
    ones = int(np.unpackbits(r["action_bits"].view(np.uint8)).sum())
    assert ones == 102450
    assert [int(v) for v in r["ep_return_sum"][:8]] == [198, 176, 192, 193, 189, 181, 190, 199]
    assert [int(v) for v in r["ep_count"][:8]] == [7, 8, 8, 6, 9, 9, 9, 10]
    db = np.unpackbits(r["done_bits"].view(np.uint8), bitorder="little", axis=1)
    assert list(np.nonzero(db[:, 0])[0]) == [25, 50, 93, 108, 154, 183, 197]
    assert list(np.nonzero(db[:, 1])[0]) == [11, 33, 50, 64, 113, 138, 163, 175]
    # a handful of envs pass within 1e-5 of a threshold, so another libm may move these by a few units
    assert abs(int(r["totals"][1]) - 8832) <= 3
    assert abs(int(r["totals"][0]) - 190839) <= 60


# ------------------------------------------------------------------ policies
def test_linear_policy_is_an_fma_chain(oracle):
    w = inputs.policy_weights(inputs.POLICY_LINEAR, 1)
    zs = inputs.random_states(200, seed=2, spread="live")
    for i in range(zs.shape[1]):
        got = oracle.linear_logits(w, zs[:, i])
        for k in range(2):
            want = fma_chain_exact(w[4 * k:4 * k + 4], zs[:, i], w[8 + k])
            assert got[k] == want


def test_mlp_policy_structure(oracle):
    w = inputs.policy_weights(inputs.POLICY_MLP, 2)
    zs = inputs.random_states(100, seed=3, spread="live")
    for i in range(zs.shape[1]):
        z = zs[:, i]
        h64 = np.tanh(w[:64].reshape(16, 4).astype(np.float64) @ z.astype(np.float64) + w[64:80])
        want = w[80:112].reshape(2, 16).astype(np.float64) @ h64 + w[112:114]
        got = oracle.mlp_logits(w, z)
        assert np.all(np.abs(got - want) < 2e-6)
    # a one-hot probe isolates each weight: hidden unit j, input i
    for j in (0, 5, 15):
        probe = np.zeros(114, np.float32)
        probe[4 * j + 2] = 1.0      # W1[j][2]
        probe[80 + j] = 1.0         # W2[0][j]
        probe[96 + j] = -2.0        # W2[1][j]
        probe[112:] = (0.25, -0.5)
        got = oracle.mlp_logits(probe, [9, 9, 0.3, 9])
        t = np.tanh(0.3)
        assert abs(got[0] - (0.25 + t)) < 1e-6 and abs(got[1] - (-0.5 - 2 * t)) < 1e-6


def test_policy_rollout_uses_pre_step_observation_and_tie_rule(oracle):
    n, T = 64, 30
    w = inputs.policy_weights(inputs.POLICY_LINEAR, 1)
    r = oracle.rollout(n, T, 0, inputs.POLICY_LINEAR, w, trajectory=True, action_bits=True)
    z = oracle.initial_state(n, 0)
    for t in range(T):
        ab = np.unpackbits(r["action_bits"][t].view(np.uint8), bitorder="little")[:n]
        for i in range(n):
            lg = oracle.linear_logits(w, z[:, i])
            assert ab[i] == int(lg[1] > lg[0])
        z = r["trajectory"][t]
    # all-zero weights tie every step: index 0 (push left) wins
    r0 = oracle.rollout(8, 20, 0, inputs.POLICY_LINEAR, np.zeros(10, np.float32), action_bits=True, min_gap=True)
    assert not r0["action_bits"].any() and np.all(r0["min_gap"] == 0)
    # MLP path runs and reports its argmax gaps
    wm = inputs.policy_weights(inputs.POLICY_MLP, 2)
    rm = oracle.rollout(16, 20, 0, inputs.POLICY_MLP, wm, min_gap=True)
    assert np.all(np.isfinite(rm["min_gap"])) and rm["totals"][1] > 0


def test_threshold_margin_diagnostic_matches_a_walk(oracle):
    """min_margin (used by the GPU comparison rules to excuse envs that came within 1e-5 of a
    termination threshold) against a per-env walk composed from the scalar calls."""
    n, T, seed = 40, 120, 6
    r = oracle.rollout(n, T, seed, min_margin=True, done_bits=True)
    xt, tt = float(np.float32(2.4)), float(np.float32(12 * 2 * np.pi / 360))
    for i in range(n):
        z = oracle.reset_state(seed, i, 0)
        best = np.inf
        for t in range(T):
            zn, d = oracle.dynamics_f32(z, oracle.action(seed, i, t))
            best = min(best, abs(abs(float(zn[0])) - xt), abs(abs(float(zn[2])) - tt))
            z = oracle.reset_state(seed, i, t + 1) if d else zn
        assert r["min_margin"][i] == np.float32(best)
    # an env that terminates has passed a threshold by less than one step's travel
    assert (r["min_margin"] < 0.05).all() and (r["min_margin"] >= 0).all()
