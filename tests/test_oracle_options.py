"""Pins for the oracle's optional behaviours (CPU only): the episode step limit of
CartPole-v1 (an episode is cut off after a fixed number of steps and the environment restarts
as after a fall) and actions supplied as a packed bit stream instead of drawn by the policy.
Both are checked by brute force against per-environment scalar calls composed in Python and
by the invariants the definitions imply."""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs


def pack_bits(bits: np.ndarray) -> np.ndarray:
    """[T, n] 0/1 -> [T, ceil(n/32)] uint32, bit i%32 of word i//32."""
    T, n = bits.shape
    words = (n + 31) // 32
    padded = np.zeros((T, words * 32), np.uint8)
    padded[:, :n] = bits
    return np.packbits(padded, axis=1, bitorder="little").view(np.uint32).reshape(T, words)


def unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    return np.unpackbits(np.ascontiguousarray(words).view(np.uint8), axis=-1, bitorder="little")[..., :n]


def brute_rollout(oracle, n, T, seed, limit=0, actions=None, env_offset=0):
    """Scalar composition: dynamics_f32 / action / reset_state per env and step."""
    ret = np.zeros(n, np.int64)
    cnt = np.zeros(n, np.int64)
    done = np.zeros((T, n), np.uint8)
    final = np.zeros((4, n), np.float32)
    for i in range(n):
        e = env_offset + i
        z = oracle.reset_state(seed, e, 0)
        ep_len = 0
        for t in range(T):
            a = int(actions[t, i]) if actions is not None else oracle.action(seed, e, t)
            z, d = oracle.dynamics_f32(z, a)
            ep_len += 1
            if limit and ep_len >= limit:
                d = True
            if d:
                ret[i] += ep_len
                cnt[i] += 1
                ep_len = 0
                z = oracle.reset_state(seed, e, t + 1)
            done[t, i] = d
        final[:, i] = z
    return ret, cnt, done, final


@pytest.mark.parametrize("limit", [1, 3, 7, 25])
def test_step_limit_matches_brute_force(oracle, limit):
    n, T, seed = 37, 60, 4
    r = oracle.rollout(n, T, seed, max_episode_steps=limit, done_bits=True, final_state=True, env_offset=5)
    ret, cnt, done, final = brute_rollout(oracle, n, T, seed, limit, env_offset=5)
    assert np.array_equal(r["ep_return_sum"], ret.astype(np.float32))
    assert np.array_equal(r["ep_count"], cnt.astype(np.uint32))
    assert np.array_equal(unpack_bits(r["done_bits"], n), done)
    assert np.array_equal(r["final_state"], final)


def test_step_limit_invariants(oracle):
    n, T, seed = 300, 200, 1
    free = oracle.rollout(n, T, seed, done_bits=True)
    # a limit of 1 ends an episode at every step
    one = oracle.rollout(n, T, seed, max_episode_steps=1)
    assert np.all(one["ep_count"] == T) and np.all(one["ep_return_sum"] == T)
    # a limit nothing reaches changes nothing
    big = oracle.rollout(n, T, seed, max_episode_steps=T + 1, done_bits=True)
    assert np.array_equal(big["done_bits"], free["done_bits"])
    # with a limit, no gap between consecutive done flags exceeds it, and every cut-off shows up
    lim = 12
    r = oracle.rollout(n, T, seed, max_episode_steps=lim, done_bits=True)
    d = unpack_bits(r["done_bits"], n)
    for i in range(n):
        times = np.concatenate(([-1], np.nonzero(d[:, i])[0]))
        gaps = np.diff(times)
        assert gaps.size == 0 or gaps.max() <= lim
        assert T - 1 - times[-1] < lim  # the running episode is shorter than the limit
        assert r["ep_return_sum"][i] == times[-1] + 1
    assert r["totals"][1] > free["totals"][1]
    # until an env's first cut-off its done stream equals the unlimited one
    df = unpack_bits(free["done_bits"], n)
    for i in range(0, n, 7):
        gaps = np.diff(np.concatenate(([-1], np.nonzero(df[:, i])[0])))
        first_long = np.nonzero(gaps > lim)[0]
        upto = T if first_long.size == 0 else (np.concatenate(([-1], np.nonzero(df[:, i])[0]))[first_long[0]] + lim)
        assert np.array_equal(d[:upto, i], df[:upto, i])


def test_step_limited_equals_limited_rollout(oracle):
    n, T, seed, lim = 50, 40, 2, 9
    r = oracle.rollout(n, T, seed, max_episode_steps=lim, trajectory=True, done_bits=True)
    z = oracle.initial_state(n, seed)
    ep_len = np.zeros(n, np.uint32)
    d = unpack_bits(r["done_bits"], n)
    for t in range(T):
        s = oracle.step_limited(z, seed, t, ep_len, lim)
        z, ep_len = s["state"], s["ep_len"]
        assert np.array_equal(z, r["trajectory"][t]) and np.array_equal(s["done"], d[t])
        assert np.all(s["reward"] == 1.0) and ep_len.max() < lim
    # no limit: step_limited is the plain step plus a length counter
    z0 = inputs.random_states(200, seed=3, spread="edge")
    a = oracle.step(z0, seed, 5)
    b = oracle.step_limited(z0, seed, 5, np.full(200, 7, np.uint32), 0)
    assert np.array_equal(a["state"], b["state"]) and np.array_equal(a["done"], b["done"])
    assert np.array_equal(b["ep_len"], np.where(a["done"] == 1, 0, 8))


def test_chunked_limited_rollout_resumes_exactly(oracle):
    n, seed, lim = 100, 3, 15
    whole = oracle.rollout(n, 70, seed, max_episode_steps=lim, final_state=True)
    a = oracle.rollout(n, 33, seed, max_episode_steps=lim, final_state=True, ep_len=np.zeros(n, np.uint32))
    b = oracle.rollout(n, 37, seed, t0=33, init_state=a["final_state"], ep_len=a["ep_len"], max_episode_steps=lim,
                       final_state=True)
    assert np.array_equal(whole["final_state"], b["final_state"])
    assert np.array_equal(whole["ep_return_sum"], a["ep_return_sum"] + b["ep_return_sum"])
    assert np.array_equal(whole["ep_count"], a["ep_count"] + b["ep_count"])


def test_supplied_action_stream(oracle):
    n, T, seed = 45, 50, 6
    rng = np.random.default_rng(0)
    acts = rng.integers(0, 2, (T, n)).astype(np.uint8)
    r = oracle.rollout(n, T, seed, action_bits_in=pack_bits(acts), done_bits=True, action_bits=True,
                       final_state=True, min_gap=True)
    ret, cnt, done, final = brute_rollout(oracle, n, T, seed, actions=acts)
    assert np.array_equal(r["ep_return_sum"], ret.astype(np.float32))
    assert np.array_equal(r["ep_count"], cnt.astype(np.uint32))
    assert np.array_equal(unpack_bits(r["done_bits"], n), done)
    assert np.array_equal(unpack_bits(r["action_bits"], n), acts)  # echoed back unchanged
    assert np.array_equal(r["final_state"], final) and np.all(np.isinf(r["min_gap"]))
    # feeding the hashed actions back in reproduces the random-policy rollout
    h = oracle.rollout(n, T, seed, action_bits=True, final_state=True)
    g = oracle.rollout(n, T, seed, action_bits_in=h["action_bits"], final_state=True)
    for k in ("ep_return_sum", "ep_count", "final_state", "totals"):
        assert np.array_equal(h[k], g[k])
    # a supplied stream overrides a policy; padding bits beyond n are ignored
    w = inputs.policy_weights(inputs.POLICY_LINEAR, 1)
    p = oracle.rollout(n, T, seed, inputs.POLICY_LINEAR, w, action_bits_in=pack_bits(acts))
    assert np.array_equal(p["ep_return_sum"], r["ep_return_sum"])
    full = pack_bits(acts).copy()
    full[:, -1] |= np.uint32((0xFFFFFFFF << (n % 32)) & 0xFFFFFFFF)
    q = oracle.rollout(n, T, seed, action_bits_in=full)
    assert np.array_equal(q["ep_return_sum"], r["ep_return_sum"])
    # constant push right from the start states: the pole falls to the negative side quickly
    ones = np.ones((20, 8), np.uint8)
    c = oracle.rollout(8, 20, seed, action_bits_in=pack_bits(ones), done_bits=True)
    first = np.argmax(unpack_bits(c["done_bits"], 8), axis=0)
    assert np.all((first >= 6) & (first <= 12))


def test_supplied_start_states(oracle):
    """All randomness as data (the paper's baseline, Sec. V-A): start states read from an array."""
    n, T, seed, off = 37, 60, 3, 500
    # (1) feeding the hashed start states of times t0+1 .. t0+T back in reproduces the hashed rollout
    t0 = 11
    pool = np.stack([oracle.initial_state(n, seed, t0 + k + 1, off) for k in range(T)])
    h = oracle.rollout(n, T, seed, env_offset=off, t0=t0, trajectory=True, done_bits=True)
    g = oracle.rollout(n, T, seed, env_offset=off, t0=t0, start_states_in=pool, trajectory=True, done_bits=True)
    for k in ("ep_return_sum", "ep_count", "trajectory", "done_bits", "totals"):
        assert np.array_equal(h[k], g[k]), k
    # (2) arbitrary supplied states: after every done the state is exactly row k of the array, and
    # between restarts the trajectory is the one-step dynamics (brute force with co_step's pieces)
    rng = np.random.default_rng(4)
    pool = (0.05 * rng.uniform(-1, 1, (T, 4, n))).astype(np.float32)
    pool[:, 2, ::3] = np.float32(0.2)      # some start states sit right at the edge: very short episodes
    acts = rng.integers(0, 2, (T, n)).astype(np.uint8)
    r = oracle.rollout(n, T, seed, action_bits_in=pack_bits(acts), start_states_in=pool, trajectory=True,
                       done_bits=True)
    done = unpack_bits(r["done_bits"], n)
    z = oracle.initial_state(n, seed)
    ep_len = np.zeros(n, np.int64)
    ret = np.zeros(n, np.int64)
    cnt = np.zeros(n, np.int64)
    for k in range(T):
        for i in range(n):
            zn, d = oracle.dynamics_f32(z[:, i], int(acts[k, i]))
            ep_len[i] += 1
            assert int(d) == done[k, i]
            if d:
                ret[i] += ep_len[i]
                cnt[i] += 1
                ep_len[i] = 0
                zn = pool[k, :, i]
            assert np.array_equal(np.asarray(zn, np.float32).view(np.uint32), r["trajectory"][k, :, i].view(np.uint32))
            z[:, i] = zn
    assert np.array_equal(r["ep_return_sum"], ret.astype(np.float32)) and np.array_equal(r["ep_count"], cnt.astype(np.uint32))
    assert cnt[::3].min() >= 3 and done.sum() > 0


@pytest.mark.parametrize("kind,hidden", [(inputs.POLICY_MLP32, 32), (inputs.POLICY_MLP64, 64)])
def test_wider_mlp_policies(oracle, kind, hidden):
    w = inputs.policy_weights(kind, 7)
    assert w.size == 7 * hidden + 2
    zs = inputs.random_states(100, seed=5, spread="live")
    w1 = w[:4 * hidden].reshape(hidden, 4).astype(np.float64)
    b1 = w[4 * hidden:5 * hidden].astype(np.float64)
    w2 = w[5 * hidden:7 * hidden].reshape(2, hidden).astype(np.float64)
    b2 = w[7 * hidden:].astype(np.float64)
    for i in range(zs.shape[1]):
        z = zs[:, i]
        want = w2 @ np.tanh(w1 @ z.astype(np.float64) + b1) + b2
        got = oracle.mlp_logits_wide(w, hidden, z)
        assert np.all(np.abs(got - want) < 4e-6)
    # one-hot probe isolates unit j, input 1 and both output rows
    for j in (0, hidden // 2, hidden - 1):
        probe = np.zeros(7 * hidden + 2, np.float32)
        probe[4 * j + 1] = 2.0
        probe[5 * hidden + j] = 1.0
        probe[6 * hidden + j] = -3.0
        probe[7 * hidden:] = (0.5, 0.25)
        got = oracle.mlp_logits_wide(probe, hidden, [9, 0.1, 9, 9])
        t = np.tanh(0.2)
        assert abs(got[0] - (0.5 + t)) < 1e-6 and abs(got[1] - (0.25 - 3 * t)) < 1e-6
    # rollouts use the pre-step observation and the tie rule
    n, T = 32, 25
    r = oracle.rollout(n, T, 0, kind, w, trajectory=True, action_bits=True, min_gap=True)
    z = oracle.initial_state(n, 0)
    for t in range(T):
        ab = unpack_bits(r["action_bits"][t], n)
        for i in range(n):
            lg = oracle.mlp_logits_wide(w, hidden, z[:, i])
            assert ab[i] == int(lg[1] > lg[0])
        z = r["trajectory"][t]
    assert np.all(np.isfinite(r["min_gap"]))


def test_wide_mlp_routine_reduces_to_the_16_unit_network(oracle):
    w = inputs.policy_weights(inputs.POLICY_MLP, 2)
    zs = inputs.random_states(300, seed=6, spread="wide")
    for i in range(zs.shape[1]):
        a = oracle.mlp_logits(w, zs[:, i])
        b = oracle.mlp_logits_wide(w, 16, zs[:, i])
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_deep_mlp_policy(oracle):
    """4 -> 16 (tanh) -> 16 (tanh) -> 2: against a float64 matrix evaluation, a probe that isolates
    one path through both hidden layers (catches a transposed or shifted weight block), the
    reduction to the one-hidden-layer network when the second layer is a scaled identity in the
    linear range of tanh, and the use of the pre-step observation in rollouts."""
    kind = inputs.POLICY_MLP_DEEP
    w = inputs.policy_weights(kind, 4)
    assert w.size == 386 == inputs.N_WEIGHTS[kind]
    w1, b1 = w[:64].reshape(16, 4).astype(np.float64), w[64:80].astype(np.float64)
    w2, b2 = w[80:336].reshape(16, 16).astype(np.float64), w[336:352].astype(np.float64)
    w3, b3 = w[352:384].reshape(2, 16).astype(np.float64), w[384:].astype(np.float64)
    zs = inputs.random_states(100, seed=8, spread="live")
    for i in range(zs.shape[1]):
        z = zs[:, i].astype(np.float64)
        want = w3 @ np.tanh(w2 @ np.tanh(w1 @ z + b1) + b2) + b3
        got = oracle.mlp_deep_logits(w, zs[:, i])
        assert np.all(np.abs(got - want) < 6e-6)
    # one path: input 2 -> first-layer unit j -> second-layer unit k -> both outputs
    for j, k in ((0, 15), (7, 3), (15, 0)):
        probe = np.zeros(386, np.float32)
        probe[4 * j + 2] = 1.5                 # W1[j][2]
        probe[64 + j] = 0.25                   # b1[j]
        probe[80 + 16 * k + j] = 2.0           # W2[k][j]
        probe[336 + k] = -0.125                # b2[k]
        probe[352 + k] = 1.0                   # W3[0][k]
        probe[352 + 16 + k] = -2.0             # W3[1][k]
        probe[384:] = (0.5, 0.75)
        got = oracle.mlp_deep_logits(probe, [9, 9, 0.2, 9])
        h2 = np.tanh(2.0 * np.tanh(1.5 * 0.2 + 0.25) - 0.125)
        assert abs(got[0] - (0.5 + h2)) < 1e-6 and abs(got[1] - (0.75 - 2 * h2)) < 1e-6
    # second layer = eps * identity: tanh(eps*h) ~ eps*h, so logits ~ b3 + eps * W3 h1, i.e. the
    # one-hidden-layer network with its output weights scaled by eps
    shallow = inputs.policy_weights(inputs.POLICY_MLP, 2)
    eps = 1e-3
    deep = np.zeros(386, np.float32)
    deep[:80] = shallow[:80]
    deep[80:336] = (eps * np.eye(16)).astype(np.float32).ravel()
    deep[352:384] = shallow[80:112]
    for i in range(20):
        a = oracle.mlp_logits(shallow, zs[:, i]) - shallow[112:]
        b = oracle.mlp_deep_logits(deep, zs[:, i])
        assert np.all(np.abs(b - eps * a) < 1e-8)
    # rollouts: the action is the argmax of the logits on the state BEFORE the step
    n, T = 32, 25
    r = oracle.rollout(n, T, 0, kind, w, trajectory=True, action_bits=True, min_gap=True)
    z = oracle.initial_state(n, 0)
    for t in range(T):
        ab = unpack_bits(r["action_bits"][t], n)
        for i in range(n):
            lg = oracle.mlp_deep_logits(w, z[:, i])
            assert ab[i] == int(lg[1] > lg[0])
        z = r["trajectory"][t]
    assert np.all(np.isfinite(r["min_gap"])) and 0 < unpack_bits(r["action_bits"], n).mean() < 1


def test_per_env_linear_policies(oracle):
    n, T, seed = 70, 40, 2
    kind = inputs.POLICY_LINEAR_PER_ENV
    wp = inputs.per_env_linear_weights(n, 5)
    assert wp.shape == (10, n)
    r = oracle.rollout(n, T, seed, kind, wp, trajectory=True, action_bits=True, done_bits=True, nthreads=3)
    # brute force: every env is a one-env rollout of the shared linear policy with its own column
    for i in range(0, n, 3):
        one = oracle.rollout(1, T, seed, inputs.POLICY_LINEAR, wp[:, i], env_offset=i, trajectory=True)
        assert np.array_equal(one["trajectory"][:, :, 0], r["trajectory"][:, :, i])
        assert one["ep_return_sum"][0] == r["ep_return_sum"][i] and one["ep_count"][0] == r["ep_count"][i]
    # the action at every step is the argmax of that env's own logits on the pre-step state
    z = oracle.initial_state(n, seed)
    for t in range(T):
        ab = unpack_bits(r["action_bits"][t], n)
        for i in range(n):
            lg = oracle.linear_logits(wp[:, i], z[:, i])
            assert ab[i] == int(lg[1] > lg[0])
        z = r["trajectory"][t]
    # identical columns reduce to the shared policy
    w = inputs.policy_weights(inputs.POLICY_LINEAR, 1)
    same = oracle.rollout(n, T, seed, kind, np.repeat(w[:, None], n, axis=1))
    shared = oracle.rollout(n, T, seed, inputs.POLICY_LINEAR, w)
    assert np.array_equal(same["ep_return_sum"], shared["ep_return_sum"])
    # policies differ between envs: so do the outcomes
    assert len(set(r["ep_return_sum"].tolist())) > 5
