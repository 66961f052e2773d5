"""ctypes loader for the scalar CPU oracle (``cartpole_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline leg use this; the CUDA library and its Python binding never do.

The functions here only marshal numpy arrays; all arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cartpole_oracle.c")
_LIB = os.path.join(_HERE, "libcartpole_oracle.so")

POLICY_RANDOM, POLICY_LINEAR, POLICY_MLP, POLICY_MLP32, POLICY_MLP64 = 0, 1, 2, 4, 5
POLICY_LINEAR_PER_ENV = 6
POLICY_MLP_DEEP = 7
N_WEIGHTS = {POLICY_RANDOM: 0, POLICY_LINEAR: 10, POLICY_MLP: 114, POLICY_MLP32: 226, POLICY_MLP64: 450,
             POLICY_MLP_DEEP: 386}


def build(force: bool = False) -> str:
    """Compile the oracle with strict float32 semantics (no contraction, no fast-math)."""
    import hashlib
    with open(_SRC, "rb") as f:
        want = hashlib.sha256(f.read()).hexdigest()
    stamp = _LIB + ".stamp"
    have = open(stamp).read().strip() if os.path.exists(stamp) else ""
    if force or not os.path.exists(_LIB) or have != want:  # content hash, not file times
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-o", _LIB + ".tmp", _SRC, "-lm", "-lpthread"]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
        with open(stamp, "w") as f:
            f.write(want + "\n")
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u32, i64, i32 = C.c_uint32, C.c_int64, C.c_int
        p = C.c_void_p
        L.co_mix32.restype = u32
        L.co_mix32.argtypes = [u32]
        L.co_salt.restype = u32
        L.co_salt.argtypes = [u32, u32]
        L.co_keys.restype = None
        L.co_keys.argtypes = [u32, u32, u32, C.POINTER(u32), C.POINTER(u32)]
        L.co_step_hash.restype = u32
        L.co_step_hash.argtypes = [u32, u32, u32]
        L.co_action.restype = u32
        L.co_action.argtypes = [u32, u32, u32]
        L.co_reset_state.restype = None
        L.co_reset_state.argtypes = [u32, u32, u32, p]
        L.co_accel_f32.restype = None
        L.co_accel_f32.argtypes = [p, i32, p, p]
        L.co_dynamics_f32.restype = i32
        L.co_dynamics_f32.argtypes = [p, i32, p]
        L.co_accel_f64.restype = None
        L.co_accel_f64.argtypes = [p, i32, p, p]
        L.co_dynamics_f64.restype = i32
        L.co_dynamics_f64.argtypes = [p, i32, p]
        L.co_linear_logits.restype = None
        L.co_linear_logits.argtypes = [p, p, p]
        L.co_mlp_logits.restype = None
        L.co_mlp_logits.argtypes = [p, p, p]
        L.co_mlp_logits_wide.restype = None
        L.co_mlp_logits_wide.argtypes = [p, i32, p, p]
        L.co_mlp_deep_logits.restype = None
        L.co_mlp_deep_logits.argtypes = [p, p, p]
        L.co_step.restype = None
        L.co_step.argtypes = [u32, i64, i64, i64, u32, u32, p, p, p, p, p, p, p]
        L.co_rollout.restype = None
        L.co_rollout.argtypes = [u32, i64, i64, u32, u32, i32, p, p, p, p, p, p, p, p, p, p, p, p, i32]
        L.co_rollout_ex.restype = None
        L.co_rollout_ex.argtypes = [u32, i64, i64, u32, u32, i32, p, p, p, p, p, p, p, p, p, p, p, p, i32, u32, p, p, p]
        L.co_step_limited.restype = None
        L.co_step_limited.argtypes = [u32, i64, i64, i64, u32, u32, p, p, p, p, p, p, u32]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ----------------------------------------------------------------- hash
def mix32(h: int) -> int:
    return int(lib().co_mix32(h & 0xFFFFFFFF))


def salt(seed: int, stream: int) -> int:
    return int(lib().co_salt(seed, stream))


def keys(seed: int, env: int, stream: int) -> tuple[int, int]:
    k0, k1 = C.c_uint32(), C.c_uint32()
    lib().co_keys(seed, env, stream, C.byref(k0), C.byref(k1))
    return int(k0.value), int(k1.value)


def step_hash(k0: int, k1: int, c: int) -> int:
    return int(lib().co_step_hash(k0, k1, c & 0xFFFFFFFF))


def action(seed: int, env: int, t: int) -> int:
    return int(lib().co_action(seed, env, t))


def reset_state(seed: int, env: int, t: int) -> np.ndarray:
    out = np.empty(4, np.float32)
    lib().co_reset_state(seed, env, t, _ptr(out))
    return out


# ------------------------------------------------------------- dynamics
def accel_f32(z, a: int) -> tuple[np.float32, np.float32]:
    z = np.ascontiguousarray(z, np.float32)
    xa, ta = np.empty(1, np.float32), np.empty(1, np.float32)
    lib().co_accel_f32(_ptr(z), int(a), _ptr(xa), _ptr(ta))
    return xa[0], ta[0]


def dynamics_f32(z, a: int) -> tuple[np.ndarray, bool]:
    z = np.ascontiguousarray(z, np.float32)
    out = np.empty(4, np.float32)
    d = lib().co_dynamics_f32(_ptr(z), int(a), _ptr(out))
    return out, bool(d)


def accel_f64(z, a: int) -> tuple[float, float]:
    z = np.ascontiguousarray(z, np.float64)
    xa, ta = np.empty(1, np.float64), np.empty(1, np.float64)
    lib().co_accel_f64(_ptr(z), int(a), _ptr(xa), _ptr(ta))
    return float(xa[0]), float(ta[0])


def dynamics_f64(z, a: int) -> tuple[np.ndarray, bool]:
    z = np.ascontiguousarray(z, np.float64)
    out = np.empty(4, np.float64)
    d = lib().co_dynamics_f64(_ptr(z), int(a), _ptr(out))
    return out, bool(d)


def linear_logits(w, z) -> np.ndarray:
    w = np.ascontiguousarray(w, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    assert w.size == 10
    out = np.empty(2, np.float32)
    lib().co_linear_logits(_ptr(w), _ptr(z), _ptr(out))
    return out


def mlp_logits(w, z) -> np.ndarray:
    w = np.ascontiguousarray(w, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    assert w.size == 114
    out = np.empty(2, np.float32)
    lib().co_mlp_logits(_ptr(w), _ptr(z), _ptr(out))
    return out


def mlp_logits_wide(w, hidden: int, z) -> np.ndarray:
    w = np.ascontiguousarray(w, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    assert w.size == 7 * hidden + 2
    out = np.empty(2, np.float32)
    lib().co_mlp_logits_wide(_ptr(w), int(hidden), _ptr(z), _ptr(out))
    return out


def mlp_deep_logits(w, z) -> np.ndarray:
    w = np.ascontiguousarray(w, np.float32)
    z = np.ascontiguousarray(z, np.float32)
    assert w.size == 386
    out = np.empty(2, np.float32)
    lib().co_mlp_deep_logits(_ptr(w), _ptr(z), _ptr(out))
    return out


# ---------------------------------------------------------------- batch
def step(planes: np.ndarray, seed: int, t: int, action_u8: np.ndarray | None = None,
         env_offset: int = 0, want_pre_reset: bool = False) -> dict:
    """One batched step. ``planes`` is float32 [4, n] (x, x_dot, theta, theta_dot)."""
    planes = np.ascontiguousarray(planes, np.float32)
    assert planes.ndim == 2 and planes.shape[0] == 4
    n = planes.shape[1]
    out = np.empty((4, n), np.float32)
    reward = np.empty(n, np.float32)
    done = np.empty(n, np.uint8)
    act = np.empty(n, np.uint8)
    pre = np.empty((4, n), np.float32) if want_pre_reset else None
    if action_u8 is not None:
        action_u8 = np.ascontiguousarray(action_u8, np.uint8)
        assert action_u8.size == n
    lib().co_step(env_offset, n, n, n, seed, t, _ptr(planes), _ptr(action_u8), _ptr(out),
                  _ptr(reward), _ptr(done), _ptr(act), _ptr(pre))
    return {"state": out, "reward": reward, "done": done, "action": act, "pre_reset": pre}


def initial_state(n: int, seed: int, t: int = 0, env_offset: int = 0) -> np.ndarray:
    out = np.empty((4, n), np.float32)
    for i in range(n):
        out[:, i] = reset_state(seed, env_offset + i, t)
    return out


def rollout(n: int, T: int, seed: int, policy_kind: int = POLICY_RANDOM, weights=None, *,
            env_offset: int = 0, t0: int = 0, init_state: np.ndarray | None = None,
            ep_len: np.ndarray | None = None, per_env: bool = True,
            reward_stream: bool = False, done_bits: bool = False,
            action_bits: bool = False, final_state: bool = False, trajectory: bool = False,
            min_gap: bool = False, min_margin: bool = False, nthreads: int = 1, max_episode_steps: int = 0,
            action_bits_in: np.ndarray | None = None, start_states_in: np.ndarray | None = None) -> dict:
    """Rollout of n envs for T steps. Returns a dict of the requested outputs.

    max_episode_steps > 0 cuts episodes off at that length; action_bits_in ([T, ceil(n/32)]
    uint32, bit i%32 of word i//32) supplies the actions instead of the policy;
    start_states_in (float32 [T, 4, n]) supplies the start states: an env that finishes at the
    k-th step of the call continues from row k instead of the hashed start state.
    min_gap / min_margin report, per env, the smallest policy logit gap and the smallest distance
    of an updated |x| or |theta| from its termination threshold seen during the rollout."""
    w = None
    if policy_kind != POLICY_RANDOM:
        w = np.ascontiguousarray(weights, np.float32).ravel()
        # kind 6: one linear policy per environment, weights [10, n] (parameter-major)
        assert w.size == (10 * n if policy_kind == POLICY_LINEAR_PER_ENV else N_WEIGHTS[policy_kind])
    words = (n + 31) // 32
    res = {
        "ep_return_sum": np.empty(n, np.float32) if per_env else None,
        "ep_count": np.empty(n, np.uint32) if per_env else None,
        "totals": np.zeros(2, np.uint64),
        "reward_stream": np.empty((T, n), np.float32) if reward_stream else None,
        "done_bits": np.zeros((T, words), np.uint32) if done_bits else None,
        "action_bits": np.zeros((T, words), np.uint32) if action_bits else None,
        "final_state": np.empty((4, n), np.float32) if final_state else None,
        "trajectory": np.empty((T, 4, n), np.float32) if trajectory else None,
        "min_gap": np.empty(n, np.float32) if min_gap else None,
        "min_margin": np.empty(n, np.float32) if min_margin else None,
    }
    if init_state is not None:
        init_state = np.ascontiguousarray(init_state, np.float32)
        assert init_state.shape == (4, n)
    if ep_len is not None:
        ep_len = np.ascontiguousarray(ep_len, np.uint32).copy()
        assert ep_len.size == n
        res["ep_len"] = ep_len
    if action_bits_in is not None:
        action_bits_in = np.ascontiguousarray(action_bits_in).view(np.uint32)
        assert action_bits_in.shape == (T, words)
    if start_states_in is not None:
        start_states_in = np.ascontiguousarray(start_states_in, np.float32)
        assert start_states_in.shape == (T, 4, n)
    lib().co_rollout_ex(env_offset, n, T, seed, t0, policy_kind, _ptr(w), _ptr(init_state), _ptr(ep_len),
                        _ptr(res["ep_return_sum"]), _ptr(res["ep_count"]), _ptr(res["totals"]),
                        _ptr(res["reward_stream"]), _ptr(res["done_bits"]), _ptr(res["action_bits"]),
                        _ptr(res["final_state"]), _ptr(res["trajectory"]), _ptr(res["min_gap"]),
                        int(nthreads), int(max_episode_steps), _ptr(action_bits_in), _ptr(start_states_in),
                        _ptr(res["min_margin"]))
    return res


def step_limited(planes: np.ndarray, seed: int, t: int, ep_len: np.ndarray, max_episode_steps: int,
                 action_u8: np.ndarray | None = None, env_offset: int = 0) -> dict:
    """One batched step with an episode step limit; ep_len (uint32 [n]) is carried in and out."""
    planes = np.ascontiguousarray(planes, np.float32)
    n = planes.shape[1]
    out = np.empty((4, n), np.float32)
    reward = np.empty(n, np.float32)
    done = np.empty(n, np.uint8)
    ep_len = np.ascontiguousarray(ep_len, np.uint32).copy()
    if action_u8 is not None:
        action_u8 = np.ascontiguousarray(action_u8, np.uint8)
    lib().co_step_limited(env_offset, n, n, n, seed, t, _ptr(planes), _ptr(action_u8), _ptr(out), _ptr(reward),
                          _ptr(done), _ptr(ep_len), int(max_episode_steps))
    return {"state": out, "reward": reward, "done": done, "ep_len": ep_len}
