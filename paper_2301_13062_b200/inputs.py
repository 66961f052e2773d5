"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds none of the CartPole arithmetic and none of the counter hash:
it only draws numbers with numpy's PCG64 generator and names the benchmark
workloads. Both the CUDA library and the CPU oracle are fed from here, so
neither side ever produces an input for the other.

Workloads follow the paper's evaluation shape (Sec. V: N parallel environments
stepped T times, random actions, random start states, float32); the start
states and random actions themselves are functions of (seed, env, step) that
each side computes on its own, so a workload is fully named by
``(n_envs, T, seed, policy)``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

POLICY_RANDOM, POLICY_LINEAR, POLICY_MLP, POLICY_MLP32, POLICY_MLP64 = 0, 1, 2, 4, 5
POLICY_MLP_DEEP = 7  # 4 -> 16 (tanh) -> 16 (tanh) -> 2
N_WEIGHTS = {POLICY_RANDOM: 0, POLICY_LINEAR: 10, POLICY_MLP: 114, POLICY_MLP32: 226, POLICY_MLP64: 450,
             POLICY_MLP_DEEP: 386}
MLP_HIDDEN = 16
HIDDEN_OF = {POLICY_MLP: 16, POLICY_MLP32: 32, POLICY_MLP64: 64}
POLICY_LINEAR_PER_ENV = 6  # a different linear policy for every environment (population search)


@dataclass(frozen=True)
class Workload:
    name: str
    n_envs: int
    T: int
    seed: int
    policy: int
    policy_seed: int
    path: str          # "step" (per-step launches), "rollout" (one launch)
    streams: bool      # per-step reward plane + done bitmask written to HBM


# The five benchmark configurations plus the paper's own batch shape (Sec. V:
# 2,048 environments x 10,000 steps), kept as context.
WORKLOADS = {
    "c1": Workload("c1", 1_024, 200, 0, POLICY_RANDOM, 0, "rollout", False),
    "c2": Workload("c2", 65_536, 1_000, 0, POLICY_RANDOM, 0, "step", False),
    "c3": Workload("c3", 1_048_576, 500, 0, POLICY_RANDOM, 0, "rollout", False),
    "c4": Workload("c4", 4_194_304, 1_000, 0, POLICY_LINEAR, 1, "rollout", True),
    "c5": Workload("c5", 16_777_216, 200, 0, POLICY_MLP, 2, "rollout", False),
    "paper": Workload("paper", 2_048, 10_000, 0, POLICY_RANDOM, 0, "rollout", False),
}


def policy_weights(kind: int, seed: int) -> np.ndarray:
    """Flat float32 policy parameters drawn once on the host.

    linear (10): W[2][4] then b[2], all N(0, std=0.5).
    MLP (114): W1[16][4], b1[16] with std 1/sqrt(4)=0.5, then W2[2][16], b2[2]
    with std 1/sqrt(16)=0.25 (std = 1/sqrt(fan_in), biases like their layer).
    """
    rng = np.random.default_rng(seed)
    if kind == POLICY_RANDOM:
        return np.zeros(0, np.float32)
    if kind == POLICY_LINEAR:
        return (0.5 * rng.standard_normal(10)).astype(np.float32)
    if kind in HIDDEN_OF:  # W1[H][4], b1[H] with std 1/sqrt(4); W2[2][H], b2[2] with std 1/sqrt(H)
        h = HIDDEN_OF[kind]
        l1 = 0.5 * rng.standard_normal(4 * h + h)
        l2 = (1.0 / np.sqrt(h)) * rng.standard_normal(2 * h + 2)
        return np.concatenate([l1, l2]).astype(np.float32)
    if kind == POLICY_MLP_DEEP:  # W1[16][4], b1[16]; W2[16][16], b2[16]; W3[2][16], b3[2]; std 1/sqrt(fan_in)
        l1 = 0.5 * rng.standard_normal(64 + 16)
        l2 = 0.25 * rng.standard_normal(256 + 16)
        l3 = 0.25 * rng.standard_normal(32 + 2)
        return np.concatenate([l1, l2, l3]).astype(np.float32)
    raise ValueError(f"unknown policy kind {kind}")


def per_env_linear_weights(n: int, seed: int) -> np.ndarray:
    """float32 [10, n]: one linear policy per environment, parameter-major (row q holds parameter
    q of every env: rows 0-7 the 2x4 matrix row-major, rows 8-9 the biases), all N(0, std=0.5)."""
    return (0.5 * np.random.default_rng(seed).standard_normal((10, n))).astype(np.float32)


def random_states(n: int, seed: int, spread: str = "live") -> np.ndarray:
    """float32 [4, n] states (x, x_dot, theta, theta_dot).

    "start": U(-0.05, 0.05) on every component (the start-state distribution).
    "live":  anywhere inside the termination box with episode-like velocities.
    "edge":  positions/angles within a few percent of the thresholds and rates of
             either sign, so that a good share of the next states terminate.
    "wide":  large angles and speeds, outside anything an episode reaches.
    """
    rng = np.random.default_rng(seed)
    if spread == "start":
        z = rng.uniform(-0.05, 0.05, (4, n))
    elif spread == "live":
        z = np.stack([rng.uniform(-2.4, 2.4, n), rng.uniform(-2.5, 2.5, n),
                      rng.uniform(-0.2094, 0.2094, n), rng.uniform(-3.0, 3.0, n)])
    elif spread == "edge":
        sx = rng.choice([-1.0, 1.0], n)
        st = rng.choice([-1.0, 1.0], n)
        z = np.stack([sx * rng.uniform(2.3, 2.4, n), rng.uniform(-3.0, 3.0, n),
                      st * rng.uniform(0.19, 0.2094, n), rng.uniform(-0.6, 0.6, n)])
    elif spread == "wide":
        z = np.stack([rng.uniform(-10, 10, n), rng.uniform(-20, 20, n),
                      rng.uniform(-7, 7, n), rng.uniform(-20, 20, n)])
    else:
        raise ValueError(spread)
    return np.ascontiguousarray(z, np.float32)


def random_actions(n: int, seed: int) -> np.ndarray:
    """uint8 [n] of 0/1 actions for the supplied-action form of the step."""
    return np.random.default_rng(seed).integers(0, 2, n, dtype=np.uint8)


def shard_range(n_total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous env range [lo, hi) of `rank`; ranges are multiples of 32 envs
    (one done-bit word) except possibly the last."""
    words = (n_total + 31) // 32
    per = (words + world - 1) // world
    lo = min(n_total, rank * per * 32)
    hi = min(n_total, (rank + 1) * per * 32)
    return lo, hi
