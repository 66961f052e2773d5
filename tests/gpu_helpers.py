"""Helpers of the GPU parity tests: comparison rules against the CPU oracle.

Tolerances (stated by the benchmark spec, written out here):
  * actions, done flags, rewards, start states: bit-exact, except that a done flag is
    excused where the oracle's post-update |x| or |theta| lies within 1e-5 of its
    termination threshold (a last-bit sine/cosine difference may flip it);
  * float32 state after ONE step from the same input state: relative error <= 2e-6,
    measured against max(|reference|, |input component|, tau*|rate|) so that a
    component passing through zero is judged on the scale of the update;
  * free-running rollouts: per-env episode returns identical on >= 99.9 % of envs,
    mean return within 0.1 %; envs whose policy logits come within 1e-5 of a tie
    are excused like threshold-band envs.
"""
import contextlib

import numpy as np

XT = np.float32(2.4)
TT = np.float32(12 * 2 * np.pi / 360)
TAU = np.float32(0.02)
BAND = 1e-5
REL_TOL = 2e-6


# The rollout kernel's work shapes as (rollout_ept, rollout_coop) tuning values: one env per
# thread with per-lane restarts, the same with start states computed ahead every step, one env
# per thread with restarts by the whole warp, two envs per thread (always by the warp), and the
# kernel whose helper warps hash actions and start states ahead of the stepping warps (it covers
# hashed actions without streams or step limit; other calls fall to the first shape). The
# library picks one by batch size and policy; tests force each of them on small batches.
SHAPES = [(1, 2), (1, 3), (1, 1), (2, 1), (1, 4), (2, 5)]


@contextlib.contextmanager
def rollout_shape(cp, ept: int, coop: int):
    cp.cp_tune("rollout_ept", ept)
    cp.cp_tune("rollout_coop", coop)
    try:
        yield
    finally:
        cp.cp_tune("rollout_ept", 0)
        cp.cp_tune("rollout_coop", 0)


def band_mask(pre_reset: np.ndarray) -> np.ndarray:
    """Envs whose updated x or theta is within BAND of a threshold (oracle values)."""
    return (np.abs(np.abs(pre_reset[0].astype(np.float64)) - float(XT)) <= BAND) | \
           (np.abs(np.abs(pre_reset[2].astype(np.float64)) - float(TT)) <= BAND)


def assert_step_matches(oracle_res: dict, z_in: np.ndarray, gpu_state: np.ndarray, gpu_reward: np.ndarray,
                        gpu_done: np.ndarray, gpu_action: np.ndarray | None = None) -> dict:
    """Teacher-forced comparison of one step. Returns counts for reporting."""
    pre = oracle_res["pre_reset"]
    band = band_mask(pre)
    if gpu_action is not None:
        assert np.array_equal(gpu_action, oracle_res["action"]), "actions differ"
    assert np.array_equal(gpu_reward, oracle_res["reward"]), "rewards differ"
    dd = gpu_done != oracle_res["done"]
    assert not np.any(dd & ~band), f"done differs outside the threshold band at {np.nonzero(dd & ~band)[0][:8]}"
    agree = ~dd
    both_done = agree & (oracle_res["done"] == 1)
    live = agree & (oracle_res["done"] == 0)
    # finished envs restart from the hashed start state: bit-exact
    assert np.array_equal(gpu_state[:, both_done].view(np.uint32), oracle_res["state"][:, both_done].view(np.uint32))
    # live envs: relative tolerance on the scale of value, input and update
    ref = oracle_res["state"].astype(np.float64)
    rate = np.stack([z_in[1], (ref[1] - z_in[1]) / float(TAU), z_in[3], (ref[3] - z_in[3]) / float(TAU)])
    scale = np.maximum(np.maximum(np.abs(ref), np.abs(z_in)), float(TAU) * np.abs(rate))
    err = np.abs(gpu_state.astype(np.float64) - ref)
    finite = np.isfinite(ref).all(axis=0) & live
    bad = (err > REL_TOL * scale)[:, finite]
    assert not bad.any(), f"state error above {REL_TOL} relative: max {np.max((err / np.maximum(scale, 1e-30))[:, finite])}"
    exact = float(np.mean(gpu_state[:, live].view(np.uint32) == oracle_res["state"][:, live].view(np.uint32))) \
        if live.any() else 1.0
    return {"band": int(band.sum()), "done_flips": int(dd.sum()), "bit_exact_fraction": exact}


def assert_returns_match(gpu_ret: np.ndarray, gpu_cnt: np.ndarray, ora_ret: np.ndarray, ora_cnt: np.ndarray,
                         excuse: np.ndarray | None = None, min_identical: float = 0.999,
                         mean_rel: float = 1e-3) -> dict:
    same = (gpu_ret == ora_ret) & (gpu_cnt == ora_cnt)
    frac = float(same.mean())
    frac_excused = float((same | excuse).mean()) if excuse is not None else frac
    assert frac_excused >= min_identical, f"only {frac_excused:.6f} of envs have identical returns"
    g = gpu_ret.astype(np.float64).sum() / max(1, int(gpu_cnt.astype(np.int64).sum()))
    o = ora_ret.astype(np.float64).sum() / max(1, int(ora_cnt.astype(np.int64).sum()))
    assert abs(g - o) <= mean_rel * o, f"mean return {g} vs {o}"
    return {"identical": frac, "identical_or_excused": frac_excused, "mean_gpu": g, "mean_oracle": o}


def unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    """[T, ceil(n/32)] uint32 -> [T, n] uint8 (bit i%32 of word i/32)."""
    w = np.ascontiguousarray(words).view(np.uint32)
    return np.unpackbits(w.view(np.uint8), bitorder="little", axis=-1)[..., :n]
