"""Out-of-bounds write detection without a sanitizer: every output of every kernel family is
placed inside a larger buffer filled with a sentinel, at sizes that leave ragged tails in every
unit the kernels work in (4 envs per vector, 32 per warp, 64 per two-env warp, 256 per CTA), and
the guard regions before and after — and the unused tail of every odd-stride plane — must come
back untouched. (Reads cannot be caught this way; the state planes' pad lanes are initialised so
that a vector load past n_envs reads defined values.)"""
import numpy as np
import pytest

from paper_2301_13062_b200 import inputs
from tests import gpu_helpers as H

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

PAD = 256           # guard bytes on either side
SENTINEL = 0xA5     # every guard byte


@pytest.fixture(scope="module")
def cp():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2301_13062_b200 import binding, build
    build.build()
    binding.lib()
    torch.cuda.set_device(0)
    return binding


class Guarded:
    """A tensor of `shape` in the middle of a sentinel-filled byte buffer."""

    def __init__(self, shape, dtype):
        self.numel = int(np.prod(shape))
        self.item = torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((2 * PAD + self.numel * self.item,), SENTINEL, dtype=torch.uint8, device="cuda")
        self.t = self.raw[PAD:PAD + self.numel * self.item].view(dtype).view(*shape)

    def check(self, name):
        raw = self.raw.cpu().numpy()
        lo, hi = raw[:PAD], raw[PAD + self.numel * self.item:]
        assert (lo == SENTINEL).all(), f"{name}: write before the buffer"
        assert (hi == SENTINEL).all(), f"{name}: write past the buffer"


def check_plane_tails(g, n, name, allowed=None):
    """Plane p of a [4, stride] batch may be written in [0, allowed) only (allowed defaults to n)."""
    allowed = n if allowed is None else allowed
    raw = g.t.cpu().numpy().view(np.uint8).reshape(g.t.shape[0], -1)
    assert (raw[:, allowed * 4:] == SENTINEL).all(), f"{name}: write into the tail of a plane"
    g.check(name)


SIZES = [1, 31, 33, 1025, 4164, 70001]


@pytest.mark.parametrize("n", SIZES)
def test_step_and_ladder_stay_inside_their_outputs(cp, n):
    z = inputs.random_states(n, seed=n, spread="edge")
    r4 = (n + 3) // 4 * 4
    for stride, vec_min in ((n + 5, 0), (r4 + 8, 0), (r4 + 8, 1 << 30)):
        cp.cp_tune("step_vec_min_envs", vec_min)
        try:
            src = torch.zeros(4, stride, device="cuda")
            src[:, :n] = torch.from_numpy(z).cuda()
            dst, reward, done = Guarded((4, stride), torch.float32), Guarded((n,), torch.float32), Guarded((n,), torch.uint8)
            ep_len = Guarded((n,), torch.int32)
            ep_len.t.zero_()
            s_in, s_out = cp.cp_wrap(src, n, 3, 5), cp.cp_wrap(dst.t, n, 3, 5)
            cp.cp_step(s_in, None, s_out, reward.t, done.t)
            cp.cp_set_time(s_in, 5)
            cp.cp_step_ex(s_in, None, s_out, reward.t, done.t, ep_len.t, 7)
            torch.cuda.synchronize()
            # the four-envs-per-thread kernel may fill the pad lanes up to a multiple of four
            vector_form = stride % 4 == 0 and vec_min == 0
            check_plane_tails(dst, n, "step out_state", r4 if vector_form else n)
            reward.check("step reward"), done.check("step done"), ep_len.check("step ep_len")
            assert done.t.sum().item() > 0 or n < 5
        finally:
            cp.cp_tune("step_vec_min_envs", 262144)
    # the per-op ladder (needs stride % 4 == 0): outputs and its workspace
    stride = r4 + 8
    src = torch.zeros(4, stride, device="cuda")
    src[:, :n] = torch.from_numpy(z).cuda()
    dst, reward, done = Guarded((4, stride), torch.float32), Guarded((n,), torch.float32), Guarded((n,), torch.uint8)
    ws = Guarded((cp.cp_unfused_workspace_bytes(n),), torch.uint8)
    assert ws.t.data_ptr() % 256 == 0
    cp.cp_step_unfused(cp.cp_wrap(src, n, 3, 5), None, cp.cp_wrap(dst.t, n, 3, 5), reward.t, done.t, ws.t)
    torch.cuda.synchronize()
    check_plane_tails(dst, n, "ladder out_state", r4)
    reward.check("ladder reward"), done.check("ladder done"), ws.check("ladder workspace")


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("shape", H.SHAPES)
def test_rollouts_stay_inside_their_outputs(cp, n, shape):
    T, words = 37, (n + 31) // 32
    w = inputs.policy_weights(1, 1)
    for kind, streams, limit in ((0, True, 0), (0, False, 0), (1, False, 11), (1, True, 0), (0, "rd", 9)):
        out = {"ep_return_sum": Guarded((n,), torch.float32), "ep_count": Guarded((n,), torch.int32),
               "totals": Guarded((2,), torch.int64), "final_state": Guarded((4, n), torch.float32)}
        if streams is True:
            out.update(reward_stream=Guarded((T, n), torch.float32), done_bits=Guarded((T, words), torch.int32),
                       action_bits=Guarded((T, words), torch.int32), trajectory=Guarded((T, 4, n), torch.float32))
        elif streams == "rd":   # the reward plane + done bitmask instance
            out.update(reward_stream=Guarded((T, n), torch.float32), done_bits=Guarded((T, words), torch.int32))
        out["totals"].t.zero_()
        with H.rollout_shape(cp, *shape):
            cp.cp_rollout_ex(n_envs=n, T=T, seed=2, env_offset=3, policy=cp.policy(1, w) if kind else None,
                             max_episode_steps=limit, **{k: g.t for k, g in out.items()})
        torch.cuda.synchronize()
        for k, g in out.items():
            g.check(f"rollout {k} (policy {kind}, streams {streams}, limit {limit})")
        assert int(out["totals"].t[1]) == int(out["ep_count"].t.sum())
        if streams:
            assert not (n % 32) or not np.any(out["done_bits"].t.cpu().numpy().view(np.uint32)[:, -1] >> (n % 32))
    # in place from a caller's batch with an odd plane stride, carried episode lengths in and out
    stride = n + 5
    planes, ep_len = Guarded((4, stride), torch.float32), Guarded((n,), torch.int32)
    planes.t[:, :n] = torch.from_numpy(inputs.random_states(n, seed=1, spread="live")).cuda()
    ep_len.t.zero_()
    ret = Guarded((n,), torch.float32)
    with H.rollout_shape(cp, *shape):
        cp.cp_rollout_ex(T=T, state=cp.cp_wrap(planes.t, n, 4, 9), ep_len=ep_len.t, ep_return_sum=ret.t)
    torch.cuda.synchronize()
    check_plane_tails(planes, n, "rollout state planes")
    ep_len.check("rollout ep_len"), ret.check("rollout ep_return_sum (from state)")
