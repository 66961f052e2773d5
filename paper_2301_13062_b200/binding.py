"""Thin ctypes binding of libcartpole.so: same names as the C ABI, argument
marshalling only. torch supplies device memory (tensors' ``data_ptr()``) and the
current CUDA stream; every step of the computation runs in the library's kernels.

There is no fallback: if the shared library is missing or cannot be loaded,
importing ``lib()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcartpole.so")

CP_OK, CP_EINVAL, CP_ECUDA, CP_ENOMEM = 0, -1, -2, -3
CP_POLICY_RANDOM, CP_POLICY_LINEAR, CP_POLICY_MLP, CP_POLICY_MLP32, CP_POLICY_MLP64 = 0, 1, 2, 4, 5
CP_POLICY_LINEAR_PER_ENV = 6
CP_POLICY_MLP_DEEP = 7
N_WEIGHTS = {CP_POLICY_RANDOM: 0, CP_POLICY_LINEAR: 10, CP_POLICY_MLP: 114, CP_POLICY_MLP32: 226,
             CP_POLICY_MLP64: 450, CP_POLICY_MLP_DEEP: 386}

# every symbol include/cartpole.h declares
EXPORTS = [
    "cp_reset", "cp_step", "cp_rollout", "cp_step_unfused", "cp_unfused_workspace_bytes", "cp_wrap",
    "cp_fill_start", "cp_set_time", "cp_free", "cp_state_info", "cp_actions", "cp_rollout_shard",
    "cp_rollout_from", "cp_rollout_host", "cp_step_host", "cp_shutdown", "cp_set_stream", "cp_tune",
    "cp_launch_count", "cp_selftest_sincos", "cp_last_error", "cp_version", "cp_step_unfused_noalloc",
    "cp_selftest_sincos_accuracy", "cp_selftest_arith", "cp_step_repeat", "cp_selftest_tame_div",
    "cp_rollout_ex", "cp_step_ex", "cp_rollout_host_shard", "cp_selftest_tanh", "cp_set_allocator",
    "cp_calibrate_pipe", "cp_selftest_pair",
]
CP_CALIBRATE_THREADS_PER_SM = 2048
CP_NOALLOC_MAX_ENVS = 65536


class cp_policy(C.Structure):
    _fields_ = [("kind", C.c_int32), ("weights", C.c_void_p)]


class cp_returns(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("ep_return_sum", "ep_count", "totals", "reward_stream", "done_bits",
                                          "action_bits", "final_state", "trajectory")]


class cp_rollout_args(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("env_offset", C.c_uint32), ("n_envs", C.c_int64), ("T", C.c_int64),
                ("seed", C.c_uint32), ("t0", C.c_uint32), ("policy", C.POINTER(cp_policy)),
                ("returns", C.POINTER(cp_returns)), ("state", C.c_void_p), ("ep_len", C.c_void_p),
                ("max_episode_steps", C.c_uint32), ("arithmetic", C.c_uint32), ("action_bits_in", C.c_void_p),
                ("start_states_in", C.c_void_p)]


CP_ARITH_EXACT, CP_ARITH_CONTRACTED = 0, 1


class CartpoleError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"libcartpole error {code}: {text}")
        self.code = code


_lib = None
ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t)
RELEASE_FN = C.CFUNCTYPE(None, C.c_void_p)
_allocator_callbacks = None  # keeps the ctypes thunks alive while the library may call them


def lib() -> C.CDLL:
    """Load libcartpole.so (built in-tree by ``python -m paper_2301_13062_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2301_13062_b200.build` "
                              "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        i64, u32, i32, p, sz = C.c_int64, C.c_uint32, C.c_int, C.c_void_p, C.c_size_t
        sig = {
            "cp_reset": (p, [i64, u32]),
            "cp_step": (i32, [p, p, p, p, p]),
            "cp_rollout": (i32, [i64, i64, u32, C.POINTER(cp_policy), C.POINTER(cp_returns)]),
            "cp_step_repeat": (i32, [p, i64, p, p]),
            "cp_rollout_ex": (i32, [C.POINTER(cp_rollout_args)]),
            "cp_step_ex": (i32, [p, p, p, p, p, p, u32]),
            "cp_step_unfused": (i32, [p, p, p, p, p, p, sz]),
            "cp_unfused_workspace_bytes": (sz, [i64]),
            "cp_step_unfused_noalloc": (i32, [p, p, p, p, p]),
            "cp_wrap": (p, [p, i64, i64, u32, u32, u32]),
            "cp_fill_start": (i32, [p]),
            "cp_set_time": (i32, [p, u32]),
            "cp_free": (None, [p]),
            "cp_state_info": (i32, [p, C.POINTER(i64), C.POINTER(i64), C.POINTER(u32), C.POINTER(u32),
                                    C.POINTER(u32), C.POINTER(p)]),
            "cp_actions": (i32, [i64, u32, u32, u32, p]),
            "cp_rollout_shard": (i32, [u32, i64, i64, u32, C.POINTER(cp_policy), C.POINTER(cp_returns)]),
            "cp_rollout_from": (i32, [p, i64, p, C.POINTER(cp_policy), C.POINTER(cp_returns)]),
            "cp_rollout_host": (i32, [i64, i64, u32, C.POINTER(cp_policy), p, p, p]),
            "cp_rollout_host_shard": (i32, [u32, i64, i64, u32, C.POINTER(cp_policy), p, p, p]),
            "cp_step_host": (i32, [i64, u32, u32, p, p, p, p, p]),
            "cp_shutdown": (None, []),
            "cp_set_stream": (None, [p]),
            "cp_set_allocator": (i32, [ALLOC_FN, RELEASE_FN]),
            "cp_tune": (i32, [C.c_char_p, i32]),
            "cp_launch_count": (C.c_uint64, []),
            "cp_selftest_sincos": (i32, [u32, u32, p]),
            "cp_selftest_sincos_accuracy": (i32, [u32, u32, p]),
            "cp_selftest_tanh": (i32, [u32, u32, p]),
            "cp_calibrate_pipe": (i64, [i32, p, p, i32]),
            "cp_selftest_arith": (i32, [p]),
            "cp_selftest_tame_div": (i32, [u32, p]),
            "cp_selftest_pair": (i32, [C.c_uint64, u32, p]),
            "cp_last_error": (C.c_char_p, []),
            "cp_version": (C.c_char_p, []),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != CP_OK:
        raise CartpoleError(rc, lib().cp_last_error().decode())


def _dptr(t, dtype=None):
    """Device address of a CUDA tensor (or None)."""
    if t is None:
        return None
    if not t.is_cuda:
        raise TypeError("expected a CUDA tensor")
    if not t.is_contiguous():
        raise TypeError("expected a contiguous tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _hptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        assert a.flags.c_contiguous
        return C.c_void_p(a.ctypes.data)
    assert not a.is_cuda and a.is_contiguous()
    return C.c_void_p(a.data_ptr())


def _use_current_stream() -> None:
    import torch
    lib().cp_set_stream(C.c_void_p(torch.cuda.current_stream().cuda_stream))


def cp_set_allocator(alloc=None, release=None) -> None:
    """Device allocator of cp_reset: two callables (bytes -> device address or 0, address -> None),
    or nothing for cudaMalloc / cudaFree. `use_torch_allocator()` passes torch's caching allocator."""
    global _allocator_callbacks
    if (alloc is None) != (release is None):
        raise ValueError("alloc and release go together")
    if alloc is None:
        _check(lib().cp_set_allocator(ALLOC_FN(0), RELEASE_FN(0)))
        return
    thunks = (ALLOC_FN(lambda n: alloc(n) or 0), RELEASE_FN(lambda ptr: release(ptr)))
    _check(lib().cp_set_allocator(*thunks))
    # never dropped: a live handle keeps the release function it was created under
    _allocator_callbacks = (_allocator_callbacks or []) + [thunks]


def use_torch_allocator(enable: bool = True) -> None:
    """Let cp_reset take its batches from torch's CUDA caching allocator (no cudaMalloc, hence no
    device-wide synchronisation, and the memory shows up in torch's own accounting)."""
    import torch
    if enable:
        cp_set_allocator(torch.cuda.caching_allocator_alloc, torch.cuda.caching_allocator_delete)
    else:
        cp_set_allocator(None, None)


class _Policy:
    """Keeps the host weight array alive while the C struct points at it."""

    def __init__(self, kind: int = CP_POLICY_RANDOM, weights=None):
        self.kind = int(kind)
        self.weights = None
        self.struct = cp_policy(self.kind, None)
        if self.kind == CP_POLICY_LINEAR_PER_ENV:
            # one linear policy per environment: a CUDA float32 tensor [10, n_envs], used in place
            if not (weights.is_cuda and weights.is_contiguous() and weights.dim() == 2 and weights.shape[0] == 10):
                raise ValueError("per-environment weights must be a contiguous CUDA tensor of shape [10, n_envs]")
            self.weights = weights
            self.struct.weights = weights.data_ptr()
        elif self.kind != CP_POLICY_RANDOM:
            self.weights = np.ascontiguousarray(weights, np.float32).ravel()
            if self.weights.size != N_WEIGHTS.get(self.kind, -1):
                raise ValueError(f"policy kind {kind} needs {N_WEIGHTS.get(self.kind)} weights, got {self.weights.size}")
            self.struct.weights = self.weights.ctypes.data

    def ref(self):
        return C.byref(self.struct)


def _returns_struct(ep_return_sum=None, ep_count=None, totals=None, reward_stream=None, done_bits=None,
                    action_bits=None, final_state=None, trajectory=None) -> cp_returns:
    import torch
    r = cp_returns()
    r.ep_return_sum = _dptr(ep_return_sum, torch.float32)
    r.ep_count = _dptr(ep_count, torch.int32)
    r.totals = _dptr(totals, torch.int64)
    r.reward_stream = _dptr(reward_stream, torch.float32)
    r.done_bits = _dptr(done_bits, torch.int32)
    r.action_bits = _dptr(action_bits, torch.int32)
    r.final_state = _dptr(final_state, torch.float32)
    r.trajectory = _dptr(trajectory, torch.float32)
    return r


class State:
    """Owner of a ``cp_state*`` handle (and of the torch tensor it wraps, if any)."""

    def __init__(self, handle: int, planes=None):
        if not handle:
            raise CartpoleError(CP_EINVAL, lib().cp_last_error().decode())
        self.handle = C.c_void_p(handle)
        self.planes = planes  # torch tensor kept alive when wrapped

    def info(self) -> dict:
        n, stride = C.c_int64(), C.c_int64()
        seed, t, off = C.c_uint32(), C.c_uint32(), C.c_uint32()
        ptr = C.c_void_p()
        _check(lib().cp_state_info(self.handle, C.byref(n), C.byref(stride), C.byref(seed), C.byref(t),
                                   C.byref(off), C.byref(ptr)))
        return {"n_envs": n.value, "plane_stride": stride.value, "seed": seed.value, "t": t.value,
                "env_offset": off.value, "planes": ptr.value}

    def close(self) -> None:
        if self.handle:
            lib().cp_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ------------------------------------------------------------------ C ABI, same names
def cp_reset(n_envs: int, seed: int) -> State:
    _use_current_stream()
    return State(lib().cp_reset(n_envs, seed))


def cp_wrap(planes, n_envs: int, seed: int, t: int = 0, env_offset: int = 0, plane_stride: int | None = None) -> State:
    """planes: CUDA float32 tensor holding the four planes; plane_stride defaults to planes.shape[-1]."""
    import torch
    if plane_stride is None:
        plane_stride = planes.shape[-1]
    assert planes.dtype == torch.float32 and planes.is_cuda
    return State(lib().cp_wrap(C.c_void_p(planes.data_ptr()), n_envs, plane_stride, seed, t, env_offset), planes)


def cp_fill_start(state: State) -> None:
    _use_current_stream()
    _check(lib().cp_fill_start(state.handle))


def cp_set_time(state: State, t: int) -> None:
    _check(lib().cp_set_time(state.handle, t))


def cp_free(state: State) -> None:
    state.close()


def cp_step(state: State, action, out_state: State, reward, done) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_step(state.handle, _dptr(action, torch.uint8), out_state.handle, _dptr(reward, torch.float32),
                         _dptr(done, torch.uint8)))


def cp_step_repeat(state: State, k: int, reward, done) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_step_repeat(state.handle, k, _dptr(reward, torch.float32), _dptr(done, torch.uint8)))


def cp_unfused_workspace_bytes(n_envs: int) -> int:
    return int(lib().cp_unfused_workspace_bytes(n_envs))


def cp_step_unfused(state: State, action, out_state: State, reward, done, workspace) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_step_unfused(state.handle, _dptr(action, torch.uint8), out_state.handle,
                                 _dptr(reward, torch.float32), _dptr(done, torch.uint8), _dptr(workspace),
                                 workspace.numel() * workspace.element_size()))


def cp_step_unfused_noalloc(state: State, action, out_state: State, reward, done) -> None:
    """The per-op step for callers that cannot allocate device memory (no workspace argument:
    the intermediates live in an array built into the library). At most CP_NOALLOC_MAX_ENVS
    environments; calls that overlap on the GPU race on that shared array."""
    import torch
    _use_current_stream()
    _check(lib().cp_step_unfused_noalloc(state.handle, _dptr(action, torch.uint8), out_state.handle,
                                         _dptr(reward, torch.float32), _dptr(done, torch.uint8)))


def cp_actions(n_envs: int, seed: int, t: int, env_offset: int, out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_actions(n_envs, seed, t, env_offset, _dptr(out, torch.uint8)))


def cp_rollout(n_envs: int, T: int, seed: int, policy: _Policy | None = None, **returns) -> None:
    cp_rollout_shard(0, n_envs, T, seed, policy, **returns)


def cp_rollout_shard(env_offset: int, n_envs: int, T: int, seed: int, policy: _Policy | None = None, **returns) -> None:
    _use_current_stream()
    r = _returns_struct(**returns)
    _check(lib().cp_rollout_shard(env_offset, n_envs, T, seed, policy.ref() if policy else None, C.byref(r)))


def cp_rollout_from(state: State, T: int, ep_len=None, policy: _Policy | None = None, **returns) -> None:
    import torch
    _use_current_stream()
    r = _returns_struct(**returns)
    _check(lib().cp_rollout_from(state.handle, T, _dptr(ep_len, torch.int32), policy.ref() if policy else None,
                                 C.byref(r)))


def cp_rollout_ex(*, n_envs: int = 0, T: int, seed: int = 0, t0: int = 0, env_offset: int = 0,
                  policy: _Policy | None = None, state: State | None = None, ep_len=None,
                  max_episode_steps: int = 0, action_bits_in=None, arithmetic: int = CP_ARITH_EXACT,
                  start_states_in=None, **returns) -> None:
    """General rollout: optional episode step limit, optional supplied action bit stream and
    start states ([T, 4, n] float32), choice of arithmetic, either from start states (n_envs,
    seed, t0, env_offset) or advancing `state` in place."""
    import torch
    _use_current_stream()
    r = _returns_struct(**returns)
    a = cp_rollout_args()
    a.struct_size = C.sizeof(cp_rollout_args)
    a.env_offset, a.n_envs, a.T, a.seed, a.t0 = env_offset, n_envs, T, seed, t0
    a.policy = C.pointer(policy.struct) if policy else None
    a.returns = C.pointer(r)
    a.state = state.handle if state is not None else None
    a.ep_len = _dptr(ep_len, torch.int32)
    a.max_episode_steps = max_episode_steps
    a.arithmetic = arithmetic
    a.action_bits_in = _dptr(action_bits_in, torch.int32)
    if start_states_in is not None:
        n = state.info()["n_envs"] if state is not None else n_envs
        assert tuple(start_states_in.shape) == (T, 4, n), "start_states_in must be [T, 4, n_envs]"
    a.start_states_in = _dptr(start_states_in, torch.float32)
    _check(lib().cp_rollout_ex(C.byref(a)))


def cp_step_ex(state: State, action, out_state: State, reward, done, ep_len, max_episode_steps: int = 0) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_step_ex(state.handle, _dptr(action, torch.uint8), out_state.handle, _dptr(reward, torch.float32),
                            _dptr(done, torch.uint8), _dptr(ep_len, torch.int32), max_episode_steps))


def cp_rollout_host(n_envs: int, T: int, seed: int, policy: _Policy | None, h_ep_return_sum, h_ep_count, h_totals) -> None:
    cp_rollout_host_shard(0, n_envs, T, seed, policy, h_ep_return_sum, h_ep_count, h_totals)


def cp_rollout_host_shard(env_offset: int, n_envs: int, T: int, seed: int, policy: _Policy | None,
                          h_ep_return_sum, h_ep_count, h_totals) -> None:
    _use_current_stream()
    _check(lib().cp_rollout_host_shard(env_offset, n_envs, T, seed, policy.ref() if policy else None,
                                       _hptr(h_ep_return_sum), _hptr(h_ep_count), _hptr(h_totals)))


def cp_step_host(n_envs: int, seed: int, t: int, h_planes_in, h_action, h_planes_out, h_reward, h_done) -> None:
    _use_current_stream()
    _check(lib().cp_step_host(n_envs, seed, t, _hptr(h_planes_in), _hptr(h_action), _hptr(h_planes_out),
                              _hptr(h_reward), _hptr(h_done)))


def cp_shutdown() -> None:
    lib().cp_shutdown()


def cp_tune(key: str, value: int) -> None:
    _check(lib().cp_tune(key.encode(), value))


def cp_launch_count() -> int:
    return int(lib().cp_launch_count())


def cp_selftest_sincos(lo_bits: int, hi_bits: int, mismatches) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_sincos(lo_bits, hi_bits, _dptr(mismatches, torch.int64)))


def cp_selftest_sincos_accuracy(lo_bits: int, hi_bits: int, out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_sincos_accuracy(lo_bits, hi_bits, _dptr(out, torch.int64)))


def cp_selftest_tanh(lo_bits: int, hi_bits: int, out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_tanh(lo_bits, hi_bits, _dptr(out, torch.int64)))


def cp_calibrate_pipe(kind: int, seed, sink, iters: int) -> int:
    """Enqueue the calibration launch; returns the thread-instructions it executes."""
    import torch
    _use_current_stream()
    n = lib().cp_calibrate_pipe(kind, _dptr(seed, torch.float32), _dptr(sink, torch.float32), iters)
    if n < 0:
        _check(int(n))
    return int(n)


def cp_selftest_arith(out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_arith(_dptr(out, torch.int64)))


def cp_selftest_tame_div(den_step: int, out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_tame_div(den_step, _dptr(out, torch.int64)))


def cp_selftest_pair(count: int, seed: int, out) -> None:
    import torch
    _use_current_stream()
    _check(lib().cp_selftest_pair(count, seed, _dptr(out, torch.int64)))


def cp_version() -> str:
    return lib().cp_version().decode()


def policy(kind: int = CP_POLICY_RANDOM, weights=None) -> _Policy:
    return _Policy(kind, weights)
