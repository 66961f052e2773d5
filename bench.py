#!/usr/bin/env python
"""Benchmark of the batched CartPole step on B200: env-steps/s of the fused rollout
(headline), the fused per-step kernel and the unfused per-op ladder, each with its
roofline fraction, plus the CPU oracle timed on the host cores as a baseline.

    python bench.py --gpus 1 --steps 20 --warmup 3
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference      # the scalar CPU oracle on the same workload

One "step" is one pass of the whole hot path over one batch: one fused-rollout launch
covering every environment and all T time steps of the workload (action, dynamics,
termination, reward, restart for every env-step). Inputs are synthetic and fully
defined by (n_envs, T, seed): start states and actions are a counter hash evaluated
inside the kernels, so there is nothing to stage in HBM for the headline path.
Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "env_steps_per_sec"
UNIT = "env-steps/s"
SMS = 148
# Work per env-step of each rollout variant, counted by ncu (summaries under profiles/).
# "thread" = smsp__thread_inst_executed.sum / (N*T) of the per-lane formulation on 1,048,576 x 100 (one env per thread, each lane restarts its own env; tuning
# rollout_ept=1 rollout_coop=2): the instructions an environment needs, none counted for
# lanes that idle or help a neighbour — the algorithmic figure. "slot" = 32 *
# smsp__inst_executed.sum / (N*T) of the kernel the library launches by default at this size
# ("kernel"): the issue slots it really occupies; the deferred-restart kernel steps two
# environments per packed float32 instruction, so its slots fall below the thread figure.
# "fp32" = float32 multiply / add / fma lane operations of the method per env-step (37 in the
# dynamics with the shortcuts of the kernels, 22 in the contracted arithmetic, 0.2 for the start
# states of the 4.5 % of env-steps that restart, 8 more for the linear policy).
# COUNTED_AT = build.kernel_hash() of the sources these were captured from (a test compares it
# with the current sources, so that the fractions cannot go stale unnoticed).
COUNTED_AT = "24d7494f85ce7c00"
# pipe_busy: sm__pipe_fmaheavy_cycles_active (share of the launch's cycles) in the same captures — the
# resource that bounds these kernels; it counts idle slots' arithmetic and the integer multiply-adds too.
ROLLOUT_OPS = {
    # slots: 1,048,576 x 500 (the deferred kernel's ragged end makes them depend a little on T)
    "random": {"thread": 65.6, "slot": 48.8, "fp32": 37.2, "pipe_busy": 0.837, "kernel": "rollout_deferred_kernel"},
    "linear": {"thread": 70.8, "slot": 40.8, "fp32": 45.2, "pipe_busy": 0.813, "kernel": "rollout_deferred_kernel"},
    # slots: 1,048,576 x 1,000 with the reward plane and the done bitmask
    "linear+streams": {"thread": 88.9, "slot": 46.2, "fp32": 45.2, "pipe_busy": 0.800, "kernel": "rollout_deferred_kernel"},
    # slots: 2,097,152 x 200; both sides of the branch-free tanh are evaluated for every value
    "mlp": {"thread": 210.7, "slot": 311.6, "pipe_busy": 0.740, "kernel": "rollout_deferred_kernel"},
    "random+contracted": {"thread": 55.6, "slot": 40.0, "fp32": 22.2, "pipe_busy": 0.813, "kernel": "rollout_deferred_kernel"},
}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch in the same captures (the per-env
# results stay in L2); with the per-step streams: bytes per env-step (4,385.6 MB for 1,048,576 x
# 1,000; the algorithmic figure is 4.125), which scale with N*T; the launch that zeroes the done bit
# plane before the rollout writes another 0.125 B per env-step.
ROLLOUT_DRAM_BYTES = {"random": 55.6e3, "linear": 62.2e3, "mlp": 58.6e3, "random+contracted": 54.8e3}
STREAM_DRAM_BYTES_PER_ENV_STEP = 4.1825
STEP_DRAM_BYTES_16M = 567.2e6  # step_kernel at 16,777,216 envs, same kind of capture
# Algorithmic HBM bytes per env-step of the step paths.
LAST_TIMING: dict = {}  # median / best / worst of the per-iteration event times of the last timed() call
STEP_BYTES = 37.0      # 16 in + 16 out + 4 reward + 1 done, hashed action
LADDER_BYTES = 375.0   # sum over the 46 one-op kernels of their input and output planes


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_name(w) -> str:
    pol = {0: "random", 1: "linear", 2: "mlp"}[w.policy]
    return (f"{w.name}: {w.n_envs} envs x {w.T} steps per GPU, fused rollout, policy={pol}, seed={w.seed}"
            + (", reward+done streams" if w.streams else ""))


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------ reference arm
def run_reference(args) -> None:
    """The scalar CPU oracle, as it stands, on the headline workload's config. Each step is a
    bounded sample (the first `sample_envs` environments for all T time steps)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import cartpole_oracle as oracle
    from paper_2301_13062_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    cores = min(host_cores(), 256)
    weights = inputs.policy_weights(w.policy, w.policy_seed) if w.policy else None
    sample = min(w.n_envs, 1 << 17)
    for _ in range(args.warmup):
        oracle.rollout(sample, w.T, w.seed, w.policy, weights, per_env=True, nthreads=cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.rollout(sample, w.T, w.seed, w.policy, weights, per_env=True, nthreads=cores)
    dt = time.perf_counter() - t0
    value = sample * w.T * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(w), "envs_per_gpu": w.n_envs, "T": w.T,
                   "sample": f"each step = the first {sample} envs x {w.T} steps on the host cores"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} envs x {w.T} steps, {args.steps} repeats"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ our arm
def launch_plan(gpus: int, environ, argv: list[str], port: int | None = None):
    """How `--gpus N` is honoured. Returns ("run", None): this process is a rank (or the only one);
    ("spawn", cmd): no launcher started us and N > 1, so re-run this script as N local ranks, one
    per GPU; ("error", text): the launcher's world size contradicts --gpus."""
    if gpus < 1:
        return "error", f"--gpus must be >= 1 (got {gpus})"
    if "WORLD_SIZE" in environ:
        world = int(environ["WORLD_SIZE"])
        if world != gpus:
            return "error", f"launched with WORLD_SIZE={world} but --gpus {gpus}: they must agree"
        return "run", None
    if gpus == 1:
        return "run", None
    if port is None:
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return "spawn", cmd


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", help="headline rollout workload (c1, c3, c4, c5, paper)")
    ap.add_argument("--no-paths", action="store_true", help="skip the ladder / fused-step / other-config lines")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--step-envs", type=int, default=1 << 24, help="batch of the HBM-bound fused-step measurement")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every GPU runs the whole workload on its own env-id range; strong: the "
                         "workload's environments are split over the GPUs")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    kind, detail = launch_plan(args.gpus, os.environ, sys.argv[1:])
    if kind == "error":
        print(f"bench.py: {detail}", file=sys.stderr)
        sys.exit(2)
    if kind == "spawn":  # --gpus N without a launcher: one rank per GPU under torch.distributed.run
        sys.exit(subprocess.call(detail))

    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2301_13062_b200 import binding as cp
    from paper_2301_13062_b200 import inputs, sharding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if torch.cuda.device_count() <= local_rank:
        print(f"bench.py: rank {rank} needs GPU {local_rank}, this machine shows {torch.cuda.device_count()}",
              file=sys.stderr)
        sys.exit(2)
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    cp.lib()
    peaks = load_peaks()
    peak_inst = SMS * 4 * 32 * peaks["sm_max_mhz"] * 1e6  # thread-instructions/s at the maximum SM clock

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return sharding.max_over_ranks(x, device="cuda")

    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    def timed(fn, steps, warmup, flush=True, all_ranks=True):
        """Sum of per-iteration CUDA-event times on the launching stream (ms), L2 flushed
        between iterations outside the timed events; barrier on both sides and max over ranks
        (all_ranks=False: a measurement only rank 0 makes, no collective)."""
        sync = barrier if all_ranks else torch.cuda.synchronize
        for _ in range(warmup):
            fn()
        sync()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        launches0 = cp.cp_launch_count()
        for a, b in evs:
            if flush:
                flush_buf.fill_(1)
            a.record()
            fn()
            b.record()
        sync()
        launches = cp.cp_launch_count() - launches0
        per = [a.elapsed_time(b) for a, b in evs]
        ms = sum(per)
        LAST_TIMING.update(median_ms=sorted(per)[len(per) // 2], best_ms=min(per), worst_ms=max(per))
        return (max_over_ranks(ms) if all_ranks else ms), launches

    # ---- headline: fused rollout ----
    w = inputs.WORKLOADS[args.workload]
    pol_name = {0: "random", 1: "linear", 2: "mlp"}[w.policy]
    weights = inputs.policy_weights(w.policy, w.policy_seed) if w.policy else None
    pol = cp.policy(w.policy, weights) if w.policy else None
    T = w.T
    if args.scaling == "strong":  # the workload's environments split over the ranks by global id
        lo, hi = sharding.rank_env_range(w.n_envs, rank, world)
        n, env_offset, job_envs = hi - lo, lo, w.n_envs
    else:                          # weak: a full batch per rank on its own env-id range
        n, env_offset, job_envs = w.n_envs, sharding.weak_env_offset(w.n_envs, rank), world * w.n_envs
    ret = torch.empty(n, dtype=torch.float32, device="cuda")
    cnt = torch.empty(n, dtype=torch.int32, device="cuda")
    tot = torch.zeros(2, dtype=torch.int64, device="cuda")
    outs = {"ep_return_sum": ret, "ep_count": cnt, "totals": tot}
    if w.streams:
        outs["reward_stream"] = torch.empty(T, n, dtype=torch.float32, device="cuda")
        outs["done_bits"] = torch.empty(T, (n + 31) // 32, dtype=torch.int32, device="cuda")

    def rollout_step():
        cp.cp_rollout_shard(env_offset, n, T, w.seed, pol, **outs)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    t_load = time.perf_counter()
    while time.perf_counter() - t_load < 1.5:  # keep the GPU loaded while nvidia-smi starts sampling
        rollout_step()
        torch.cuda.synchronize()
    ms, launches = timed(rollout_step, args.steps, args.warmup)
    step_stats = dict(LAST_TIMING)  # this rank's own per-iteration times
    clocks = sampler.stop() if rank == 0 else {}
    ms_per_step = ms / args.steps
    value = job_envs * T / (ms_per_step * 1e-3)
    variant = pol_name + ("+streams" if w.streams else "")
    ops = ROLLOUT_OPS[variant]
    rate = n * T / (ms_per_step * 1e-3)  # per GPU
    roofline = {"bound": "alu", "kernel": ops["kernel"], "achieved": rate * ops["thread"] / 1e12,
                "peak": peak_inst / 1e12, "unit": "Tinst/s", "frac": rate * ops["thread"] / peak_inst,
                "issue_slot_frac": rate * ops["slot"] / peak_inst,
                "fp32_pipe_frac": rate * ops["fp32"] / peak_inst if "fp32" in ops else None,
                "traffic": (n * T * STREAM_DRAM_BYTES_PER_ENV_STEP if w.streams else ROLLOUT_DRAM_BYTES.get(variant)),
                "traffic_note": "ncu dram bytes of one launch at 1,048,576 envs (the 8 B/env of per-env results stay "
                                "in L2); with per-step streams the capture's bytes per env-step x N x T",
                "thread_inst_per_env_step": ops["thread"], "issue_slots_per_env_step": ops["slot"],
                "fp32_lane_ops_per_env_step": ops.get("fp32"),
                "fp32_pipe_busy_ncu": ops.get("pipe_busy"),
                "counted_at": COUNTED_AT,
                "peak_source": f"148 SMs x 4 schedulers x 32 lanes x {peaks['sm_max_mhz']:.0f} MHz ({peaks['source']} max clock)",
                "note": "frac counts instructions executed by active lanes only in the per-lane formulation (what "
                        "an environment needs); issue_slot_frac counts whole warp instructions x 32 of the kernel "
                        "launched (a packed float32 instruction serves two environments in one slot); "
                        "fp32_pipe_frac counts the float32 multiply/add/fma lane operations of the method "
                        "against the same 128 lanes per SM and clock; fp32_pipe_busy_ncu is the share of cycles the "
                        "profiler saw that pipe busy in the capture the counts come from (the kernel's bound)"}
    if w.streams:
        roofline["stream_write_gbs"] = n * T * 4.125 / (ms_per_step * 1e-3) / 1e9
        roofline["stream_write_frac_of_hbm"] = roofline["stream_write_gbs"] / peaks["hbm_gbs"]

    # ---- end to end through the C ABI with host buffers ----
    h_ret = torch.empty(n, dtype=torch.float32).pin_memory()
    h_cnt = torch.empty(n, dtype=torch.int32).pin_memory()
    h_tot = torch.empty(2, dtype=torch.int64).pin_memory()

    def e2e_step():
        cp.cp_rollout_host_shard(env_offset, n, T, w.seed, pol, h_ret, h_cnt, h_tot)

    e2e_ms, _ = timed(e2e_step, max(3, args.steps // 2), 3)
    e2e_ms /= max(3, args.steps // 2)
    e2e = {"value": job_envs * T / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": int(4 * inputs.N_WEIGHTS[w.policy]) + 24, "d2h_bytes_per_step": 8 * n + 16,
           "ms_per_step": e2e_ms,
           "note": "cp_rollout_host_shard: host scalars (n_envs, T, seed) and policy weights in; per-env returns and "
                   "counts land in pinned host memory (stored there by the kernel over PCIe while it runs), "
                   "totals copied back, stream synchronised, every step"}

    # side measurements and the CPU baseline belong to the one-GPU run (under torchrun they would
    # only keep the other ranks waiting in the final reduction)
    paths = {}
    if not args.no_paths and world == 1:
        paths = measure_paths(cp, inputs, torch, lambda *a, **k: timed(*a, all_ranks=False, **k), peaks, peak_inst, args)

    cpu = None
    if not args.no_cpu and world == 1:
        from oracle import cartpole_oracle as oracle
        cores = min(host_cores(), 256)
        sample = min(n, 1 << 20)
        t0 = time.perf_counter()
        o = oracle.rollout(sample, T, w.seed, w.policy, weights, nthreads=cores)
        dt = time.perf_counter() - t0
        same = float((o["ep_return_sum"] == ret[:sample].cpu().numpy()).mean()) if env_offset == 0 else None
        one = min(n, 1 << 16)
        t1 = time.perf_counter()
        oracle.rollout(one, T, w.seed, w.policy, weights, nthreads=1)
        dt1 = time.perf_counter() - t1
        cpu = {"value": sample * T / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"first {sample} envs x {T} steps of the workload, one pass, {dt:.2f} s",
               "returns_identical_to_gpu": same,
               "one_core": {"value": one * T / dt1, "unit": UNIT, "cores": 1,
                            "sample": f"first {one} envs x {T} steps, one pass, {dt1:.2f} s"}}

    sharding.reduce_totals(tot)  # the only exchange the path has: 16 bytes, outside the timed region
    # the other two rungs of the metric, inside the object the record keeps
    for key, name in (("fused_step_hbm", "step_kernel"), ("ladder_hbm", "ladder")):
        if key in paths:
            e = paths[key]
            roofline[name] = {"n_envs": e["n_envs"], "ms": e.get("ms_per_launch", e.get("ms_per_step")),
                              "env_steps_per_sec": e["env_steps_per_sec"], **e["roofline"]}
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_median": step_stats["median_ms"],
            "ms_per_step_best": step_stats["best_ms"], "higher_is_better": True, "scaling": args.scaling,
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(w),
                       "l2": "flushed between iterations (256 MiB fill outside the timed events)",
                       "envs_per_gpu": n, "T": T},
            "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "roofline": roofline,
            "cpu_baseline": cpu, "paths": paths,
            "paper_context": {"hardware": "RTX 2080 Ti, 2048 envs x 10000 steps", "eager_vs_baseline": 0.13,
                              "fused_step_vs_baseline": 3.41, "unroll10_vs_fused_step": 3.5,
                              "hand_cuda_vs_best_xla": 2.7},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def measure_paths(cp, inputs, torch, timed, peaks, peak_inst, args) -> dict:
    """Ladder, fused step and the other rollout configurations (rank 0, one GPU each)."""
    out = {}
    hbm = peaks["hbm_gbs"] * 1e9

    # what the pipes sustain on this GPU: single-kind instruction streams (float32 fused
    # multiply-add, 32-bit integer multiply-add, special-function reciprocal), beside the issue
    # peak the rollout's roofline is derived from
    seed = torch.linspace(0.5, 1.5, 10, device="cuda")
    sink = torch.empty(cp.CP_CALIBRATE_THREADS_PER_SM * torch.cuda.get_device_properties(0).multi_processor_count,
                       device="cuda")
    calib = {"issue_peak_tinst_per_s": peak_inst / 1e12}
    # (kinds 3-7: the packed FFMA2 alone and half-and-half mixes, which show what shares a pipe with it)
    for name, kind, iters in (("ffma", 0, 20000), ("imad", 1, 20000), ("mufu_rcp", 2, 5000), ("ffma2", 3, 20000),
                              ("ffma2+ffma", 4, 20000), ("ffma2+imad", 5, 20000), ("ffma2+alu_x2", 6, 20000),
                              ("ffma+imad", 7, 20000)):
        count = {"n": 0}

        def fn():
            count["n"] = cp.cp_calibrate_pipe(kind, seed, sink, iters)
        ms, _ = timed(fn, 3, 2, flush=False)
        calib[name + "_tinst_per_s"] = 3 * count["n"] / (ms * 1e-3) / 1e12
    out["pipe_calibration"] = calib
    del seed, sink

    def step_setup(n):
        stride = (n + 3) // 4 * 4
        a = torch.zeros(4, stride, device="cuda")
        b = torch.zeros(4, stride, device="cuda")
        sa, sb = cp.cp_wrap(a, n, 0), cp.cp_wrap(b, n, 0)
        cp.cp_fill_start(sa)
        reward = torch.empty(n, device="cuda")
        done = torch.empty(n, dtype=torch.uint8, device="cuda")
        return a, b, sa, sb, reward, done

    # fused step, HBM-bound size: ping-pong between two batches
    n = args.step_envs
    a, b, sa, sb, reward, done = step_setup(n)
    for _ in range(40):  # reach the steady-state mix of restarts
        cp.cp_step(sa, None, sb, reward, done)
        cp.cp_step(sb, None, sa, reward, done)
    state = {"flip": False}

    def fused_step():
        if state["flip"]:
            cp.cp_step(sb, None, sa, reward, done)
        else:
            cp.cp_step(sa, None, sb, reward, done)
        state["flip"] = not state["flip"]

    ms, _ = timed(fused_step, 20, 4)
    ms /= 20
    gbs = n * STEP_BYTES / (ms * 1e-3) / 1e9
    out["fused_step_hbm"] = {"n_envs": n, "ms_per_launch": ms, "ms_median": LAST_TIMING["median_ms"],
                             "ms_best": LAST_TIMING["best_ms"], "env_steps_per_sec": n / (ms * 1e-3),
                             "roofline": {"bound": "hbm", "kernel": "step_kernel", "achieved": gbs,
                                          "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs * 1e9 / hbm,
                                          "traffic": STEP_DRAM_BYTES_16M if n == 1 << 24 else None,
                                          "bytes_per_env_step": STEP_BYTES}}
    # ladder at the same size
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")

    def ladder_step():
        cp.cp_set_time(sa, 41)
        cp.cp_step_unfused(sa, None, sb, reward, done, ws)

    ms, launches = timed(ladder_step, 5, 3)
    ms /= 5
    gbs = n * LADDER_BYTES / (ms * 1e-3) / 1e9
    out["ladder_hbm"] = {"n_envs": n, "ms_per_step": ms, "launches_per_step": launches // 5,
                         "env_steps_per_sec": n / (ms * 1e-3),
                         "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                      "frac": gbs * 1e9 / hbm, "bytes_per_env_step": LADDER_BYTES}}
    del a, b, sa, sb, reward, done, ws
    torch.cuda.empty_cache()

    # size sweep of the fused step, 2^16 .. 2^26 envs: launch-bound -> L2-resident -> HBM-bound
    sweep = []
    for lg in range(16, 27, 2):
        n = 1 << lg
        a, b, sa, sb, reward, done = step_setup(n)
        cp.cp_rollout_from(sa, 40)
        flip = {"f": False}

        def one():
            if flip["f"]:
                cp.cp_step(sb, None, sa, reward, done)
            else:
                cp.cp_step(sa, None, sb, reward, done)
            flip["f"] = not flip["f"]

        ms, _ = timed(one, 10, 4)
        ms /= 10
        sweep.append({"n_envs": n, "us_per_launch": 1e3 * ms, "gbs": n * STEP_BYTES / (ms * 1e-3) / 1e9,
                      "frac_of_hbm": n * STEP_BYTES / (ms * 1e-3) / hbm})
        del a, b, sa, sb, reward, done
        torch.cuda.empty_cache()
    out["fused_step_sweep"] = sweep

    # config 2: 65,536 envs, per-step launches (launch-bound), 1,000 steps per timed iteration
    w2 = inputs.WORKLOADS["c2"]
    n = w2.n_envs
    a, b, sa, sb, reward, done = step_setup(n)
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")

    def c2_fused():
        cp.cp_set_time(sa, 0)
        cp.cp_step_repeat(sa, w2.T, reward, done)  # T launches issued from one C call

    def c2_ladder():
        cp.cp_set_time(sa, 0)
        for _ in range(50):
            cp.cp_step_unfused(sa, None, sb, reward, done, ws)
            cp.cp_step_unfused(sb, None, sa, reward, done, ws)

    ms, _ = timed(c2_fused, 3, 3, flush=False)
    ms /= 3
    out["c2_fused_step"] = {"n_envs": n, "T": w2.T, "ms_total": ms, "us_per_launch": 1e3 * ms / w2.T,
                            "env_steps_per_sec": n * w2.T / (ms * 1e-3), "note": "launch-bound: 2.4 MB per launch"}
    # the same 1,000 launches replayed from a CUDA graph (removes the host launch cost)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        c2_fused()
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            c2_fused()
    torch.cuda.synchronize()
    ms, _ = timed(graph.replay, 3, 3, flush=False)
    ms /= 3
    out["c2_fused_step_graph"] = {"n_envs": n, "T": w2.T, "ms_total": ms, "us_per_launch": 1e3 * ms / w2.T,
                                  "env_steps_per_sec": n * w2.T / (ms * 1e-3),
                                  "note": "the same launches captured once in a CUDA graph and replayed"}
    ms, _ = timed(c2_ladder, 3, 3, flush=False)
    ms /= 3
    out["c2_ladder"] = {"n_envs": n, "T": 100, "ms_total": ms, "us_per_step": 1e3 * ms / 100,
                        "env_steps_per_sec": n * 100 / (ms * 1e-3), "launches_per_step": 46}
    out["ratios"] = {"fused_step_over_ladder_c2": out["c2_fused_step"]["env_steps_per_sec"] / out["c2_ladder"]["env_steps_per_sec"],
                     "fused_step_over_ladder_hbm": out["fused_step_hbm"]["env_steps_per_sec"] / out["ladder_hbm"]["env_steps_per_sec"]}
    del a, b, sa, sb, reward, done, ws

    # the paper's own batch shape (2,048 envs; Sec. V) on the per-step paths, for its ratios:
    # ladder -> fused step -> (paper_rollout below), all launch-bound at this size
    wp = inputs.WORKLOADS["paper"]
    n = wp.n_envs
    a, b, sa, sb, reward, done = step_setup(n)
    ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")

    def paper_fused():
        cp.cp_set_time(sa, 0)
        cp.cp_step_repeat(sa, 1000, reward, done)

    def paper_ladder():
        cp.cp_set_time(sa, 0)
        for _ in range(50):
            cp.cp_step_unfused(sa, None, sb, reward, done, ws)
            cp.cp_step_unfused(sb, None, sa, reward, done, ws)

    ms, _ = timed(paper_fused, 3, 3, flush=False)
    ms /= 3
    out["paper_fused_step"] = {"n_envs": n, "T": 1000, "us_per_launch": 1e3 * ms / 1000, "env_steps_per_sec": n * 1000 / (ms * 1e-3)}
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        paper_fused()
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            paper_fused()
    torch.cuda.synchronize()
    ms, _ = timed(graph.replay, 3, 3, flush=False)
    ms /= 3
    out["paper_fused_step_graph"] = {"n_envs": n, "T": 1000, "us_per_launch": 1e3 * ms / 1000,
                                     "env_steps_per_sec": n * 1000 / (ms * 1e-3)}
    ms, _ = timed(paper_ladder, 3, 3, flush=False)
    ms /= 3
    out["paper_ladder"] = {"n_envs": n, "T": 100, "us_per_step": 1e3 * ms / 100,
                           "env_steps_per_sec": n * 100 / (ms * 1e-3), "launches_per_step": 46}
    del a, b, sa, sb, reward, done, ws, graph

    # options of the general rollout call on the headline shape: CartPole-v1's 500-step episode
    # limit, and actions supplied as a packed bit stream (here: the hashed ones, written by a
    # first rollout) instead of drawn in the kernel
    w3 = inputs.WORKLOADS["c3"]
    n, T = w3.n_envs, w3.T
    outs = {"ep_return_sum": torch.empty(n, device="cuda"), "ep_count": torch.empty(n, dtype=torch.int32, device="cuda"),
            "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
    act = torch.empty(T, (n + 31) // 32, dtype=torch.int32, device="cuda")
    cp.cp_rollout(n, T, w3.seed, None, action_bits=act, **outs)
    # ... and the contracted arithmetic (fused multiply-adds, folded constants): within the
    # tolerances, but not the bits of the per-op ladder, so never the headline
    mlp_pol = cp.policy(inputs.POLICY_MLP, inputs.policy_weights(inputs.POLICY_MLP, inputs.WORKLOADS["c5"].policy_seed))
    for key, kwargs in (("c3_rollout_step_limit_500", {"max_episode_steps": 500}),
                        ("c3_rollout_supplied_actions", {"action_bits_in": act}),
                        ("c3_rollout_contracted_arithmetic", {"arithmetic": cp.CP_ARITH_CONTRACTED}),
                        ("c3_rollout_mlp", {"policy": mlp_pol}),
                        ("c3_rollout_mlp_contracted_arithmetic",
                         {"policy": mlp_pol, "arithmetic": cp.CP_ARITH_CONTRACTED})):
        def fn():
            cp.cp_rollout_ex(n_envs=n, T=T, seed=w3.seed, **kwargs, **outs)
        ms, _ = timed(fn, 10, 3)
        ms /= 10
        out[key] = {"n_envs": n, "T": T, "ms_per_launch": ms, "env_steps_per_sec": n * T / (ms * 1e-3)}
    # a population of linear policies, one per environment (weights read once into registers)
    pop = cp.policy(cp.CP_POLICY_LINEAR_PER_ENV, torch.from_numpy(inputs.per_env_linear_weights(n, 11)).cuda())

    def pop_fn():
        cp.cp_rollout(n, T, w3.seed, pop, **outs)
    ms, _ = timed(pop_fn, 10, 3)
    ms /= 10
    out["c3_rollout_per_env_linear"] = {"n_envs": n, "T": T, "ms_per_launch": ms,
                                        "env_steps_per_sec": n * T / (ms * 1e-3)}
    # every random value as data, as in the paper's baseline (Sec. V-A): the action bits of above
    # and the start states (here the hashed ones of each time step: [T][4][n] floats = 8.4 GB)
    starts = torch.empty(T, 4, n, device="cuda")
    for k in range(T):
        cp.cp_fill_start(cp.cp_wrap(starts[k], n, w3.seed, k + 1))

    def data_fn():
        cp.cp_rollout_ex(n_envs=n, T=T, seed=w3.seed, action_bits_in=act, start_states_in=starts, **outs)
    ms, _ = timed(data_fn, 10, 3)
    ms /= 10
    out["c3_rollout_all_randomness_supplied"] = {"n_envs": n, "T": T, "ms_per_launch": ms,
                                                 "env_steps_per_sec": n * T / (ms * 1e-3)}
    del outs, act, pop, starts
    torch.cuda.empty_cache()

    # wider in-kernel policies on config 5's shape (16,777,216 envs x 200 steps)
    w5 = inputs.WORKLOADS["c5"]
    n, T = w5.n_envs, w5.T
    outs = {"ep_return_sum": torch.empty(n, device="cuda"), "ep_count": torch.empty(n, dtype=torch.int32, device="cuda"),
            "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
    for key, kind in (("c5_rollout_mlp32", inputs.POLICY_MLP32), ("c5_rollout_mlp64", inputs.POLICY_MLP64),
                      ("c5_rollout_mlp_deep_16_16", inputs.POLICY_MLP_DEEP)):
        # weight draws for which the network uses both actions (3; 7 for the deep one)
        pol = cp.policy(kind, inputs.policy_weights(kind, 7 if kind == inputs.POLICY_MLP_DEEP else 3))

        def fn():
            cp.cp_rollout(n, T, w5.seed, pol, **outs)
        ms, _ = timed(fn, 2, 3)
        ms /= 2
        out[key] = {"n_envs": n, "T": T, "hidden": inputs.HIDDEN_OF.get(kind, "16+16"), "ms_per_launch": ms,
                    "env_steps_per_sec": n * T / (ms * 1e-3)}
    # config 5 itself in the contracted arithmetic (FMA dynamics and the five-instruction tanh)
    pol = cp.policy(w5.policy, inputs.policy_weights(w5.policy, w5.policy_seed))

    def c5_contracted():
        cp.cp_rollout_ex(n_envs=n, T=T, seed=w5.seed, policy=pol, arithmetic=cp.CP_ARITH_CONTRACTED, **outs)
    ms, _ = timed(c5_contracted, 2, 3)
    ms /= 2
    out["c5_rollout_contracted_arithmetic"] = {"n_envs": n, "T": T, "ms_per_launch": ms,
                                               "env_steps_per_sec": n * T / (ms * 1e-3)}
    del outs
    torch.cuda.empty_cache()

    # the other rollout configurations
    for name in ("c1", "c3", "c4", "c5", "paper"):
        w = inputs.WORKLOADS[name]
        if name == args.workload:
            continue
        weights = inputs.policy_weights(w.policy, w.policy_seed) if w.policy else None
        pol = cp.policy(w.policy, weights) if w.policy else None
        n, T = w.n_envs, w.T
        outs = {"ep_return_sum": torch.empty(n, device="cuda"), "ep_count": torch.empty(n, dtype=torch.int32, device="cuda"),
                "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
        if w.streams:
            outs["reward_stream"] = torch.empty(T, n, dtype=torch.float32, device="cuda")
            outs["done_bits"] = torch.empty(T, (n + 31) // 32, dtype=torch.int32, device="cuda")

        def fn():
            cp.cp_rollout(n, T, w.seed, pol, **outs)

        k = 5 if n * T > 1e9 else 10
        ms, _ = timed(fn, k, 3)
        ms /= k
        pol_name = {0: "random", 1: "linear", 2: "mlp"}[w.policy]
        rate = n * T / (ms * 1e-3)
        ops = ROLLOUT_OPS[pol_name + ("+streams" if w.streams else "")]
        entry = {"n_envs": n, "T": T, "policy": pol_name, "ms_per_launch": ms, "env_steps_per_sec": rate,
                 "alu_frac": rate * ops["thread"] / peak_inst, "issue_slot_frac": rate * ops["slot"] / peak_inst}
        if w.streams:
            entry["stream_write_gbs"] = rate * 4.125 / 1e9
            entry["stream_write_frac_of_hbm"] = rate * 4.125 / hbm
        if name in ("c1", "paper"):
            # a few warps on the whole chip: one warp's per-step latency is what is paid, so the
            # fractions above say nothing; the figure to read is the time per step against the
            # step's dependency chain (14 dependent float operations, about 60 SM cycles)
            entry["kernel"] = "rollout_assisted_kernel"
            entry["bound"] = "latency"
            entry["ns_per_step"] = ms * 1e6 / T
            entry["sm_cycles_per_step"] = ms * 1e-3 / T * peaks["sm_max_mhz"] * 1e6
        out[f"{name}_rollout"] = entry
        del outs
        torch.cuda.empty_cache()
    return out


if __name__ == "__main__":
    main()
