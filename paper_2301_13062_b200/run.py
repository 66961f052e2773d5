"""Command-line runner for one path of the library on synthetic input — handy for
profiling a single kernel on a chosen size.

    python -m paper_2301_13062_b200.run rollout --n 1048576 --T 100 --policy random --reps 2
    python -m paper_2301_13062_b200.run step --n 16777216 --reps 4
    python -m paper_2301_13062_b200.run ladder --n 4194304 --reps 1

Prints one JSON line with the mean CUDA-event time per repetition.
"""
from __future__ import annotations

import argparse
import json


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("path", choices=["rollout", "step", "ladder"])
    ap.add_argument("--n", type=int, default=1 << 20)
    ap.add_argument("--T", type=int, default=100)
    ap.add_argument("--policy", default="random", choices=["random", "linear", "mlp"])
    ap.add_argument("--streams", action="store_true", help="rollout: also write the reward plane and done bitmask")
    ap.add_argument("--contracted", action="store_true", help="rollout: contracted arithmetic (CP_ARITH_CONTRACTED)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    ap.add_argument("--tune", action="append", default=[], help="key=value for cp_tune, repeatable")
    args = ap.parse_args()

    import torch

    from . import binding as cp
    from . import inputs

    cp.lib()
    torch.cuda.set_device(0)
    for kv in args.tune:
        k, v = kv.split("=")
        cp.cp_tune(k, int(v))
    n, T = args.n, args.T
    if args.path == "rollout":
        kind = {"random": 0, "linear": 1, "mlp": 2}[args.policy]
        pol = cp.policy(kind, inputs.policy_weights(kind, kind)) if kind else None
        outs = {"ep_return_sum": torch.empty(n, device="cuda"),
                "ep_count": torch.empty(n, dtype=torch.int32, device="cuda"),
                "totals": torch.zeros(2, dtype=torch.int64, device="cuda")}
        if args.streams:
            outs["reward_stream"] = torch.empty(T, n, device="cuda")
            outs["done_bits"] = torch.empty(T, (n + 31) // 32, dtype=torch.int32, device="cuda")

        def fn():
            if args.contracted:
                cp.cp_rollout_ex(n_envs=n, T=T, seed=args.seed, policy=pol, arithmetic=cp.CP_ARITH_CONTRACTED, **outs)
            else:
                cp.cp_rollout(n, T, args.seed, pol, **outs)
        units = n * T
    else:
        stride = (n + 3) // 4 * 4
        a = torch.zeros(4, stride, device="cuda")
        b = torch.zeros(4, stride, device="cuda")
        sa, sb = cp.cp_wrap(a, n, args.seed), cp.cp_wrap(b, n, args.seed)
        cp.cp_fill_start(sa)
        reward = torch.empty(n, device="cuda")
        done = torch.empty(n, dtype=torch.uint8, device="cuda")
        # bring the batch to the steady-state mix of restarts with one short rollout in place
        cp.cp_rollout_from(sa, 40)
        if args.path == "step":
            flip = [False]

            def fn():
                if flip[0]:
                    cp.cp_step(sb, None, sa, reward, done)
                else:
                    cp.cp_step(sa, None, sb, reward, done)
                flip[0] = not flip[0]
        else:
            ws = torch.empty(cp.cp_unfused_workspace_bytes(n), dtype=torch.uint8, device="cuda")

            def fn():
                cp.cp_set_time(sa, 40)
                cp.cp_step_unfused(sa, None, sb, reward, done, ws)
        units = n
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.reps
    print(json.dumps({"path": args.path, "n_envs": n, "T": T if args.path == "rollout" else 1, "policy": args.policy,
                      "ms_per_rep": ms, "env_steps_per_sec": units / (ms * 1e-3), "launches": cp.cp_launch_count()}))


if __name__ == "__main__":
    main()
