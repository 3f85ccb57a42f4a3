"""Run one seeded workload through the library and print its device time.

    python -m paper_2607_17855_b200.run_case --config 4 --algo mmp --agents 296

Useful for profiling a single kernel on a case of chosen size (the profiler
summaries under profiles/ give the exact command lines they were made with).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, required=True, help="1..4, or 5 with --member")
    ap.add_argument("--member", type=int, default=0, help="member of the randomised sweep (config 5)")
    ap.add_argument("--algo", default=None, choices=["filter", "vmp", "mmp"])
    ap.add_argument("--agents", type=int, default=None)
    ap.add_argument("--steps", type=int, default=None, help="time steps T")
    ap.add_argument("--iters", type=int, default=None, help="iterations K")
    ap.add_argument("--arith", default="f64", choices=["f64", "f32"])
    ap.add_argument("--reps", type=int, default=3, help="warm-up calls before the timed one")
    ap.add_argument("--soft", action="store_true", help="give the observations as (one-hot) categorical vectors")
    args = ap.parse_args()

    import torch
    import paper_2607_17855_b200 as bi
    from biwl import make_config, make_sweep_config

    if args.config == 5:
        w = make_sweep_config(args.member, N=args.agents, T=args.steps, K=args.iters)
    else:
        w = make_config(args.config, N=args.agents, T=args.steps, K=args.iters)
    algo = args.algo or (w.algo if w.algo != "all" else "filter")
    md = bi.model_from_workload(w, arith=args.arith)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda() if w.act.size else None
    q = torch.empty((w.N, w.T, w.S), device="cuda")
    if args.soft:
        import numpy as np
        off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
        soft = np.zeros((w.N, w.T, int(off[-1])), np.float32)
        for i in range(w.M):
            np.put_along_axis(soft[:, :, off[i]:off[i + 1]], w.obs[:, :, i:i + 1], 1.0, axis=2)
        soft = torch.from_numpy(soft).cuda()
        call = lambda: md.run_soft(algo, soft, act, w.K, q_out=q)  # noqa: E731
    else:
        call = lambda: md.run(algo, obs, act, w.K, q_out=q)  # noqa: E731
    for _ in range(args.reps):
        call()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    call()
    b.record()
    b.synchronize()
    ms = a.elapsed_time(b)
    print(json.dumps({"workload": w.name, "algo": algo, "agents": w.N, "T": w.T, "K": w.K, "arith": args.arith,
                      "soft": bool(args.soft), "kernel": md.last_kernel, "ms": ms, "updates_per_s": w.updates / (ms * 1e-3)}))


if __name__ == "__main__":
    main()
