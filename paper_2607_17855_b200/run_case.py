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
    for _ in range(args.reps):
        md.run(algo, obs, act, w.K, q_out=q)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    md.run(algo, obs, act, w.K, q_out=q)
    b.record()
    b.synchronize()
    ms = a.elapsed_time(b)
    print(json.dumps({"workload": w.name, "algo": algo, "agents": w.N, "T": w.T, "K": w.K, "arith": args.arith,
                      "kernel": md.last_kernel, "ms": ms, "updates_per_s": w.updates / (ms * 1e-3)}))


if __name__ == "__main__":
    main()
