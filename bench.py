#!/usr/bin/env python
"""Benchmark: batched belief updates per second on B200.

A step is one pass of the whole hot path over one batch: one ``bi_filter``
call on the headline workload (4096 agents sharing one model, F = 3 factors
[8, 8, 6], M = 3 modalities, T = 50 steps, K = 16 iterations), inputs resident
in HBM.  A belief update is one softmax update of one factor of one agent at
one step in one iteration, so a step performs N*T*F*K of them.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints one JSON line.  With ``--impl reference`` the CPU oracle is timed
instead (rank 0 only), each step on a bounded sample of the same workload.

    python bench.py --case 4:mmp [--agents N] [--T T] [--K K] [--member j] [--soft] [--arith f32]

runs ONE secondary workload of a chosen size a few times and prints its device
time (one JSON line of its own, not the benchmark's): the command the profiler
summaries were captured with.
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

METRIC = "belief_updates_per_sec"
UNIT = "updates/s"
HEADLINE = 2  # configuration the metric is quoted on
# the end-to-end run filters the trajectory in consecutive blocks of steps of these lengths (short last
# blocks: the last block's beliefs are the only ones whose way to the host nothing overlaps)
E2E_BLOCKS = "8,14,14,9,5"

# Nominal ALU peaks derived from the unit counts: 148 SMs x lanes x 2 flops x 1.965 GHz.
FP64_PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12   # 37.2
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12  # 74.4


# dram__bytes_read.sum + dram__bytes_write.sum per call on the timed workloads, from ncu captures of the
# same kernels (bytes; the captures and how they scale to these sizes are written up beside the code,
# in the profiler summaries).  A record of those captures: the run itself does not measure DRAM traffic.
NCU_DRAM_BYTES_PER_CALL = {
    "tile3_filter_f64": 8.05e6,    # config 2, full size, one launch (read 8.05 MB, written 3.3 KB: outputs stay in L2)
    "batch_vmp_f64": 6.8e8,        # config 3: 16 x (9.6 + 2.3 MB contraction, 30.5 MB update), each launch with the
                                   # cold L2 the profiler gives it; back to back the partial messages stay in L2
    "tile3_mmp_f64": 7.3e8,        # config 4: (101.8 + 3.4) MB captured on 296 agents x 2048 / 296 (per-agent models:
                                   # traffic grows in proportion to the agents)
}


def fma_probe(arith: str) -> float:
    """Measured multiply-add rate of this GPU in TFLOP/s: a kernel of independent chains from
    bench_probe.cu (built on first use with nvcc for sm_100a, beside this file)."""
    import ctypes
    import torch
    src, lib = os.path.join(ROOT, "bench_probe.cu"), os.path.join(ROOT, "bench_probe.so")
    if not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(src):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.run([nvcc, "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-Xcompiler", "-fPIC",
                        "-shared", "-o", tmp, src], check=True, capture_output=True)
        os.replace(tmp, lib)
    L = ctypes.CDLL(lib)
    L.bench_probe_fma.restype = ctypes.c_int
    L.bench_probe_fma.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.c_void_p]
    v = ctypes.c_double(0.0)
    rc = L.bench_probe_fma(1 if arith == "f64" else 0, ctypes.byref(v), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != 0:
        raise RuntimeError("bench_probe_fma failed")
    return float(v.value)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def algorithmic_flops(w) -> float:
    """4 * P flops (2 P multiply-adds) per dependency group with >= 2 factors,
    per agent, step and iteration (all leave-one-out messages of the group)."""
    groups = {}
    for d in w.dep:
        key = tuple(sorted(f for f in d if w.n[f] > 1))
        if len(key) >= 2:
            p = 1
            for f in key:
                p *= int(w.n[f])
            groups[key] = p
    return 4.0 * sum(groups.values()) * w.N * w.T * w.K


def algorithmic_bytes(w, elem_bytes: int) -> float:
    """Each needed slice log A_i[o_{t,i}] read once per (agent, step) plus the
    index inputs and belief outputs."""
    slices = 0
    for d in w.dep:
        p = 1
        for f in d:
            p *= int(w.n[f])
        slices += p
    io = w.obs.nbytes + w.act.nbytes + w.N * w.T * w.S * 4
    if w.G == 1:
        model = sum(a.size for a in w.A) * elem_bytes  # shared: read once
        return float(io + model)
    return float(w.N * w.T * slices * elem_bytes + io)


def rank_seed(rank: int) -> int:
    """Seed of the batch a rank draws: agents are independent, so ranks shard by
    drawing disjoint batches of the same workload (weak scaling)."""
    return 1000 + HEADLINE + 7919 * rank


def max_over_ranks(dist, seconds: float, device) -> float:
    """Slowest rank's device time (the job finishes when the last rank does)."""
    if dist is None:
        return seconds
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(updates_per_rank: int, world: int, seconds: float) -> float:
    """Whole-job belief updates per second over all ranks."""
    return updates_per_rank * world / seconds


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while timing runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def time_steps(fn, steps, warmup, flush, torch):
    """Device time of ``steps`` calls of fn, L2 flushed before each; returns seconds per step list."""
    for _ in range(warmup):
        flush.zero_()
        fn()
    torch.cuda.synchronize()
    times = []
    for _ in range(steps):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        times.append(a.elapsed_time(b) * 1e-3)
    return times


def bench_config(torch, bi, w, algo, arith, steps, warmup, flush):
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    md = bi.model_from_workload(w, arith=arith)
    torch.cuda.synchronize()
    pack_ms = (time.perf_counter() - t0) * 1e3   # host arrays -> device, packing kernels, handle
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda() if w.act.size else None
    q = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
    l0 = md.launch_count
    times = time_steps(lambda: md.run(algo, obs, act, w.K, q_out=q), steps, warmup, flush, torch)
    launches = (md.launch_count - l0) // (steps + warmup)
    assert md.status() == 0
    res = {"seconds": sum(times) / len(times), "best": min(times), "median": sorted(times)[len(times) // 2],
           "pack_ms": pack_ms, "kernel": md.last_kernel,
           "launches_per_step": launches, "model": md, "obs": obs, "act": act, "q": q}
    return res


def reference_arm(args, rank, world):
    """The CPU oracle, as it stands, on the GPU machine's host cores."""
    if rank != 0:
        return
    import oracle
    from biwl import make_config
    w = make_config(HEADLINE)
    sample_agents = 128
    sub = w.take_agents(range(sample_agents))
    cores = oracle.max_threads()
    for _ in range(args.warmup):
        oracle.run_workload(sub.take_agents(range(8)))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.run_workload(sub)
    dt = (time.perf_counter() - t0) / args.steps
    value = sub.updates / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {HEADLINE}: filtering, shared model n=[8,8,6] m=[16,8,8], T=50, K=16; "
                               f"each step = the first {sample_agents} of 4096 agents"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample_agents} agents x 50 steps x 16 iterations per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_case(args):
    """One call of one workload at a chosen size, timed after a few warm-up calls."""
    import numpy as np
    import torch
    import paper_2607_17855_b200 as bi
    from biwl import make_config, make_sweep_config
    cfg, _, algo = args.case.partition(":")
    cfg = int(cfg)
    if cfg == 5:
        w = make_sweep_config(args.member, N=args.agents, T=args.T, K=args.K)
    else:
        w = make_config(cfg, N=args.agents, T=args.T, K=args.K)
    algo = algo or (w.algo if w.algo != "all" else "filter")
    md = bi.model_from_workload(w, arith=args.arith)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda() if w.act.size else None
    q = torch.empty((w.N, w.T, w.S), device="cuda")
    if args.soft:
        off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
        soft = np.zeros((w.N, w.T, int(off[-1])), np.float32)
        for i in range(w.M):
            np.put_along_axis(soft[:, :, off[i]:off[i + 1]], w.obs[:, :, i:i + 1], 1.0, axis=2)
        soft = torch.from_numpy(soft).cuda()
        call = lambda: md.run_soft(algo, soft, act, w.K, q_out=q)  # noqa: E731
    else:
        call = lambda: md.run(algo, obs, act, w.K, q_out=q)  # noqa: E731
    for _ in range(args.warmup):
        call()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    call()
    b.record()
    b.synchronize()
    ms = a.elapsed_time(b)
    assert md.status() == 0
    print(json.dumps({"workload": w.name, "algo": algo, "agents": w.N, "T": w.T, "K": w.K, "arith": args.arith,
                      "soft": bool(args.soft), "kernel": md.last_kernel, "ms": ms,
                      "updates_per_s": w.updates / (ms * 1e-3)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--arith", default="f64", choices=["f64", "f32"])
    ap.add_argument("--e2e-blocks", default=E2E_BLOCKS,
                    help="the end-to-end run filters the trajectory in consecutive blocks of steps: their number, "
                         "or their lengths as a comma-separated list")
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary workloads and the CPU baseline")
    ap.add_argument("--case", default=None, help="CONFIG[:ALGO], e.g. 4:mmp: run that one workload and print its time")
    ap.add_argument("--agents", type=int, default=None, help="with --case: agents N")
    ap.add_argument("--T", type=int, default=None, help="with --case: time steps")
    ap.add_argument("--K", type=int, default=None, help="with --case: iterations")
    ap.add_argument("--member", type=int, default=0, help="with --case 5: member of the randomised sweep")
    ap.add_argument("--soft", action="store_true", help="with --case: observations as (one-hot) categorical vectors")
    args = ap.parse_args()
    if args.case:
        run_case(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        reference_arm(args, rank, world)
        return

    import numpy as np
    import torch
    import paper_2607_17855_b200 as bi
    from biwl import make_config

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # agents are independent: each rank runs its own full-size batch (weak scaling),
    # drawn from its own seed; there is no collective on the data path
    w = make_config(HEADLINE, seed=rank_seed(rank))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")  # > 126 MB L2

    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    head = bench_config(torch, bi, w, "filter", args.arith, args.steps, args.warmup, flush)
    torch.cuda.synchronize()
    sec = head["seconds"]
    sec = max_over_ranks(dist, sec, "cuda")
    value = aggregate_throughput(w.updates, world, sec)

    # ---- end to end: pinned host inputs -> device -> filtering -> host beliefs.  The trajectory is
    # run as consecutive blocks of steps (bi_filter, then bi_filter_continue from the handle's
    # full-precision record of the previous block's last belief: bit for bit the single call's result),
    # so a block's beliefs travel to the host while the next block runs.
    md, q = head["model"], head["q"]
    spec = str(args.e2e_blocks)
    if "," in spec:
        lens = [int(x) for x in spec.split(",")]
    else:
        nb = max(1, int(spec))
        lens = [w.T // nb] * nb if w.T % nb == 0 else [w.T]
    if sum(lens) != w.T or min(lens) < 1:
        lens = [w.T]
    nchunk = len(lens)
    starts = [sum(lens[:i]) for i in range(nchunk)]
    copy_out, copy_in = torch.cuda.Stream(), torch.cuda.Stream()
    # host inputs block by block, each block packed into one pinned buffer so that it reaches the device
    # in one copy; the copies are issued in order on one stream (side by side they would share the link and
    # the first block would wait for all of them) and a block's call waits for its own copy only
    parts = []
    for i in range(nchunk):
        t0, tc = starts[i], lens[i]
        parts.append([np.ascontiguousarray(w.obs[:, t0:t0 + tc]), np.ascontiguousarray(w.act[:, t0:t0 + tc - 1]),
                      np.ascontiguousarray(w.act[:, t0 - 1]) if i else np.empty((w.N, 0), np.int32)])
    h_in = [torch.from_numpy(np.concatenate([x.reshape(-1) for x in blk]).astype(np.int32)).pin_memory()
            for blk in parts]
    d_buf = [torch.empty(h.shape, dtype=torch.int32, device="cuda") for h in h_in]
    d_in = []
    for buf, blk in zip(d_buf, parts):
        pos, views = 0, []
        for x in blk:
            views.append(buf[pos:pos + x.size].view(x.shape))
            pos += x.size
        d_in.append(views)
    d_q = [torch.empty((w.N, tc, w.S), dtype=torch.float32, device="cuda") for tc in lens]
    h_q = [torch.empty((w.N, tc, w.S), dtype=torch.float32).pin_memory() for tc in lens]
    done = [torch.cuda.Event() for _ in range(nchunk)]
    arrived = [torch.cuda.Event() for _ in range(nchunk)]

    def e2e_step():
        cur = torch.cuda.current_stream()
        copy_in.wait_stream(cur)
        with torch.cuda.stream(copy_in):
            for i in range(nchunk):
                d_buf[i].copy_(h_in[i], non_blocking=True)
                arrived[i].record(copy_in)
        for i in range(nchunk):
            obs_i, act_i, actp_i = d_in[i]
            cur.wait_event(arrived[i])
            if i == 0:
                md.bi_filter(obs_i, act_i, w.K, q_out=d_q[0])
            else:
                md.bi_filter_continue(obs_i, act_i, actp_i, w.K, q_out=d_q[i])
            done[i].record(cur)
            copy_out.wait_event(done[i])
            with torch.cuda.stream(copy_out):
                h_q[i].copy_(d_q[i], non_blocking=True)
        cur.wait_stream(copy_out)   # the step ends when the last block has reached the host

    e2e_times = time_steps(e2e_step, max(3, args.steps // 2), 3, flush, torch)
    e2e_sec = sum(e2e_times) / len(e2e_times)
    clocks = sampler.stop()  # sampled over both timed regions
    e2e_sec = max_over_ranks(dist, e2e_sec, "cuda")
    # the blockwise result is the single call's, bit for bit (the parity tests compare both with the oracle)
    torch.cuda.synchronize()
    blocks_equal = bool(torch.equal(torch.cat(h_q, dim=1), q.cpu()))
    e2e = {"value": aggregate_throughput(w.updates, world, e2e_sec), "unit": UNIT,
           "h2d_bytes_per_step": int(w.obs.nbytes + w.act.nbytes), "d2h_bytes_per_step": int(q.numel() * 4),
           "blocks_of_steps": lens, "equals_single_call_bit_for_bit": blocks_equal}

    flops = algorithmic_flops(w)
    peak = FP64_PEAK_TFLOPS if args.arith == "f64" else FP32_PEAK_TFLOPS
    achieved = flops / head["seconds"] / 1e12
    roofline = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": None,
                "kernel": head["kernel"],
                "peak_source": f"derived: 148 SMs x {64 if args.arith == 'f64' else 128} lanes x 2 x 1.965 GHz"}
    roofline["traffic"] = NCU_DRAM_BYTES_PER_CALL.get(head["kernel"])
    # the same run's own measurements beside the derived peak: the rate of independent multiply-add
    # chains in this arithmetic, and a large device-to-device copy
    try:
        fma_peak = fma_probe(args.arith)
        src = torch.empty(1 << 28, dtype=torch.float32, device="cuda")   # 1 GiB
        dst = torch.empty_like(src)
        for _ in range(2):
            dst.copy_(src)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(5):
            dst.copy_(src)
        ev1.record()
        ev1.synchronize()
        copy_gbs = 5 * 2 * src.numel() * 4 / (ev0.elapsed_time(ev1) * 1e-3) / 1e9
        del src, dst
        roofline["measured_in_this_run"] = {"fma_tflops": fma_peak, "frac_of_fma": achieved / fma_peak,
                                            "copy_gbs": copy_gbs}
    except Exception as exc:  # noqa: BLE001  (a measurement aid must not fail the benchmark)
        roofline["measured_in_this_run"] = {"error": str(exc)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": args.arith, "data": "synthetic",
        "config": {"workload": "config 2: variational filtering, 4096 agents sharing one model, "
                               "n=[8,8,6], m=[16,8,8], T=50, K=16",
                   "updates_per_step": w.updates, "l2": "flushed with a 256 MiB write before every timed step",
                   "agents_per_gpu": w.N, "ms_median": head["median"] * 1e3, "ms_best": head["best"] * 1e3,
                   "agent_steps_per_s": w.N * w.T * world / sec, "model_pack_ms": head["pack_ms"]},
        "e2e": e2e, "gpu_launches": head["launches_per_step"] * args.steps, "clocks": clocks,
        "roofline": roofline,
    }

    if rank == 0 and world == 1 and not args.no_extras:
        hbm_peak, hbm_src = measured_peaks()
        others = {}
        # the float32-arithmetic mode on the same workload
        alt = "f32" if args.arith == "f64" else "f64"
        r = bench_config(torch, bi, w, "filter", alt, max(3, args.steps // 2), 3, flush)
        others[f"config2_filter_{alt}"] = {"value": w.updates / r["seconds"], "unit": UNIT,
                                           "ms_per_step": r["seconds"] * 1e3, "kernel": r["kernel"]}
        # damped updates (step 0.5 on the log-beliefs): the iteration stops amplifying rounding errors,
        # so float32 arithmetic lands on the float64 result; both timed, and compared with each other
        damped = {}
        for ar in ("f64", "f32"):
            mdd = bi.model_from_workload(w, arith=ar)
            mdd.set_damping(0.5)
            qd = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
            ts = time_steps(lambda: mdd.bi_filter(head["obs"], head["act"], w.K, q_out=qd), max(3, args.steps // 2),
                            3, flush, torch)
            damped[ar] = (sum(ts) / len(ts), qd, mdd.last_kernel)
            mdd.close()
        dd = (damped["f32"][1] - damped["f64"][1]).abs().reshape(w.N, -1).max(dim=1).values
        others["config2_filter_damped_0.5"] = {
            "f64": {"value": w.updates / damped["f64"][0], "unit": UNIT, "ms_per_step": damped["f64"][0] * 1e3,
                    "kernel": damped["f64"][2]},
            "f32": {"value": w.updates / damped["f32"][0], "unit": UNIT, "ms_per_step": damped["f32"][0] * 1e3,
                    "kernel": damped["f32"][2]},
            "f32_vs_f64_max_abs_diff": float(dd.max()),
            "agents_within_1e-5": float((dd <= 1e-5).float().mean())}
        del damped, dd
        for c, algo in ((3, "vmp"), (4, "mmp")):
            wc = make_config(c)
            r = bench_config(torch, bi, wc, algo, args.arith, max(3, args.steps // 2), 3, flush)
            tfl = algorithmic_flops(wc) / r["seconds"] / 1e12
            entry = {"value": wc.updates / r["seconds"], "unit": UNIT, "ms_per_step": r["seconds"] * 1e3,
                     "kernel": r["kernel"], "launches_per_step": r["launches_per_step"], "alu_tflops": tfl}
            traffic = NCU_DRAM_BYTES_PER_CALL.get(r["kernel"])
            if wc.G == 1:
                # the shared model stays on chip / in L2: the arithmetic pipe bounds the call
                entry["roofline"] = {"bound": "alu", "achieved": tfl, "peak": peak, "unit": "TFLOP/s",
                                     "frac": tfl / peak, "traffic": traffic,
                                     "peak_source": roofline["peak_source"]}
            else:
                # per-agent models: every slice crosses HBM once.  Two byte counts: the slices as the
                # handle stores them (float64 logs in this arithmetic), and the float32 slices the method
                # itself needs (4 bytes per entry of A)
                stored = algorithmic_bytes(wc, 8 if args.arith == "f64" else 4)
                method = algorithmic_bytes(wc, 4)
                gbs = stored / r["seconds"] / 1e9
                entry["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s",
                                     "frac": gbs / hbm_peak, "traffic": traffic, "peak_source": hbm_src,
                                     "bytes_as_stored": stored, "bytes_of_the_method_fp32": method,
                                     "frac_on_the_method_bytes": method / r["seconds"] / 1e9 / hbm_peak}
            others[f"config{c}_{algo}_{args.arith}"] = entry
            del r
        # the headline workload with its observations given as categorical vectors (one-hot here):
        # the call forms sum_o o[o] ln A[o, .] per (agent, step) first, then runs the same kernels
        off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
        soft = np.zeros((w.N, w.T, int(off[-1])), np.float32)
        for i in range(w.M):
            np.put_along_axis(soft[:, :, off[i]:off[i + 1]], w.obs[:, :, i:i + 1], 1.0, axis=2)
        d_soft = torch.from_numpy(soft).cuda()
        md_s = bi.model_from_workload(w, arith=args.arith)
        d_act_s = torch.from_numpy(w.act).cuda()
        q_s = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
        l0 = md_s.launch_count
        ts = time_steps(lambda: md_s.run_soft("filter", d_soft, d_act_s, w.K, q_out=q_s), max(3, args.steps // 4), 3,
                        flush, torch)
        sec_s = sum(ts) / len(ts)
        slice_flops = 2.0 * w.N * w.T * float(off[-1]) * sum(int(np.prod([w.n[f] for f in d])) for d in w.dep[:1])
        others[f"config2_filter_soft_{args.arith}"] = {
            "value": w.updates / sec_s, "unit": UNIT, "ms_per_step": sec_s * 1e3, "kernel": md_s.last_kernel,
            "launches_per_step": (md_s.launch_count - l0) // (max(3, args.steps // 4) + 3),
            "slice_forming_gflop": slice_flops / 1e9}
        md_s.close()
        del d_soft, q_s
        # configuration 4 again with the handle's compressed slices switched on (sparse per-agent models:
        # a mask per lane and the values above the floor; bit for bit the dense result), with both sizes
        w4 = make_config(4)
        md4 = bi.model_from_workload(w4, arith=args.arith)
        d_obs4, d_act4 = torch.from_numpy(w4.obs).cuda(), torch.from_numpy(w4.act).cuda()
        q4 = torch.empty((w4.N, w4.T, w4.S), dtype=torch.float32, device="cuda")
        dense_b, comp_b = md4.slice_bytes()
        if comp_b:
            md4.set_compressed(True)
            ts = time_steps(lambda: md4.bi_mmp(d_obs4, d_act4, w4.K, q_out=q4), max(3, args.steps // 4), 3, flush, torch)
            sec4 = sum(ts) / len(ts)
            others[f"config4_mmp_compressed_{args.arith}"] = {
                "value": w4.updates / sec4, "unit": UNIT, "ms_per_step": sec4 * 1e3, "kernel": md4.last_kernel,
                "slice_bytes_dense": int(dense_b), "slice_bytes_compressed": int(comp_b)}
        md4.close()
        del d_obs4, d_act4, q4, w4
        # a model with non-trivial B-dependencies (transitions that read other factors' previous states):
        # config 3's factors and modalities, every factor's transition depending on itself and its
        # neighbour; filtering and VMP on the general kernel that contracts transition tensors
        from biwl import make_model, sample_streams, Workload
        rngb = np.random.default_rng(4242)
        nb_, mb_, depb, Ub = [10, 10, 8, 6], [12, 10, 8, 6], [[0, 1], [1, 2], [0, 2, 3], [0, 1, 2, 3]], [3, 3, 3, 3]
        bdep = [[0, 1], [1, 2], [2, 3], [3, 0]]
        Ab, Bb, Db = make_model(rngb, nb_, mb_, depb, Ub, 1, bdep=bdep)
        Nb, Tb = 1024, 20
        ob_, ab_ = sample_streams(rngb, nb_, mb_, depb, Ub, 1, Ab, Bb, Db, Nb, Tb, bdep=bdep)
        wb = Workload(name="bdep", algo="filter", n=np.asarray(nb_, np.int32), m=np.asarray(mb_, np.int32), dep=depb,
                      U=np.asarray(Ub, np.int32), G=1, A=Ab, B=Bb, D=Db, N=Nb, T=Tb, K=16, obs=ob_, act=ab_, bdep=bdep)
        entry = {}
        for algo in ("filter", "vmp"):
            r = bench_config(torch, bi, wb, algo, args.arith, 3, 3, flush)
            entry[algo] = {"value": wb.updates / r["seconds"], "unit": UNIT, "ms_per_step": r["seconds"] * 1e3,
                           "kernel": r["kernel"]}
            del r
        entry["workload"] = "1024 agents, n=[10,10,8,6], T=20, K=16, two parents per transition"
        others[f"bdep_{args.arith}"] = entry
        # configuration 1 (8 agents, 0.5 KB working set): latency per call, beside a one-element fill
        # kernel timed the same way (what a launch alone costs here)
        w1 = make_config(1)
        small_flush = torch.empty(0, dtype=torch.uint8, device="cuda")  # nothing to flush: below L2 anyway
        r = bench_config(torch, bi, w1, "filter", args.arith, 20, 3, small_flush)
        one = torch.empty(1, device="cuda")
        null_times = time_steps(lambda: one.zero_(), 20, 3, small_flush, torch)
        others[f"config1_filter_{args.arith}"] = {"us_per_call": r["seconds"] * 1e6, "kernel": r["kernel"],
                                                  "one_element_fill_us": sum(null_times) / len(null_times) * 1e6,
                                                  "value": w1.updates / r["seconds"], "unit": UNIT}
        del r
        # configuration 5: 128 random structures (256 agents, T=10 each), all three algorithms;
        # aggregate = sum of updates / sum of device time, plus the per-structure spread
        from biwl import make_sweep_config, SWEEP_SIZE
        sweep = {}
        members = [make_sweep_config(j) for j in range(SWEEP_SIZE)]
        for algo in ("filter", "vmp", "mmp"):
            tot_u, tot_s, rates, kernels = 0, 0.0, [], {}
            for wj in members:
                r = bench_config(torch, bi, wj, algo, args.arith, 2, 1, small_flush)
                tot_u += wj.updates
                tot_s += r["seconds"]
                rates.append(wj.updates / r["seconds"])
                kernels[r["kernel"]] = kernels.get(r["kernel"], 0) + 1
                del r
            rates.sort()
            sweep[algo] = {"value": tot_u / tot_s, "unit": UNIT, "min": rates[0], "median": rates[len(rates) // 2],
                           "max": rates[-1], "ms_total": tot_s * 1e3, "kernels": kernels}
        sweep["cap_entries_per_modality"] = 2 ** 18
        others[f"config5_sweep_{args.arith}"] = sweep
        line["others"] = others
        # ---- the oracle on this machine's host cores, on a bounded sample of the workload
        import oracle
        sample = 1024
        sub = w.take_agents(range(sample))
        t0 = time.perf_counter()
        ref_q = oracle.run_workload(sub)[0]
        dt = time.perf_counter() - t0
        # the same agents from the timed GPU call, while the oracle's result is at hand
        parity_err = float(np.abs(q[:sample].cpu().numpy() - ref_q).max())
        cores = oracle.max_threads()
        one = w.take_agents(range(64))
        t0 = time.perf_counter()
        oracle.run_workload(one, threads=1)
        dt1 = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": sub.updates / dt, "unit": UNIT, "cores": cores,
                                "kind": "oracle", "sample": f"first {sample} of 4096 agents, all 50 steps, "
                                                            f"16 iterations ({dt:.1f} s wall)",
                                "gpu_max_abs_err_on_sample": parity_err,
                                "single_thread_value": one.updates / dt1,
                                "single_thread_sample": f"first 64 agents ({dt1:.1f} s)"}
    elif rank == 0:
        line["cpu_baseline"] = None

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
