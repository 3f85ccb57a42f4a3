"""Shared comparison rules for GPU-vs-oracle parity tests.

Tolerances: beliefs within 1e-5 absolute per entry, every factor's beliefs
summing to 1 within 1e-6; log-beliefs within 1e-4 absolute where the oracle's
log-belief is >= -30 and within 1e-5 relative below that (float32 spacing at
-150 is already 1.5e-5); argmax identical wherever the oracle's two largest
beliefs of that factor differ by more than 2e-5.

Sixteen undamped Jacobi iterations amplify rounding differences without bound
on sparse or sharp models (the oracle's own result can flip under a 1e-13
perturbation of its start), so a full-length run of such an agent cannot be
held to 1e-5 by any arithmetic.  Those agents are not let off: ``strict_checks``
compares every agent element by element where nothing is amplified -- one
iteration at a time from the oracle's own iterate, one filtering step at a time
from the oracle's own previous belief -- with the plain tolerances.
"""
from __future__ import annotations

import numpy as np

Q_TOL = 1e-5
SUM_TOL = 1e-6
LOGQ_TOL = 1e-4
ARGMAX_GAP = 2e-5


def error_stats(w, q_gpu, q_ref):
    """Validity checks (finite, non-negative, normalised) plus per-agent maxima
    of the belief error; no tolerance is asserted."""
    q_gpu = np.asarray(q_gpu, np.float64)
    assert q_gpu.shape == q_ref.shape and np.isfinite(q_gpu).all()
    off = np.concatenate([[0], np.cumsum(w.n)]).astype(int)
    for f in range(len(w.n)):
        blk = q_gpu[..., off[f]:off[f + 1]]
        assert (blk >= 0).all()
        assert np.abs(blk.sum(-1) - 1.0).max(initial=0.0) <= SUM_TOL
    per_agent = np.abs(q_gpu - q_ref).reshape(q_ref.shape[0], -1).max(axis=1)
    return {"q_max_err": float(per_agent.max(initial=0.0)),
            "q_median_agent_err": float(np.median(per_agent)) if per_agent.size else 0.0,
            "frac_agents_within_tol": float((per_agent <= Q_TOL).mean()) if per_agent.size else 1.0}


def compare(w, q_gpu, lq_gpu, am_gpu, q_ref, lq_ref, am_ref):
    """Returns a dict of maxima; raises AssertionError on a violation."""
    q_gpu = np.asarray(q_gpu, np.float64)
    assert q_gpu.shape == q_ref.shape, (q_gpu.shape, q_ref.shape)
    assert np.isfinite(q_gpu).all()
    dq = np.abs(q_gpu - q_ref)
    res = {"q_max_err": float(dq.max()) if dq.size else 0.0}
    assert res["q_max_err"] <= Q_TOL, f"belief error {res['q_max_err']:.3e} > {Q_TOL}"
    off = np.concatenate([[0], np.cumsum(w.n)]).astype(int)
    for f in range(len(w.n)):
        blk = q_gpu[..., off[f]:off[f + 1]]
        assert (blk >= 0).all()
        assert np.abs(blk.sum(-1) - 1.0).max(initial=0.0) <= SUM_TOL
    if lq_gpu is not None:
        lq_gpu = np.asarray(lq_gpu, np.float64)
        assert np.isfinite(lq_gpu).all()
        tol = np.where(lq_ref >= -30.0, LOGQ_TOL, 1e-5 * np.abs(lq_ref) + 0.0)
        tol = np.maximum(tol, LOGQ_TOL * (lq_ref >= -30.0))
        dl = np.abs(lq_gpu - lq_ref)
        res["logq_max_err"] = float(dl.max()) if dl.size else 0.0
        bad = dl > tol
        assert not bad.any(), f"log-belief error {dl[bad].max():.3e} at oracle value {lq_ref[bad][0]:.3f}"
    if am_gpu is not None:
        am_gpu = np.asarray(am_gpu)
        ambiguous = 0
        for f in range(len(w.n)):
            blk = q_ref[..., off[f]:off[f + 1]]
            if blk.shape[-1] == 1:
                assert (am_gpu[..., f] == 0).all()
                continue
            top2 = np.sort(blk, axis=-1)[..., -2:]
            decided = (top2[..., 1] - top2[..., 0]) > ARGMAX_GAP
            ambiguous += int((~decided).sum())
            assert (am_gpu[..., f][decided] == am_ref[..., f][decided]).all(), "argmax mismatch"
            # undecided entries must still point at a near-maximal state
            pick = np.take_along_axis(blk, am_gpu[..., f][..., None].astype(np.int64), axis=-1)[..., 0]
            assert (top2[..., 1] - pick <= ARGMAX_GAP + 1e-12).all()
        res["argmax_ambiguous"] = ambiguous
    return res


def oracle_self_sensitivity(w, algo, eps=1e-13, seeds=(0, 1, 2)):
    """Per-agent maximum change of the oracle's own beliefs when its uniform
    start is perturbed by a relative ``eps`` (largest over a few random
    perturbations): the conditioning of the K-step Jacobi iteration for that
    agent.  (On sharp or sparse models the iteration is chaotic: one ulp in the
    start can flip beliefs.)"""
    import oracle
    ref = oracle.run_workload(w, algo)[0]
    N, T = w.obs.shape[:2]
    uniform = np.concatenate([np.full((N, T, int(n)), 1.0 / n) for n in w.n], axis=2)
    moved = np.zeros(N)
    for seed in seeds:
        start = uniform * (1.0 + eps * np.random.default_rng(seed).standard_normal(uniform.shape))
        pert = oracle.run_workload(w, algo, q_init=start)[0]
        moved = np.maximum(moved, np.abs(pert - ref).reshape(N, -1).max(axis=1))
    return moved


def compare_conditioned(w, algo, q_gpu, lq_gpu, am_gpu, ref):
    """The full-length run with its conditioning taken into account.  Agents
    whose oracle result moves by less than 1e-9 under 1e-13 perturbations of the
    start get the full strict comparison (beliefs 1e-5, log-beliefs, argmax).
    Every other agent must be a valid distribution and no further from the
    oracle than max(1e-5, 100 x the oracle's own movement): the kernels round in
    a different order at every operation of every iteration, not once at the
    start, so their deviation can exceed the probe's by such a factor.  What the
    full-length run cannot show for those agents, ``strict_checks`` does."""
    stats = error_stats(w, q_gpu, ref[0])
    moved = oracle_self_sensitivity(w, algo)
    err = np.abs(np.asarray(q_gpu, np.float64) - ref[0]).reshape(ref[0].shape[0], -1).max(axis=1)
    bad = err > np.maximum(Q_TOL, 100.0 * moved)
    assert not bad.any(), (err[bad], moved[bad])
    well = np.flatnonzero(moved < 1e-9)
    if len(well):
        sub = w.take_agents(well)
        compare(sub, q_gpu[well], lq_gpu[well] if lq_gpu is not None else None,
                am_gpu[well] if am_gpu is not None else None, ref[0][well], ref[1][well], ref[2][well])
    stats["well_conditioned_agents"] = int(len(well))
    stats["agents"] = int(len(err))
    stats["agents_beyond_tol_at_full_length"] = int((err > Q_TOL).sum())
    return stats


def _gpu_outputs(N, T, w):
    import torch
    return (torch.full((N, T, w.S), float("nan"), device="cuda"),
            torch.full((N, T, w.S), float("nan"), device="cuda"),
            torch.full((N, T, w.F), -7, dtype=torch.int32, device="cuda"))


def _numpy(q, lq, am):
    return q.cpu().numpy(), lq.cpu().numpy(), am.cpu().numpy()


def _one_step_problems(sub, q_ref, steps=None):
    """Every (agent, step >= 1) of ``sub`` as an agent of its own with T = 1 that continues from the
    oracle's belief of the step before (rounded to float32, the form the library takes it in).
    Per-agent models are repeated to match.  Returns (workload, q_prev float32, act_prev)."""
    from biwl import Workload
    n, T = sub.obs.shape[:2]
    ts = np.arange(1, T) if steps is None else np.asarray(steps)
    obs = np.ascontiguousarray(sub.obs[:, ts].reshape(n * len(ts), 1, sub.M))
    q_prev = np.ascontiguousarray(q_ref[:, ts - 1].reshape(n * len(ts), sub.S).astype(np.float32))
    act_prev = np.ascontiguousarray(sub.act[:, ts - 1].reshape(n * len(ts), sub.F))
    if sub.G == 1:
        A, B, D, G = sub.A, sub.B, sub.D, 1
    else:
        rep = len(ts)
        A = [np.repeat(a, rep, axis=0) for a in sub.A]
        B = [np.repeat(b, rep, axis=0) for b in sub.B]
        D = [np.repeat(d, rep, axis=0) for d in sub.D]
        G = n * rep
    ws = Workload(name=sub.name + "_steps", algo="filter", n=sub.n, m=sub.m, dep=sub.dep, U=sub.U, G=G, A=A, B=B, D=D,
                  N=n * len(ts), T=1, K=sub.K, obs=obs, act=np.zeros((n * len(ts), 0, sub.F), np.int32))
    return ws, q_prev, act_prev


def strict_checks(sub, algo, ref=None, arith="f64"):
    """Element-wise comparisons, at the plain tolerances, that every agent of ``sub`` must pass
    whatever its conditioning, because nothing in them is amplified by further iterations:

    * windows (VMP, MMP): one iteration from the uniform start; one iteration from the oracle's own
      iterate K/2 and one from its iterate K-1 (``bi_*_warm`` with ``iters = 1``, both sides starting
      from the same float32-rounded beliefs) -- the last of these is the final iteration of the full run;
    * filtering: the first step at K = 1, 2, 4 and the full K from the prior D; every later step run
      on its own from the oracle's previous belief (``bi_filter_from`` with T = 1, both sides from the
      same float32-rounded belief) at K = 1, 2, 4, and at the full K for the steps whose oracle result
      moves by less than 1e-9 when that belief is perturbed by 1e-13.

    Returns counts for the test's report."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    md = bi.model_from_workload(sub, arith=arith)
    n, T = sub.obs.shape[:2]
    obs = torch.from_numpy(sub.obs).cuda()
    act = torch.from_numpy(sub.act).cuda() if sub.act.size else None
    out = {"strict_comparisons": 0}

    def check(w, gpu, ref_):
        compare(w, *gpu, *ref_)
        out["strict_comparisons"] += 1

    if algo in ("vmp", "mmp"):
        q, lq, am = _gpu_outputs(n, T, sub)
        md.run(algo, obs, act, 1, q_out=q, logq_out=lq, argmax_out=am)
        check(sub, _numpy(q, lq, am), oracle.run_workload(dict_k(sub, 1), algo))
        warm = md.bi_vmp_warm if algo == "vmp" else md.bi_mmp_warm
        for k0 in sorted({max(sub.K // 2, 1), sub.K - 1} - {0}):
            start = oracle.run_workload(dict_k(sub, k0), algo)[0].astype(np.float32)
            q, lq, am = _gpu_outputs(n, T, sub)
            warm(obs, act, torch.from_numpy(start).cuda(), 1, q_out=q, logq_out=lq, argmax_out=am)
            check(sub, _numpy(q, lq, am), oracle.run_workload(dict_k(sub, 1), algo, q_init=start.astype(np.float64)))
    else:
        if ref is None:
            ref = oracle.run_workload(sub, "filter")
        first = sub_steps(sub, 0, 1)
        obs0 = torch.from_numpy(first.obs).cuda()
        for K in sorted({1, 2, 4, sub.K}):
            q, lq, am = _gpu_outputs(n, 1, sub)
            md.bi_filter(obs0, None, K, q_out=q, logq_out=lq, argmax_out=am)
            check(first, _numpy(q, lq, am), oracle.run_workload(dict_k(first, K), "filter"))
        if T > 1:
            # bound the pseudo-batch of per-agent models (each step repeats its agent's model)
            steps = None
            if sub.G != 1:
                per_model = sum(a[0].nbytes for a in sub.A)
                cap = max(1, int(256e6 // max(per_model * n, 1)))
                if cap < T - 1:
                    steps = np.unique(np.linspace(1, T - 1, cap).astype(int))
            ws, q_prev, act_prev = _one_step_problems(sub, ref[0], steps)
            mds = md if sub.G == 1 else bi.model_from_workload(ws, arith=arith)
            d_obs, d_qp, d_ap = (torch.from_numpy(x).cuda() for x in (ws.obs, q_prev, act_prev))
            okw = dict(q_prev=q_prev.astype(np.float64), act_prev=act_prev)
            for K in (1, 2, 4):
                q, lq, am = _gpu_outputs(ws.N, 1, ws)
                mds.bi_filter_from(d_obs, None, d_qp, d_ap, K, q_out=q, logq_out=lq, argmax_out=am)
                check(ws, _numpy(q, lq, am), oracle.run_workload(dict_k(ws, K), "filter", **okw))
            # the full iteration count, where one step on its own is well conditioned
            full = oracle.run_workload(ws, "filter", **okw)
            pert = okw["q_prev"] * (1.0 + 1e-13 * np.random.default_rng(0).standard_normal(q_prev.shape))
            moved = np.abs(oracle.run_workload(ws, "filter", q_prev=pert, act_prev=act_prev)[0] - full[0])
            well = np.flatnonzero(moved.reshape(ws.N, -1).max(axis=1) < 1e-9)
            q, lq, am = _gpu_outputs(ws.N, 1, ws)
            mds.bi_filter_from(d_obs, None, d_qp, d_ap, ws.K, q_out=q, logq_out=lq, argmax_out=am)
            gq, glq, gam = _numpy(q, lq, am)
            error_stats(ws, gq, full[0])
            if len(well):
                check(ws.take_agents(well), (gq[well], glq[well], gam[well]), tuple(x[well] for x in full))
            out["single_steps"] = int(ws.N)
            out["single_steps_strict_at_full_K"] = int(len(well))
            if mds is not md:
                mds.close()
    assert md.status() == 0
    md.close()
    return out


def dict_k(w, K):
    """The workload with another iteration count."""
    import dataclasses
    return dataclasses.replace(w, K=K)


def sub_steps(w, t0, t1):
    """The workload restricted to steps [t0, t1) (a window of its own, starting from the prior D)."""
    import dataclasses
    return dataclasses.replace(w, T=t1 - t0, obs=np.ascontiguousarray(w.obs[:, t0:t1]),
                               act=np.ascontiguousarray(w.act[:, t0:max(t1 - 1, t0)]))


def run_gpu(w, algo=None, want_logq=True, want_argmax=True, model=None, arith="f64"):
    """Run the CUDA library on a workload; returns numpy (q, logq, argmax, model)."""
    import torch
    import paper_2607_17855_b200 as bi
    algo = algo or w.algo
    md = model or bi.model_from_workload(w, arith=arith)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda() if w.act.size else None
    N, T = w.obs.shape[:2]
    q = torch.full((N, T, w.S), float("nan"), device="cuda")
    lq = torch.full((N, T, w.S), float("nan"), device="cuda") if want_logq else None
    am = torch.full((N, T, w.F), -7, dtype=torch.int32, device="cuda") if want_argmax else None
    md.run(algo, obs, act, w.K, q_out=q, logq_out=lq, argmax_out=am)
    torch.cuda.synchronize()
    assert md.status() == 0
    return (q.cpu().numpy(), lq.cpu().numpy() if lq is not None else None,
            am.cpu().numpy() if am is not None else None, md)


def check_workload(w, algo=None, agents=None, arith="f64", strict=True, conditioned=False):
    """GPU on the whole workload, oracle on ``agents`` (all if None); compares those.
    ``strict=False`` only checks validity and returns the error statistics."""
    import oracle
    algo = algo or w.algo
    q, lq, am, md = run_gpu(w, algo, arith=arith)
    sub = w
    if agents is not None:
        agents = np.asarray(agents)
        sub = w.take_agents(agents)
        q, lq, am = q[agents], lq[agents], am[agents]
    ref = oracle.run_workload(sub, algo)
    if conditioned:
        out = compare_conditioned(sub, algo, q, lq, am, ref)
        out.update(strict_checks(sub, algo, ref=ref, arith=arith))
    else:
        out = compare(sub, q, lq, am, *ref) if strict else error_stats(sub, q, ref[0])
    out["kernel"] = md.last_kernel
    md.close()
    return out
