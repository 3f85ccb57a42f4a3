"""Shared comparison rules for GPU-vs-oracle parity tests.

Tolerances: beliefs within 1e-5 absolute per entry; log-beliefs within 1e-4
absolute where the oracle's log-belief is >= -30 and within 1e-5 relative below
that (float32 spacing at -150 is already 1.5e-5); argmax identical wherever the
oracle's two largest beliefs of that factor differ by more than 2e-5.
"""
from __future__ import annotations

import numpy as np

Q_TOL = 1e-5
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
        assert np.abs(blk.sum(-1) - 1.0).max(initial=0.0) <= 1e-5
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
        assert np.abs(blk.sum(-1) - 1.0).max(initial=0.0) <= 1e-5
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


def oracle_self_sensitivity(w, algo, eps=1e-13, seed=0):
    """Per-agent maximum change of the oracle's own beliefs when its uniform
    start is perturbed by a relative ``eps``: the conditioning of the K-step
    Jacobi iteration for that agent.  (On sharp or sparse models the iteration
    is chaotic: one ulp in the start can flip beliefs.)"""
    import oracle
    ref = oracle.run_workload(w, algo)[0]
    N, T = w.obs.shape[:2]
    start = np.concatenate([np.full((N, T, int(n)), 1.0 / n) for n in w.n], axis=2)
    start = start * (1.0 + eps * np.random.default_rng(seed).standard_normal(start.shape))
    pert = oracle.run_workload(w, algo, q_init=start)[0]
    return np.abs(pert - ref).reshape(N, -1).max(axis=1)


def compare_conditioned(w, algo, q_gpu, lq_gpu, am_gpu, ref):
    """Parity with the conditioning taken into account.  Agents whose oracle
    result moves by less than 1e-9 under a 1e-13 perturbation get the full
    strict comparison (beliefs 1e-5, log-beliefs, argmax).  Every other agent
    must still be a valid distribution and no further from the oracle than
    max(1e-5, 10 x the oracle's own movement) (a fully chaotic agent, whose
    oracle result flips under the probe, is only checked for validity)."""
    stats = error_stats(w, q_gpu, ref[0])
    moved = oracle_self_sensitivity(w, algo)
    err = np.abs(np.asarray(q_gpu, np.float64) - ref[0]).reshape(ref[0].shape[0], -1).max(axis=1)
    assert (err <= np.maximum(Q_TOL, 10.0 * moved)).all(), (err.max(), moved[err.argmax()])
    well = np.flatnonzero(moved < 1e-9)
    if len(well):
        sub = w.take_agents(well)
        compare(sub, q_gpu[well], lq_gpu[well] if lq_gpu is not None else None,
                am_gpu[well] if am_gpu is not None else None, ref[0][well], ref[1][well], ref[2][well])
    stats["well_conditioned_agents"] = int(len(well))
    stats["agents"] = int(len(err))
    return stats


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
    else:
        out = compare(sub, q, lq, am, *ref) if strict else error_stats(sub, q, ref[0])
    out["kernel"] = md.last_kernel
    md.close()
    return out
