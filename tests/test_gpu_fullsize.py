"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times: the CUDA library runs the whole workload, the oracle a sample of agents
(agents are independent, so a sampled agent's result is the full problem's)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from biwl import make_config, make_sweep_config, SWEEP_SIZE  # noqa: E402
from parity import check_workload, error_stats, run_gpu  # noqa: E402


def test_config2_full_size_every_agent():
    w = make_config(2)
    res = check_workload(w, "filter")          # all 4096 agents, all 50 steps
    print(res)
    assert res["kernel"] == "tile3_filter_f64"


def test_config2_full_size_in_blocks_of_steps_every_agent():
    # the end-to-end run of bench.py: five consecutive blocks of ten steps (bi_filter, then
    # bi_filter_continue four times), compared with the oracle on all 4096 agents
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    from parity import compare
    w = make_config(2)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    lq = torch.empty((w.N, w.T, w.S), device="cuda")
    am = torch.empty((w.N, w.T, w.F), dtype=torch.int32, device="cuda")
    q = torch.empty((w.N, w.T, w.S), device="cuda")
    nb = 5
    tc = w.T // nb
    for i in range(nb):
        t0 = i * tc
        o = obs[:, t0:t0 + tc].contiguous()
        a = act[:, t0:t0 + tc - 1].contiguous()
        outs = [torch.empty((w.N, tc, d), dtype=dt, device="cuda") for d, dt in
                ((w.S, torch.float32), (w.S, torch.float32), (w.F, torch.int32))]
        if i == 0:
            md.bi_filter(o, a, w.K, q_out=outs[0], logq_out=outs[1], argmax_out=outs[2])
        else:
            md.bi_filter_continue(o, a, act[:, t0 - 1].contiguous(), w.K, q_out=outs[0], logq_out=outs[1],
                                  argmax_out=outs[2])
        q[:, t0:t0 + tc], lq[:, t0:t0 + tc], am[:, t0:t0 + tc] = outs
    torch.cuda.synchronize()
    assert md.last_kernel == "tile3_filter_f64" and md.status() == 0
    whole = md.bi_filter(obs, act, w.K).cpu().numpy()
    assert np.array_equal(q.cpu().numpy(), whole)
    print(compare(w, q.cpu().numpy(), lq.cpu().numpy(), am.cpu().numpy(), *oracle.run_workload(w)))
    md.close()


def test_config3_full_size_sampled_agents():
    w = make_config(3)
    rng = np.random.default_rng(3)
    res = check_workload(w, "vmp", agents=np.sort(rng.choice(w.N, 192, replace=False)))
    print(res)


def test_config4_full_size_sampled_agents():
    # The sparse per-agent models make the Jacobi iteration chaotic for some
    # agents: the oracle's own result moves by up to 1e-4 when its uniform start
    # is perturbed by 1e-13 (amplification 1e9 in 16 iterations), so float64
    # rounding-order differences alone can exceed 1e-5 at full length there.
    # Every sampled agent must be at least as close to the oracle as the oracle is
    # to its own perturbed run (or within 1e-5), all but a few must be within 1e-5,
    # and every one of them passes the strict single-iteration comparisons.
    w = make_config(4)
    rng = np.random.default_rng(4)
    res = check_workload(w, "mmp", agents=np.sort(rng.choice(w.N, 256, replace=False)), conditioned=True)
    print(res)
    assert res["kernel"] == "tile3_mmp_f64"
    assert res["frac_agents_within_tol"] >= 0.98
    assert res["strict_comparisons"] >= 3


SWEEP_SAMPLE = np.unique(np.linspace(0, 255, 32).astype(int))   # 32 of the 256 agents of every structure


@pytest.mark.parametrize("algo", ["filter", "vmp", "mmp"])
def test_config5_every_member_sampled_agents(algo):
    # 128 random structures x 256 agents on the GPU, 32 sampled agents each on
    # the oracle.  Several sparse members are chaotic under filtering (one ulp in
    # the start flips the oracle's own beliefs), hence the conditioned comparison
    # of the full-length run; every sampled agent also goes through the strict
    # comparisons that nothing amplifies (one iteration, one step at a time).
    kernels, agents, within, well, beyond, strict, steps, steps_full = {}, 0, 0.0, 0, 0, 0, 0, 0
    for j in range(SWEEP_SIZE):
        w = make_sweep_config(j)               # 256 agents, T = 10, K = 16
        res = check_workload(w, algo, agents=SWEEP_SAMPLE, conditioned=True)
        kernels[res["kernel"]] = kernels.get(res["kernel"], 0) + 1
        agents += res["agents"]
        within += res["frac_agents_within_tol"] * res["agents"]
        well += res["well_conditioned_agents"]
        beyond += res["agents_beyond_tol_at_full_length"]
        strict += res["strict_comparisons"]
        steps += res.get("single_steps", 0)
        steps_full += res.get("single_steps_strict_at_full_K", 0)
    print(algo, kernels, f"sampled agents {agents}, within 1e-5 at full length: {within / agents:.4f} "
          f"(beyond: {beyond}), well conditioned: {well}, strict comparison batches: {strict}, "
          f"single filtering steps: {steps} (strict at full K: {steps_full})")
    assert within / agents > 0.9
    assert strict >= 3 * SWEEP_SIZE


def test_config5_every_structure_with_the_extended_call_forms():
    """Continued calls, warm starts, observation vectors and damping on all 128 random
    structures, on a small batch (warp / CTA kernels) and on the sweep's own 256 agents
    (batched kernels), three agents each against the oracle."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    rng = np.random.default_rng(123)
    worst = 0.0
    for j in range(SWEEP_SIZE):
        for N in (9, 256):
            w = make_sweep_config(j, N=N, T=10, K=6)
            md = bi.model_from_workload(w)
            obs = torch.from_numpy(w.obs).cuda()
            act = torch.from_numpy(w.act).cuda() if w.act.size else None
            sel = [0, N // 2, N - 1]
            sub = w.take_agents(sel)
            q_prev = np.concatenate([rng.dirichlet(np.full(int(nf), 1.5), size=N) for nf in w.n], axis=1).astype(np.float32)
            act_prev = np.stack([rng.integers(0, int(u), size=N) for u in w.U], axis=1).astype(np.int32)
            q_init = np.concatenate([rng.dirichlet(np.full(int(nf), 2.0), size=(N, w.T)) for nf in w.n],
                                    axis=2).astype(np.float32)
            off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
            soft = np.zeros((N, w.T, int(off[-1])), np.float32)
            for i, mi in enumerate(w.m):
                soft[:, :, off[i]:off[i + 1]] = rng.dirichlet(np.full(int(mi), 0.7), size=(N, w.T))
            d_prev, d_ap = torch.from_numpy(q_prev).cuda(), torch.from_numpy(act_prev).cuda()
            for lam in (1.0, 0.5):
                md.set_damping(lam)
                kw = {} if lam == 1.0 else dict(damping=lam)
                for algo in ("filter", "vmp", "mmp"):
                    okw = dict(q_prev=q_prev[sel].astype(np.float64), act_prev=act_prev[sel])
                    q = md.run_from(algo, obs, act, d_prev, d_ap, w.K).cpu().numpy()[sel]
                    ref = oracle.run_workload(sub, algo, **okw, **kw)[0]
                    err = np.abs(q - ref).reshape(3, -1).max(axis=1)
                    if algo == "filter" and lam == 1.0 and err.max() > 1e-5:
                        # undamped filtering is chaotic on a few sparse structures: allow what the oracle
                        # itself moves by when the carried belief is perturbed in its last place
                        pert = okw["q_prev"] * (1.0 + 1e-13 * rng.standard_normal(okw["q_prev"].shape))
                        ref2 = oracle.run_workload(sub, algo, q_prev=pert, act_prev=okw["act_prev"])[0]
                        sens = np.abs(ref2 - ref).reshape(3, -1).max(axis=1)
                        assert ((err <= np.maximum(1e-5, 10 * sens)) | (sens > 0.05)).all(), (j, N, err, sens)
                        # ... and where the full length is ill conditioned, the same continued call is held
                        # to 1e-5 at iteration counts that amplify nothing
                        for Ks in (1, 2, 4):
                            qs = md.run_from(algo, obs, act, d_prev, d_ap, Ks).cpu().numpy()[sel]
                            import dataclasses
                            refs = oracle.run_workload(dataclasses.replace(sub, K=Ks), algo, **okw)[0]
                            es = np.abs(qs[:, :2] - refs[:, :2]).max()   # the first two steps: later ones recurse
                            assert es <= 1e-5, (j, N, Ks, es)
                    else:
                        assert err.max() <= 1e-5, (j, N, algo, lam, md.last_kernel, err)
                        worst = max(worst, float(err.max()))
                    if algo != "filter":
                        fn = md.bi_vmp_warm if algo == "vmp" else md.bi_mmp_warm
                        q = fn(obs, act, torch.from_numpy(q_init).cuda(), w.K).cpu().numpy()[sel]
                        ref = oracle.run_workload(sub, algo, q_init=q_init[sel].astype(np.float64), **kw)[0]
                        assert np.abs(q - ref).max() <= 1e-5, (j, N, algo, lam, "warm", md.last_kernel)
                    if lam == 1.0:
                        q = md.run_soft(algo, torch.from_numpy(soft).cuda(), act, w.K).cpu().numpy()[sel]
                        ref = oracle.run(algo, sub.n, sub.m, sub.dep, sub.U, sub.G, sub.A, sub.B, sub.D, None, sub.act,
                                         sub.K, obs_soft=soft[sel])[0]
                        assert np.abs(q - ref).max() <= 1e-5, (j, N, algo, "soft", md.last_kernel)
            assert md.status() == 0
            md.close()
    print("worst error of the asserted cases", worst)
