"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle,
element by element on the same seeded inputs."""
import contextlib
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from biwl import make_config, make_model, make_sweep_config, sample_streams, Workload  # noqa: E402
from parity import check_workload, compare, run_gpu  # noqa: E402

ALGOS = ["filter", "vmp", "mmp"]


@contextlib.contextmanager
def family_forced(name):
    """The library's testing aid BI_TEST_FAMILY ("batch", "cta", "warp" or "generic"), read when a handle is made: its
    calls skip the kernel families ahead of the named one, so that the general kernels can be checked
    on oracle-sized inputs that would otherwise go to a specialised kernel."""
    old = os.environ.get("BI_TEST_FAMILY")
    os.environ["BI_TEST_FAMILY"] = name
    try:
        yield
    finally:
        if old is None:
            del os.environ["BI_TEST_FAMILY"]
        else:
            os.environ["BI_TEST_FAMILY"] = old


def warp_filter_forced():
    return family_forced("warp")


def _custom(seed, n, m, dep, U, N, T, K, G=1, sparsity=0.0):
    rng = np.random.default_rng(seed)
    A, B, D = make_model(rng, n, m, dep, U, G, sparsity=sparsity, d_alpha=1.0)
    obs, act = sample_streams(rng, n, m, dep, U, G, A, B, D, N, T)
    return Workload(name="custom", algo="filter", n=np.asarray(n, np.int32), m=np.asarray(m, np.int32),
                    dep=dep, U=np.asarray(U, np.int32), G=G, A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act)


@pytest.mark.parametrize("algo", ALGOS)
def test_config1(algo):
    print(check_workload(make_config(1), algo))


@pytest.mark.parametrize("case", ["tile", "pair"])
def test_unnormalised_likelihoods_far_above_one(case):
    """The inputs are used as given.  With entries of A far above 1 for some outcomes and far below for
    others, agents of one warp see logits hundreds of binary orders apart: the kernels that share one
    softmax shift among a warp's agents must then shift per agent."""
    import dataclasses
    w = make_config(2, N=41, T=6, K=6) if case == "tile" else make_config(1)
    scale = [10.0 ** e for e in (30, -8, 12, 0, -20, 25, 3, -3)]
    A = []
    for a in w.A:
        a = a.astype(np.float64)
        for o in range(a.shape[1]):
            a[:, o] *= scale[o % len(scale)]
        A.append(a.astype(np.float32))
    w = dataclasses.replace(w, A=A)
    res = check_workload(w, "filter", conditioned=True)
    print(case, res)
    assert res["kernel"] == ("tile3_filter_f64" if case == "tile" else "pair_filter_f64"), res


@pytest.mark.parametrize("algo", ALGOS)
def test_config2_small(algo):
    print(check_workload(make_config(2, N=96, T=12), algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_config3_small(algo):
    print(check_workload(make_config(3, N=48, T=9), algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_config4_small(algo):
    print(check_workload(make_config(4, N=24, T=7), algo))


@pytest.mark.parametrize("j", [0, 3, 7, 19, 42, 77, 101, 127])
@pytest.mark.parametrize("algo", ALGOS)
def test_sweep_members(j, algo):
    print(check_workload(make_sweep_config(j, N=12), algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_edge_single_step_single_agent_one_iteration(algo):
    w = _custom(5, [5, 3], [4, 6], [[0, 1], [1]], [2, 1], N=1, T=1, K=1)
    print(check_workload(w, algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_edge_singleton_and_unobserved_factors(algo):
    # factor 1 has a single state, factor 3 is in no dependency list
    w = _custom(6, [3, 1, 4, 5], [3, 2, 4], [[0, 1, 2], [1], [2, 0]], [2, 1, 3, 2], N=9, T=5, K=6)
    print(check_workload(w, algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_edge_maximum_state_counts_and_rank(algo):
    w = _custom(7, [32, 2, 3, 2, 31], [2, 3], [[4, 1, 2, 3, 0], [0]], [1, 2, 1, 4, 2], N=3, T=3, K=4, sparsity=0.5)
    print(check_workload(w, algo))


@pytest.mark.parametrize("algo", ALGOS)
def test_edge_per_agent_models_with_axis_permutation(algo):
    w = _custom(8, [6, 5, 7], [4, 3], [[2, 0, 1], [1, 2]], [2, 2, 2], N=5, T=4, K=5, G=5, sparsity=0.7)
    print(check_workload(w, algo))


def test_edge_no_agents_and_bad_arguments():
    import torch
    import paper_2607_17855_b200 as bi
    w = make_config(1)
    md = bi.model_from_workload(w)
    empty = torch.empty((0, 3, w.M), dtype=torch.int32, device="cuda")
    q = md.bi_filter(empty, torch.empty((0, 2, w.F), dtype=torch.int32, device="cuda"), 4)
    assert q.shape == (0, 3, w.S)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda()
    with pytest.raises(bi.BiError) as e:
        md.bi_filter(obs, act, 0)
    assert e.value.code == -1
    with pytest.raises(bi.BiError) as e:
        md.bi_vmp(obs.repeat(1, 10, 1), act.repeat(1, 11, 1), 2)  # T = 100 > BI_MAX_T
    assert e.value.code == -3
    md.close()


def test_out_of_range_indices_are_clamped_and_flagged():
    import torch
    import paper_2607_17855_b200 as bi
    w = make_config(1)
    md = bi.model_from_workload(w)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda()
    md.bi_filter(obs, act, 2)
    assert md.status() == 0
    bad = obs.clone()
    bad[0, 0, 0] = 99
    q = md.bi_filter(bad, act, 2)
    assert md.status() == bi.BI_FLAG_OBS_RANGE
    assert torch.isfinite(q).all()
    bad_act = act.clone()
    bad_act[1, 0, 0] = -3
    md.bi_vmp(obs, bad_act, 2)
    assert md.status() == bi.BI_FLAG_ACT_RANGE
    assert md.status() == 0
    md.close()


def test_shared_model_equals_replicated_model():
    w = make_config(3, N=6, T=5)
    q1, l1, a1, m1 = run_gpu(w, "vmp")
    rep = Workload(name="rep", algo="vmp", n=w.n, m=w.m, dep=w.dep, U=w.U, G=w.N,
                   A=[np.repeat(a, w.N, axis=0) for a in w.A], B=[np.repeat(b, w.N, axis=0) for b in w.B],
                   D=[np.repeat(d, w.N, axis=0) for d in w.D], N=w.N, T=w.T, K=w.K, obs=w.obs, act=w.act)
    q2, l2, a2, m2 = run_gpu(rep, "vmp")
    np.testing.assert_allclose(q2, q1, atol=2e-6)
    assert (a1 == a2).all()
    m1.close(); m2.close()


# ---- float32 arithmetic: valid beliefs everywhere; 1e-5 wherever the iteration
# is well conditioned (the oracle itself moves by more than 1e-5 on some agents
# when its beliefs and logs are merely rounded to float32 each iteration).

@pytest.mark.parametrize("c,algo,kw", [(1, "filter", {}), (2, "filter", dict(N=96, T=12)),
                                       (3, "vmp", dict(N=48, T=9)), (4, "mmp", dict(N=24, T=7))])
def test_float32_arithmetic_mode(c, algo, kw):
    import oracle
    w = make_config(c, **kw)
    res = check_workload(w, algo, arith="f32", strict=False)
    print(res)
    assert res["kernel"].endswith("_f32")
    ref = oracle.run_workload(w, algo)[0]
    probe = oracle.run_workload(w, algo, round32=True)[0]
    floor = np.abs(probe - ref).reshape(w.N, -1).max(axis=1)
    q = run_gpu(w, algo, arith="f32")[0]
    err = np.abs(q - ref).reshape(w.N, -1).max(axis=1)
    well = floor < 1e-7  # agents whose result barely moves under float32 rounding of the state
    assert well.any() or c == 4
    assert (err[well] <= 1e-5).all()


# ---- the register-tile filtering kernels (single rank-3 dependency group)

@pytest.mark.parametrize("arith", ["f64", "f32"])
def test_tile_filter_shapes_and_ragged_batches(arith):
    strict = arith == "f64"
    # 8 lanes per agent, 4 agents per warp: a batch that does not fill the last warp
    res = check_workload(make_config(2, N=97, T=7), "filter", arith=arith, strict=strict)
    assert res["kernel"] == f"tile3_filter_{arith}", res
    # 32 lanes per agent, per-agent models
    res = check_workload(make_config(4, N=5, T=6), "filter", arith=arith, strict=strict)
    assert res["kernel"] == f"tile3_filter_{arith}", res
    # padded lanes: n = [4, 3, 2] packs as a = 3 (4 lanes), b = 2, c = 4
    w = _custom(31, [4, 3, 2], [3, 5, 2], [[0, 1, 2], [2, 0, 1], [1, 2, 0]], [2, 3, 1], N=11, T=5, K=9,
                sparsity=0.5 if strict else 0.0)
    res = check_workload(w, "filter", arith=arith, strict=strict)
    assert res["kernel"] == f"tile3_filter_{arith}", res
    if not strict:
        assert res["q_max_err"] < 1e-3
    # a tile kept in shared memory instead of registers (packed dims 10 x 6 x 8)
    w = _custom(36, [10, 6, 8], [4, 3], [[0, 1, 2], [1, 2, 0]], [2, 1, 3], N=7, T=5, K=6)
    res = check_workload(w, "filter", arith=arith, strict=strict)
    assert res["kernel"] == f"tile3_filter_{arith}", res


# ---- the register-tile window kernels (VMP / MMP), incl. multi-CTA clusters

@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_tile_window_kernels(algo):
    # 8 lanes per step, 4 steps per warp; T not a multiple of 4
    res = check_workload(make_config(2, N=9, T=11, K=7), algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    # 32 lanes per step; float64 slices of 20 steps exceed one SM: two-CTA cluster
    res = check_workload(make_config(4, N=6, T=20, K=8), algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    # odd split over the cluster (T = 19 -> 10 + 9), and a window of a single step
    res = check_workload(make_config(4, N=3, T=19, K=5), algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    res = check_workload(make_config(4, N=3, T=1, K=5), algo)
    # the longest window: four-CTA cluster
    res = check_workload(make_config(4, N=2, T=64, K=3), algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    # padded lanes
    w = _custom(33, [4, 3, 2], [3, 5], [[0, 1, 2], [2, 0, 1]], [2, 3, 1], N=7, T=6, K=9, sparsity=0.5)
    res = check_workload(w, algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    # a tile kept in shared memory instead of registers (packed dims 10 x 6 x 8)
    w = _custom(35, [10, 6, 8], [4, 3], [[0, 1, 2], [1, 2, 0]], [2, 1, 3], N=5, T=9, K=6)
    res = check_workload(w, algo)
    assert res["kernel"] == f"tile3_{algo}_f64", res
    # float32 arithmetic: single CTA holds the window
    res = check_workload(make_config(4, N=4, T=20, K=8), algo, arith="f32", strict=False)
    assert res["kernel"] == f"tile3_{algo}_f32", res


def test_tile_window_small_tile_across_a_cluster():
    # 8 lanes per step with the slices in registers: a 40-step window is split
    # over several CTAs of a cluster (the thread cap of the register variant)
    res = check_workload(make_config(2, N=5, T=40, K=6), "vmp")
    assert res["kernel"] == "tile3_vmp_f64", res
    res = check_workload(make_config(2, N=5, T=64, K=4), "mmp")
    assert res["kernel"] == "tile3_mmp_f64", res


# ---- batched window kernels (shared model, units bucketed by observed outcome)

@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_batched_window_kernels(algo):
    res = check_workload(make_config(3, N=128, T=16, K=9), algo, agents=range(0, 128, 5))
    assert res["kernel"] == f"batch_{algo}_f64", res
    # rank-3 and rank-2 groups, a single-factor modality, an unobserved factor, odd sizes
    w = _custom(41, [3, 4, 2, 5, 3], [3, 2, 4, 3], [[0, 1, 2], [3, 4], [1], [2, 0, 1]], [2, 1, 3, 2, 2],
                N=171, T=12, K=7, sparsity=0.5)
    res = check_workload(w, algo, agents=range(0, 171, 7))
    assert res["kernel"] == f"batch_{algo}_f64", res
    res = check_workload(make_config(3, N=160, T=13, K=5), algo, arith="f32", strict=False)
    assert res["kernel"] == f"batch_{algo}_f32", res


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_batched_any_shape(algo):
    # rank 5 with a two-state last axis (padded to 4); last axes of 7, 13 and 32 states; a slice of
    # 20 x 20 x 20 that is staged in several pieces; a single-factor modality
    w = _custom(43, [3, 4, 5, 3, 2], [3, 4, 2], [[0, 1, 2, 3, 4], [1, 2], [3]], [2, 1, 2, 3, 1],
                N=150, T=14, K=6, sparsity=0.5)
    res = check_workload(w, algo, agents=range(0, 150, 6))
    assert res["kernel"] == f"batch_{algo}_f64", res
    w = _custom(44, [7, 13, 32, 9], [5, 3, 2, 6], [[0, 1], [1, 2], [0, 3, 2], [3, 0]], [2, 2, 1, 3],
                N=128, T=16, K=5)
    res = check_workload(w, algo, agents=range(0, 128, 5))
    assert res["kernel"] == f"batch_{algo}_f64", res
    w = _custom(45, [20, 20, 20], [3, 2], [[0, 1, 2], [2, 0]], [1, 2, 2], N=129, T=16, K=4, sparsity=0.9)
    res = check_workload(w, algo, agents=range(0, 129, 8), conditioned=True)
    assert res["kernel"] == f"batch_{algo}_f64", res
    res = check_workload(w, algo, arith="f32", strict=False)
    assert res["kernel"] == f"batch_{algo}_f32", res


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_batched_single_factor_modalities_only(algo):
    # no contraction at all: the observed slices are the messages
    w = _custom(46, [5, 9], [4, 3, 6], [[0], [1], [0]], [2, 3], N=150, T=14, K=5)
    with family_forced("batch"):   # (by itself the dispatcher gives such a model to the pair window kernel)
        res = check_workload(w, algo, agents=range(0, 150, 4))
    assert res["kernel"] == f"batch_{algo}_f64", res
    res = check_workload(w, algo, agents=range(0, 150, 4))
    assert res["kernel"] == f"pair_{algo}_f64", res


# ---- filtering continued from a known belief (bi_filter_from)

def _continued(w, cut, arith="f64"):
    """Run the first `cut` steps with bi_filter, the rest with bi_filter_from; returns the joined
    beliefs, the oracle's result for the same two calls, and the kernels used."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    md = bi.model_from_workload(w, arith=arith)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda()
    q_head = md.bi_filter(obs[:, :cut].contiguous(), act[:, :cut - 1].contiguous(), w.K)
    q_prev = q_head[:, -1].contiguous()
    act_prev = act[:, cut - 1].contiguous()
    q_tail = md.bi_filter_from(obs[:, cut:].contiguous(), act[:, cut:].contiguous(), q_prev, act_prev, w.K)
    kernel = md.last_kernel
    assert md.status() == 0
    # the oracle continues from the very same float32 belief
    ref_tail = oracle.run("filter", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, w.obs[:, cut:], w.act[:, cut:], w.K,
                          q_prev=q_prev.cpu().numpy().astype(np.float64), act_prev=w.act[:, cut - 1])[0]
    md.close()
    return q_tail.cpu().numpy(), ref_tail, kernel


@pytest.mark.parametrize("case", ["tile", "warp", "cta", "per_agent"])
def test_filter_continuation(case):
    if case == "tile":
        w, kern = make_config(2, N=37, T=9, K=8), "tile3_filter_f64"
    elif case == "warp":
        w, kern = _custom(49, [5, 4, 3, 2], [3, 4], [[0, 1], [1, 2, 3]], [2, 2, 1, 2], N=21, T=7, K=6), "warp_filter_f64"
    elif case == "cta":   # few agents and large slices: a CTA per agent
        w, kern = make_config(3, N=21, T=7, K=6), "cta_filter_f64"
    else:
        w, kern = _custom(8, [6, 5, 7], [4, 3], [[2, 0, 1], [1, 2]], [2, 2, 2], N=5, T=6, K=5, G=5), None
    for cut in (1, 4):
        with (warp_filter_forced() if case == "warp" else contextlib.nullcontext()):
            q, ref, kernel = _continued(w, cut)
        if kern:
            assert kernel == kern, kernel
        assert np.abs(q - ref).max() <= 1e-5, (case, cut, np.abs(q - ref).max())
    # a single tick in place: q_prev and q_out are the same buffer
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    md = bi.model_from_workload(w)
    obs = torch.from_numpy(w.obs).cuda()
    act = torch.from_numpy(w.act).cuda()
    buf = md.bi_filter(obs[:, :1].contiguous(), None, w.K)          # [N, 1, S]
    start = buf[:, 0].cpu().numpy().astype(np.float64)
    md.bi_filter_from(obs[:, 1:2].contiguous(), None, buf.view(w.N, -1), act[:, 0].contiguous(), w.K, q_out=buf)
    ref = oracle.run("filter", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, w.obs[:, 1:2], w.act[:, :0], w.K,
                     q_prev=start, act_prev=w.act[:, 0])[0]
    assert np.abs(buf.cpu().numpy() - ref).max() <= 1e-5
    null = torch.empty(0, dtype=torch.int32, device="cuda")      # data_ptr() == 0
    with pytest.raises(bi.BiError) as e:
        md.bi_filter_from(obs[:, 1:2].contiguous(), None, buf.view(w.N, -1), null, w.K)
    assert e.value.code == -1
    md.close()


# ---- warm-started window algorithms (bi_vmp_warm / bi_mmp_warm)

def _random_beliefs(w, seed):
    rng = np.random.default_rng(seed)
    blocks = [rng.dirichlet(np.full(int(nf), 2.0), size=(w.N, w.T)) for nf in w.n]
    return np.concatenate(blocks, axis=2).astype(np.float32)


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
@pytest.mark.parametrize("case", ["tile", "tile_cluster", "batch", "warp", "per_agent", "pair"])
def test_warm_started_windows(case, algo):
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w, kern = {
        "tile": (make_config(2, N=9, T=11, K=3), f"tile3_{algo}_f64"),
        "tile_cluster": (make_config(4, N=4, T=20, K=3), f"tile3_{algo}_f64"),
        "batch": (make_config(3, N=128, T=16, K=3), f"batch_{algo}_f64"),
        "warp": (make_config(3, N=10, T=7, K=3), f"warp_{algo}_f64"),
        "per_agent": (_custom(8, [6, 5, 7], [4, 3], [[2, 0, 1], [1, 2]], [2, 2, 2], N=5, T=6, K=3, G=5), None),
        "pair": (_custom(92, [6, 8, 3, 1], [4, 3, 2, 5], [[1, 0], [2], [0], [3]], [2, 1, 3, 1], N=11, T=5, K=3),
                 f"pair_{algo}_f64"),
    }[case]
    q_init = _random_beliefs(w, 77)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    fn = md.bi_vmp_warm if algo == "vmp" else md.bi_mmp_warm
    lq = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
    q = fn(obs, act, torch.from_numpy(q_init).cuda(), w.K, logq_out=lq).cpu().numpy()
    if kern:
        assert md.last_kernel == kern, md.last_kernel
    assert md.status() == 0
    sel = list(range(0, w.N, max(1, w.N // 16)))
    sub = w.take_agents(sel)
    ref, lref, _ = oracle.run_workload(sub, algo, q_init=q_init[sel].astype(np.float64))
    assert np.abs(q[sel] - ref).max() <= 1e-5, np.abs(q[sel] - ref).max()
    big = lref > -30
    assert np.abs(lq.cpu().numpy()[sel][big] - lref[big]).max() <= 1e-4
    # and the start matters: the uniform-start call gives something else after so few sweeps
    q_cold = md.run(algo, obs, act, w.K).cpu().numpy()
    assert np.abs(q_cold - q).max() > 1e-4
    md.close()


# ---- observations as categorical vectors (bi_filter_soft / bi_vmp_soft / bi_mmp_soft)

def _soft_vectors(w, seed, sharp=False):
    """Random categorical vectors per modality; `sharp` gives one-hot vectors of w.obs."""
    off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
    out = np.zeros((w.N, w.T, int(off[-1])), np.float32)
    rng = np.random.default_rng(seed)
    for i, mi in enumerate(w.m):
        if sharp:
            np.put_along_axis(out[:, :, off[i]:off[i + 1]], w.obs[:, :, i:i + 1], 1.0, axis=2)
        else:
            out[:, :, off[i]:off[i + 1]] = rng.dirichlet(np.full(int(mi), 0.7), size=(w.N, w.T))
    return out


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("case", ["tile_shared", "tile_per_agent", "groups", "mixed_ranks"])
def test_soft_observations(case, algo):
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = {
        "tile_shared": make_config(2, N=21, T=9, K=4),
        "tile_per_agent": make_config(4, N=5, T=6, K=4),
        "groups": make_config(3, N=12, T=7, K=4),
        "mixed_ranks": _custom(51, [3, 4, 2, 5, 3], [3, 2, 4, 3], [[0, 1, 2], [3, 4], [1], [2, 0, 1]], [2, 1, 3, 2, 2],
                               N=9, T=8, K=4, sparsity=0.5),
    }[case]
    md = bi.model_from_workload(w)
    act = torch.from_numpy(w.act).cuda()
    # one-hot vectors reproduce the index form
    hard = md.run(algo, torch.from_numpy(w.obs).cuda(), act, w.K).cpu().numpy()
    sharp = md.run_soft(algo, torch.from_numpy(_soft_vectors(w, 0, sharp=True)).cuda(), act, w.K).cpu().numpy()
    assert np.abs(sharp - hard).max() <= 2e-6, np.abs(sharp - hard).max()
    # random vectors against the oracle
    soft = _soft_vectors(w, 5)
    lq = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
    am = torch.empty((w.N, w.T, w.F), dtype=torch.int32, device="cuda")
    q = md.run_soft(algo, torch.from_numpy(soft).cuda(), act, w.K, logq_out=lq, argmax_out=am).cpu().numpy()
    assert md.status() == 0
    ref, lref, amref = oracle.run(algo, w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, None, w.act, w.K, obs_soft=soft)
    print(case, algo, md.last_kernel, np.abs(q - ref).max())
    assert np.abs(q - ref).max() <= 1e-5
    big = lref > -30
    assert np.abs(lq.cpu().numpy()[big] - lref[big]).max() <= 1e-4
    # argmax wherever the oracle's top two are further apart than the tolerance
    off = np.concatenate([[0], np.cumsum(w.n)]).astype(int)
    for f in range(w.F):
        blk = np.sort(ref[:, :, off[f]:off[f + 1]], axis=2)
        clear = (blk[:, :, -1] - blk[:, :, -2] > 2e-5) if blk.shape[2] > 1 else np.ones(blk.shape[:2], bool)
        assert (am.cpu().numpy()[:, :, f][clear] == amref[:, :, f][clear]).all()
    md.close()


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_batched_window_of_a_single_step(algo):
    # T = 1: no actions at all, every unit is both the first and the last step of its window
    w = _custom(47, [4, 6, 3], [3, 5], [[0, 1, 2], [1, 2]], [2, 2, 1], N=2100, T=1, K=5)
    res = check_workload(w, algo, agents=range(0, 2100, 50))
    assert res["kernel"] == f"batch_{algo}_f64", res


@pytest.mark.parametrize("arith", ["f64", "f32"])
@pytest.mark.parametrize("T", [12, 20, 27, 43, 70])
def test_soft_observations_long_trajectories(T, arith):
    """The slice-forming kernels take the steps in blocks (of 32 on the float64 tensor path, of 16 on the
    other) and the last steps in a shorter block: trajectories that end in every block length, on a
    model whose groups have slices of 24, 15, 4 and 24 (padded: 24, 16, 4, 24) elements."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = _custom(53, [3, 4, 2, 5, 3], [3, 2, 4, 3], [[0, 1, 2], [3, 4], [1], [2, 0, 1]], [2, 1, 3, 2, 2],
                N=5, T=T, K=3, sparsity=0.5)
    md = bi.model_from_workload(w, arith=arith)
    soft = _soft_vectors(w, 7)
    q = md.run_soft("filter", torch.from_numpy(soft).cuda(), torch.from_numpy(w.act).cuda(), w.K).cpu().numpy()
    assert md.status() == 0
    ref = oracle.run("filter", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, None, w.act, w.K, obs_soft=soft)[0]
    assert np.abs(q - ref).max() <= (1e-5 if arith == "f64" else 2e-3), np.abs(q - ref).max()
    # a register-tile model with per-agent slices of 384 elements: three blocks of 32 columns per warp
    w = make_config(2, N=7, T=T, K=3)
    md2 = bi.model_from_workload(w, arith=arith)
    soft = _soft_vectors(w, 8)
    q = md2.run_soft("filter", torch.from_numpy(soft).cuda(), torch.from_numpy(w.act).cuda(), w.K).cpu().numpy()
    ref = oracle.run("filter", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, None, w.act, w.K, obs_soft=soft)[0]
    assert np.abs(q - ref).max() <= (1e-5 if arith == "f64" else 2e-3), np.abs(q - ref).max()
    md.close()
    md2.close()


def test_soft_observations_single_step_and_empty_batch():
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = _custom(48, [4, 3], [3, 2], [[0, 1], [1]], [2, 2], N=6, T=1, K=3)
    md = bi.model_from_workload(w)
    soft = _soft_vectors(w, 9)
    q = md.run_soft("filter", torch.from_numpy(soft).cuda(), None, w.K).cpu().numpy()
    ref = oracle.run("filter", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, None, w.act, w.K, obs_soft=soft)[0]
    assert np.abs(q - ref).max() <= 1e-5
    empty = torch.empty((0, 3, 5), dtype=torch.float32, device="cuda")
    assert md.run_soft("vmp", empty, torch.empty((0, 2, 2), dtype=torch.int32, device="cuda"), 2).shape == (0, 3, w.S)
    md.close()


# ---- window algorithms continued from a belief (bi_vmp_from / bi_mmp_from)

@pytest.mark.parametrize("algo", ["vmp", "mmp"])
@pytest.mark.parametrize("case", ["tile", "tile_cluster", "batch", "warp", "per_agent", "pair"])
def test_continued_windows(case, algo):
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w, kern = {
        "tile": (make_config(2, N=9, T=11, K=4), f"tile3_{algo}_f64"),
        "tile_cluster": (make_config(4, N=4, T=20, K=4), f"tile3_{algo}_f64"),
        "batch": (make_config(3, N=128, T=16, K=4), f"batch_{algo}_f64"),
        "warp": (make_config(3, N=10, T=7, K=4), f"warp_{algo}_f64"),
        "per_agent": (_custom(8, [6, 5, 7], [4, 3], [[2, 0, 1], [1, 2]], [2, 2, 2], N=5, T=6, K=4, G=5), None),
        "pair": (_custom(92, [6, 8, 3, 1], [4, 3, 2, 5], [[1, 0], [2], [0], [3]], [2, 1, 3, 1], N=11, T=5, K=4),
                 f"pair_{algo}_f64"),
    }[case]
    rng = np.random.default_rng(91)
    q_prev = np.concatenate([rng.dirichlet(np.full(int(nf), 1.5), size=w.N) for nf in w.n], axis=1).astype(np.float32)
    act_prev = np.stack([rng.integers(0, int(u), size=w.N) for u in w.U], axis=1).astype(np.int32)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    q = md.run_from(algo, obs, act, torch.from_numpy(q_prev).cuda(), torch.from_numpy(act_prev).cuda(), w.K)
    q = q.cpu().numpy()
    if kern:
        assert md.last_kernel == kern, md.last_kernel
    assert md.status() == 0
    sel = list(range(0, w.N, max(1, w.N // 16)))
    sub = w.take_agents(sel)
    ref = oracle.run_workload(sub, algo, q_prev=q_prev[sel].astype(np.float64), act_prev=act_prev[sel])[0]
    assert np.abs(q[sel] - ref).max() <= 1e-5, np.abs(q[sel] - ref).max()
    # the prior matters: the plain call (prior D) differs
    assert np.abs(md.run(algo, obs, act, w.K).cpu().numpy() - q).max() > 1e-4
    # ... and both a continued prior and a warm start at once
    q_init = _random_beliefs(w, 78)
    q2 = md.run_from(algo, obs, act, torch.from_numpy(q_prev).cuda(), torch.from_numpy(act_prev).cuda(), w.K,
                     q_init=torch.from_numpy(q_init).cuda()).cpu().numpy()
    ref2 = oracle.run_workload(sub, algo, q_init=q_init[sel].astype(np.float64), q_prev=q_prev[sel].astype(np.float64),
                               act_prev=act_prev[sel])[0]
    assert np.abs(q2[sel] - ref2).max() <= 1e-5
    md.close()


# ---- damped updates (bi_model_set_damping)

@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("case", ["tile", "tile_cluster", "batch", "warp", "cta", "per_agent", "pair", "pair_and_others"])
def test_damped_updates(case, algo):
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = {
        "tile": make_config(2, N=9, T=11, K=6),
        "tile_cluster": make_config(4, N=4, T=20, K=6),
        "batch": make_config(3, N=128, T=16, K=6),
        "warp": _custom(49, [5, 4, 3, 2], [3, 4], [[0, 1], [1, 2, 3]], [2, 2, 1, 2], N=10, T=7, K=6),
        "cta": make_config(3, N=10, T=7, K=6),
        "per_agent": _custom(8, [6, 5, 7], [4, 3], [[2, 0, 1], [1, 2]], [2, 2, 2], N=5, T=6, K=6, G=5),
        "pair": make_config(1, N=11, T=9, K=6),
        # two coupled factors, one with a modality of its own, and two factors outside the pair (one observed)
        "pair_and_others": _custom(54, [5, 3, 7, 4], [3, 4, 2, 3], [[2, 0], [0], [1], [0, 2]], [2, 1, 3, 2],
                                   N=37, T=8, K=5),
    }[case]
    lam = 0.45
    with (warp_filter_forced() if case == "warp" else contextlib.nullcontext()):
        md = bi.model_from_workload(w)     # (the testing aid is read when the handle is made)
    md.set_damping(lam)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    lq = torch.empty((w.N, w.T, w.S), dtype=torch.float32, device="cuda")
    q = md.run(algo, obs, act, w.K, logq_out=lq).cpu().numpy()
    kernel = md.last_kernel
    if algo == "filter" and case in ("warp", "cta"):
        assert kernel == f"{case}_filter_f64", kernel
    if case in ("pair", "pair_and_others"):
        assert kernel == f"pair_{algo}_f64", kernel
    assert md.status() == 0
    sel = list(range(0, w.N, max(1, w.N // 12)))
    sub = w.take_agents(sel)
    ref, lref, _ = oracle.run_workload(sub, algo, damping=lam)
    print(case, algo, kernel, np.abs(q[sel] - ref).max())
    assert np.abs(q[sel] - ref).max() <= 1e-5
    big = lref > -30
    assert np.abs(lq.cpu().numpy()[sel][big] - lref[big]).max() <= 1e-4
    if algo != "filter":   # damped and warm-started: the first step mixes with ln q_init
        q_init = _random_beliefs(w, 79)
        fn = md.bi_vmp_warm if algo == "vmp" else md.bi_mmp_warm
        q2 = fn(obs, act, torch.from_numpy(q_init).cuda(), w.K).cpu().numpy()
        ref2 = oracle.run_workload(sub, algo, q_init=q_init[sel].astype(np.float64), damping=lam)[0]
        assert np.abs(q2[sel] - ref2).max() <= 1e-5
    # back to the plain update
    md.set_damping(1.0)
    q1 = md.run(algo, obs, act, w.K).cpu().numpy()
    ref1 = oracle.run_workload(sub, algo)[0]
    assert np.abs(q1[sel] - ref1).max() <= 1e-5
    with pytest.raises(bi.BiError):
        md.set_damping(0.0)
    md.close()


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_batched_window_with_per_agent_models(algo):
    # per-agent models without a register tile: every unit contracts its own slice
    w = _custom(52, [5, 7, 3, 4], [4, 3, 5], [[0, 1, 3], [1, 2], [2]], [2, 1, 3, 2], N=140, T=16, K=5, G=140,
                sparsity=0.5)
    res = check_workload(w, algo, agents=range(0, 140, 7))
    assert res["kernel"] == f"batch_{algo}_f64", res
    # the same through observation vectors on a shared model (slices become per agent and step)
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = make_config(3, N=130, T=16, K=4)            # 130 x 16 x 5460 x 8 B = 91 MB of slices: L2-resident
    md = bi.model_from_workload(w)
    soft = _soft_vectors(w, 6)
    q = md.run_soft(algo, torch.from_numpy(soft).cuda(), torch.from_numpy(w.act).cuda(), w.K).cpu().numpy()
    assert md.last_kernel == f"batch_{algo}_f64", md.last_kernel
    sel = list(range(0, 130, 13))
    sub = w.take_agents(sel)
    ref = oracle.run(algo, sub.n, sub.m, sub.dep, sub.U, sub.G, sub.A, sub.B, sub.D, None, sub.act, sub.K,
                     obs_soft=soft[sel])[0]
    assert np.abs(q[sel] - ref).max() <= 1e-5
    md.close()


@pytest.mark.parametrize("j", [0, 3, 7, 19, 42, 68, 77, 101, 127])
def test_warp_filter_kernel_on_small_batches(j):
    """The warp-per-agent filtering kernel serves large batches; here it is forced onto oracle-sized ones."""
    w = make_sweep_config(j, N=12)
    with warp_filter_forced():
        res = check_workload(w, "filter")
    assert res["kernel"] == "warp_filter_f64", res


@pytest.mark.parametrize("arith", ["f64", "f32"])
def test_filter_kernels_across_batch_sizes(arith):
    """The CTA-per-agent kernel at the batch sizes that select its 8-, 4- and 2-warp CTAs, and the
    warp-per-agent kernel on the largest batch, all against the oracle on sampled agents."""
    import oracle
    import paper_2607_17855_b200 as bi
    w = _custom(53, [5, 4, 3, 6], [3, 4, 5], [[0, 1], [1, 2, 3], [3]], [2, 2, 1, 3], N=1400, T=5, K=6)
    md = bi.model_from_workload(w, arith=arith)
    sel = list(range(0, w.N, 100))
    ref = oracle.run_workload(w.take_agents(sel), "filter")[0]
    for n, kern in ((40, "cta_filter"), (400, "cta_filter"), (1400, "cta_filter"), (1400, "warp_filter")):
        sub = w.take_agents(list(range(n)))
        if kern == "warp_filter":   # (the testing aid is read when a handle is made: a handle of its own)
            with warp_filter_forced():
                mdw = bi.model_from_workload(w, arith=arith)
            q, _, _, _ = run_gpu(sub, "filter", model=mdw, arith=arith)
            name = mdw.last_kernel
            mdw.close()
        else:
            q, _, _, _ = run_gpu(sub, "filter", model=md, arith=arith)
            name = md.last_kernel
        assert name == f"{kern}_{arith}", (n, name)
        pick = [i for i in sel if i < n]
        err = np.abs(q[pick] - ref[:len(pick)]).max()
        assert err <= (1e-5 if arith == "f64" else 5e-3), (n, err)
    md.close()


@pytest.mark.parametrize("case", ["rank1_only", "rank5", "per_agent", "many_groups", "wide_last_axis", "max_counts"])
def test_cta_filter_kernel_shapes(case):
    """Shapes that stress the CTA-per-agent kernel's phases: no contraction at all, four levels, per-agent slices,
    several groups sharing a last axis (one merged reduction) next to groups that do not, a 32-state last axis."""
    w = {
        "rank1_only": _custom(61, [7, 3], [4, 5, 2], [[0], [1], [0]], [2, 1], N=6, T=5, K=5),
        "rank5": _custom(62, [3, 4, 2, 5, 3], [4, 3], [[0, 1, 2, 3, 4], [2, 4]], [2, 1, 2, 1, 3], N=5, T=4, K=5),
        "per_agent": _custom(63, [6, 5, 7, 2], [4, 3, 2], [[2, 0, 1], [1, 2], [3]], [2, 2, 2, 1], N=7, T=5, K=5, G=7,
                             sparsity=0.5),
        "many_groups": _custom(64, [9, 4, 6, 5], [3, 4, 2, 5, 3, 2], [[0, 1], [2, 0], [3, 0], [1, 2], [0, 1, 2, 3], [3]],
                               [2, 1, 3, 2], N=9, T=5, K=6),
        "wide_last_axis": _custom(65, [32, 31, 2], [3, 4], [[0, 1], [1, 2, 0]], [2, 2, 1], N=4, T=4, K=5),
        # the most factors and modalities a model may have, sixteen distinct dependency sets
        "max_counts": _custom(66, [3, 2, 4, 3, 2, 5, 2, 3], [2, 3, 2, 4, 3, 2, 3, 2, 4, 2, 3, 2, 3, 2, 2, 3],
                              [[0], [1, 2], [2, 3, 4], [5], [6, 7], [0, 1, 2, 3, 4], [7, 0], [3, 5], [4], [1, 6], [2, 7, 5],
                               [0, 3], [6], [5, 1], [4, 7], [2, 0, 6]], [2, 1, 2, 1, 3, 1, 2, 2], N=5, T=4, K=5),
    }[case]
    res = check_workload(w, "filter")
    assert res["kernel"] == ("pair_filter_f64" if case == "rank1_only" else "cta_filter_f64"), res
    with family_forced("cta"):
        res = check_workload(w, "filter")
    assert res["kernel"] == "cta_filter_f64", res


@pytest.mark.parametrize("j", list(range(2, 128, 5)))
def test_filter_kernels_on_random_structures_with_ragged_sizes(j):
    """Every fifth structure of the sweep with ragged agent, step and iteration counts, through both general
    filtering kernels (the CTA-per-agent one by dispatch, the warp-per-agent one forced)."""
    rng = np.random.default_rng(1000 + j)
    w = make_sweep_config(j, N=int(rng.integers(1, 14)), T=int(rng.integers(1, 9)), K=int(rng.integers(1, 7)))
    res = check_workload(w, "filter", conditioned=True)
    assert res["kernel"] in ("cta_filter_f64", "pair_filter_f64"), res
    with family_forced("cta"):
        res = check_workload(w, "filter", conditioned=True)
    assert res["kernel"] == "cta_filter_f64", res
    with warp_filter_forced():
        res = check_workload(w, "filter", conditioned=True)
    assert res["kernel"] == "warp_filter_f64", res


def test_golden_mmp_backward_message_on_the_gpu(golden_dir):
    """The hand-worked two-step window whose backward message varies over states (unequal row sums of
    the transition matrix), one iteration from the fixture's start, through bi_mmp_warm / bi_vmp_warm."""
    import torch
    import paper_2607_17855_b200 as bi
    from conftest import read_golden
    g = read_golden(os.path.join(golden_dir, "mmp_future_message.txt"))
    A = [torch.tensor(g["A"].reshape(1, 2, 2), dtype=torch.float32, device="cuda")]
    B = [torch.tensor(g["B"].reshape(1, 2, 2, 1), dtype=torch.float32, device="cuda")]
    D = [torch.tensor(g["D"].reshape(1, 2), dtype=torch.float32, device="cuda")]
    md = bi.Model([2], [2], [[0]], [1], 1, A, B, D)
    obs = torch.tensor(g["obs"].reshape(1, 2, 1), dtype=torch.int32, device="cuda")
    act = torch.zeros((1, 1, 1), dtype=torch.int32, device="cuda")
    start = torch.tensor(np.stack([g["q1_start"], g["q2_start"]])[None], dtype=torch.float32, device="cuda")
    for algo, fn in (("mmp", md.bi_mmp_warm), ("vmp", md.bi_vmp_warm)):
        q = fn(obs, act, start, 1).cpu().numpy()
        np.testing.assert_allclose(q[0, 0], g["q1_" + algo], atol=3e-7)
        np.testing.assert_allclose(q[0, 1], g["q2_" + algo], atol=3e-7)
    # a permutation transition: the backward message carries the later belief back through it
    perm = [2, 0, 3, 1]
    Bu = np.zeros((4, 4), np.float32)
    for s_, r_ in enumerate(perm):
        Bu[r_, s_] = 1.0
    md2 = bi.Model([4], [2], [[0]], [1], 1, [torch.full((1, 2, 4), 0.5, device="cuda")],
                   [torch.tensor(Bu.reshape(1, 4, 4, 1), device="cuda")], [torch.full((1, 4), 0.25, device="cuda")])
    q2 = np.array([0.1, 0.2, 0.3, 0.4])
    start = torch.tensor(np.stack([np.full(4, 0.25), q2])[None], dtype=torch.float32, device="cuda")
    q = md2.bi_mmp_warm(torch.zeros((1, 2, 1), dtype=torch.int32, device="cuda"), act, start, 1).cpu().numpy()
    want = np.sqrt(q2[perm])
    np.testing.assert_allclose(q[0, 0], want / want.sum(), atol=3e-7)
    md.close()
    md2.close()


def _blockwise(md, w, cuts, K):
    """bi_filter on the first block of steps, bi_filter_continue on the rest; returns q [N, T, S]."""
    import torch
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    parts, names = [], set()
    for i, (t0, t1) in enumerate(zip(cuts[:-1], cuts[1:])):
        o = obs[:, t0:t1].contiguous()
        a = act[:, t0:t1 - 1].contiguous() if t1 - t0 > 1 else None
        if i == 0:
            parts.append(md.bi_filter(o, a, K))
        else:
            parts.append(md.bi_filter_continue(o, a, act[:, t0 - 1].contiguous(), K))
        names.add(md.last_kernel)
    torch.cuda.synchronize()
    return torch.cat(parts, dim=1).cpu().numpy(), names


@pytest.mark.parametrize("case", ["tile_f64", "tile_sb2", "cta", "warp", "tile_f32"])
def test_filter_continue_equals_the_single_call_bit_for_bit(case):
    """A trajectory filtered in consecutive blocks through the handle's full-precision record equals
    the single call exactly, on every filtering kernel family."""
    import torch
    import paper_2607_17855_b200 as bi
    arith = "f32" if case == "tile_f32" else "f64"
    if case in ("tile_f64", "tile_f32"):
        w = make_config(2, N=37, T=12)
    elif case == "tile_sb2":
        w = make_config(4, N=9, T=9)
    else:
        w = make_sweep_config(42, N=13, T=11)
    ctx = warp_filter_forced() if case == "warp" else contextlib.nullcontext()
    with ctx:
        md = bi.model_from_workload(w, arith=arith)
        obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
        whole = md.bi_filter(obs, act, w.K).cpu().numpy()
        kernel = md.last_kernel
        for cuts in ([0, 1, w.T], [0, 4, 5, w.T - 2, w.T], [0, w.T - 1, w.T]):
            q, names = _blockwise(md, w, cuts, w.K)
            assert names == {kernel}
            assert np.array_equal(q, whole), (case, cuts, np.abs(q - whole).max())
    expect = {"tile_f64": "tile3_filter_f64", "tile_f32": "tile3_filter_f32", "tile_sb2": "tile3_filter_f64",
              "cta": "cta_filter_f64", "warp": "warp_filter_f64"}[case]
    assert kernel == expect
    assert md.status() == 0
    md.close()


def test_filter_continue_needs_a_matching_previous_call():
    import torch
    import paper_2607_17855_b200 as bi
    w = make_config(1)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    ap = act[:, 0].contiguous()
    with pytest.raises(bi.BiError) as e:
        md.bi_filter_continue(obs[:, 1:].contiguous(), act[:, 1:].contiguous(), ap, 2)   # nothing to continue
    assert e.value.code == -1
    md.bi_filter(obs[:, :1].contiguous(), None, 2)
    with pytest.raises(bi.BiError) as e:
        md.bi_filter_continue(obs[:4, 1:].contiguous(), act[:4, 1:].contiguous(), ap[:4].contiguous(), 2)   # other N
    assert e.value.code == -1
    md.bi_filter_continue(obs[:, 1:].contiguous(), act[:, 1:].contiguous(), ap, 2)
    # a window call in between leaves the record alone
    md.bi_vmp(obs, act, 2)
    md.bi_filter_continue(obs[:, 1:].contiguous(), act[:, 1:].contiguous(), ap, 2)
    assert md.status() == 0
    md.close()


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("case", ["config1", "sweep", "per_agent"])
def test_general_cta_kernel_when_forced(case, algo):
    """The first, fully general kernel family (one CTA per agent, every shape and algorithm): the
    fallback behind the others, forced here so that it is checked against the oracle too."""
    w = {"config1": lambda: make_config(1), "sweep": lambda: make_sweep_config(19, N=6, T=6),
         "per_agent": lambda: make_config(4, N=5, T=5)}[case]()
    with family_forced("generic"):
        res = check_workload(w, algo)
    print(res)
    assert res["kernel"].startswith("generic_"), res["kernel"]


def test_a_copy_that_never_arrives_is_reported_not_waited_for():
    """The bounded wait on a block's own bulk copy.  The testing aid BI_TEST_DROP_COPY=1 (read when the
    handle is made) makes the next batched window call announce its slice copies on their barriers
    without issuing them; every contraction block must give up after its probe limit, raise
    BI_FLAG_COPY_TIMEOUT and leave -- nothing is in flight, nothing faults, the context stays usable --
    and the next call on the same handle is an ordinary, correct one."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = make_config(3, N=128, T=16, K=4)
    old = os.environ.get("BI_TEST_DROP_COPY")
    os.environ["BI_TEST_DROP_COPY"] = "1"
    try:
        md = bi.model_from_workload(w)
    finally:
        if old is None:
            del os.environ["BI_TEST_DROP_COPY"]
        else:
            os.environ["BI_TEST_DROP_COPY"] = old
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    md.bi_vmp(obs, act, w.K)
    assert md.last_kernel == "batch_vmp_f64"
    flags = md.status()                 # synchronises; returns and clears the flags
    assert flags & 4, flags             # BI_FLAG_COPY_TIMEOUT
    q = md.bi_vmp(obs, act, w.K).cpu().numpy()
    assert md.status() == 0
    sel = list(range(0, w.N, 16))
    ref = oracle.run_workload(w.take_agents(sel), "vmp")[0]
    assert np.abs(q[sel] - ref).max() <= 1e-5
    md.close()


# ---- non-trivial B-dependencies (bi_model_create_bdep) ----

def _bdep_workload(seed, n, m, dep, U, bdep, N, T, K, G=1, sparsity=0.0, b_sparsity=0.0):
    rng = np.random.default_rng(seed)
    A, B, D = make_model(rng, n, m, dep, U, G, sparsity=sparsity, d_alpha=1.0, bdep=bdep, b_sparsity=b_sparsity)
    obs, act = sample_streams(rng, n, m, dep, U, G, A, B, D, N, T, bdep=bdep)
    return Workload(name="bdep", algo="filter", n=np.asarray(n, np.int32), m=np.asarray(m, np.int32), dep=dep,
                    U=np.asarray(U, np.int32), G=G, A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act, bdep=bdep)


BDEP_CASES = {
    "two_parents": dict(n=[4, 3], m=[5, 4], dep=[[0, 1], [1]], U=[2, 2], bdep=[[0, 1], [1]], N=9, T=6, K=6),
    "cross": dict(n=[3, 5, 2], m=[4, 3], dep=[[0, 1], [2, 1]], U=[2, 1, 3], bdep=[[1], [0, 2], [2, 1, 0]], N=7, T=5, K=5,
                  sparsity=0.5, b_sparsity=0.5),
    "wide": dict(n=[6, 5, 4, 3], m=[3, 4, 2], dep=[[0, 1, 2], [3], [1, 3]], U=[1, 2, 2, 1],
                 bdep=[[0, 1, 2, 3], [1], [3, 2], [0, 3]], N=5, T=4, K=4),
    "per_agent": dict(n=[3, 4], m=[3, 2], dep=[[0, 1], [1]], U=[2, 2], bdep=[[1, 0], [0]], N=4, T=5, K=4, G=4, sparsity=0.6),
    "ragged_edge": dict(n=[32, 2], m=[2], dep=[[0]], U=[1, 1], bdep=[[0, 1], [1, 0]], N=1, T=1, K=1),
    # five parents: the window kernel's table of parent offsets holds four, so its lanes walk the combinations themselves
    "five_parents": dict(n=[2, 3, 2, 2, 3], m=[3, 2], dep=[[0, 1], [4, 2, 3]], U=[2, 1, 1, 2, 1],
                         bdep=[[4, 3, 2, 1, 0], [1], [2, 0], [3], [4, 1]], N=6, T=5, K=4),
    # windows long enough that every warp takes several steps, parents' products of 96 and 120 entries
    "long_window": dict(n=[8, 12, 10], m=[4, 3], dep=[[0, 1], [2]], U=[2, 2, 1], bdep=[[0, 1], [1, 2], [2, 0]],
                        N=3, T=23, K=3),
}


@pytest.mark.parametrize("algo", ["filter", "vmp"])
@pytest.mark.parametrize("case", sorted(BDEP_CASES))
def test_b_dependencies(case, algo):
    """Transitions that read other factors' previous states, against the oracle's enumerated reading."""
    w = _bdep_workload(1200 + sorted(BDEP_CASES).index(case), **BDEP_CASES[case])
    res = check_workload(w, algo)
    print(case, algo, res)
    # (in filtering the transition tensors enter only the prior: the CTA-per-agent filtering kernel forms it)
    if algo == "vmp":   # the warp-per-step kernel's lanes sum the transition tensors' messages
        assert res["kernel"] == "warp_vmp_f64", res
        with family_forced("generic"):
            res = check_workload(w, algo)
        assert res["kernel"].startswith("generic_"), res
    else:
        assert res["kernel"] == "cta_filter_f64", res
        with family_forced("generic"):
            res = check_workload(w, algo)
        assert res["kernel"].startswith("generic_"), res


@pytest.mark.parametrize("algo", ["filter", "vmp"])
def test_b_dependencies_damped(algo):
    """The damped update on a model with several parents per transition, on the kernels the dispatcher
    picks and on the general kernel."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = _bdep_workload(1400, [4, 3, 5], [5, 4], [[0, 1], [1, 2]], [2, 2, 1], [[0, 1], [1, 2], [2, 0]], N=8, T=6, K=7)
    ref = oracle.run_workload(w, algo, damping=0.6)[0]
    for forced in (None, "generic"):
        with (family_forced(forced) if forced else contextlib.nullcontext()):
            md = bi.model_from_workload(w)
        md.set_damping(0.6)
        q = md.run(algo, torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda(), w.K).cpu().numpy()
        assert md.status() == 0
        if forced:
            assert md.last_kernel.startswith("generic_"), md.last_kernel
        else:
            assert md.last_kernel == ("cta_filter_f64" if algo == "filter" else "warp_vmp_f64"), md.last_kernel
        assert np.abs(q - ref).max() <= 1e-5, (forced, md.last_kernel, np.abs(q - ref).max())
        md.close()


def test_b_dependencies_call_forms_and_refusals():
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = _bdep_workload(1300, [4, 3], [5, 4], [[0, 1], [1]], [2, 2], [[0, 1], [1, 0]], N=6, T=6, K=5)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    # blocks of steps through the handle's record equal the single call; a float32 q_prev is within tolerance
    whole = md.bi_filter(obs, act, w.K).cpu().numpy()
    head = md.bi_filter(obs[:, :2].contiguous(), act[:, :1].contiguous(), w.K)
    tail = md.bi_filter_continue(obs[:, 2:].contiguous(), act[:, 2:].contiguous(), act[:, 1].contiguous(), w.K)
    assert np.array_equal(torch.cat([head, tail], dim=1).cpu().numpy(), whole)
    tail32 = md.bi_filter_from(obs[:, 2:].contiguous(), act[:, 2:].contiguous(), head[:, -1].contiguous(),
                               act[:, 1].contiguous(), w.K).cpu().numpy()
    ref = oracle.run_workload(w, "filter")[0]
    assert np.abs(whole - ref).max() <= 1e-5 and np.abs(tail32 - ref[:, 2:]).max() <= 1e-5
    # a warm start
    rng = np.random.default_rng(5)
    q_init = np.concatenate([rng.dirichlet(np.full(int(k), 2.0), size=(w.N, w.T)) for k in w.n], axis=2).astype(np.float32)
    q = md.bi_vmp_warm(obs, act, torch.from_numpy(q_init).cuda(), 3).cpu().numpy()
    ref = oracle.run("vmp", w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, w.obs, w.act, 3,
                     q_init=q_init.astype(np.float64), bdep=w.bdep)[0]
    assert np.abs(q - ref).max() <= 1e-5
    # what has no counterpart with several parents is refused
    for call in (lambda: md.bi_mmp(obs, act, 2),
                 lambda: md.bi_mmp_warm(obs, act, torch.from_numpy(q_init).cuda(), 2),
                 lambda: md.run_from("vmp", obs, act, head[:, -1].contiguous(), act[:, 1].contiguous(), 2),
                 lambda: md.run_soft("filter", torch.zeros((w.N, w.T, int(w.m.sum())), device="cuda"), act, 2)):
        with pytest.raises(bi.BiError) as e:
            call()
        assert e.value.code == -3
    assert md.status() == 0
    md.close()
    # malformed lists
    A = [torch.from_numpy(a).cuda() for a in w.A]
    B = [torch.from_numpy(b).cuda() for b in w.B]
    D = [torch.from_numpy(d).cuda() for d in w.D]
    for bad, code in (([[0, 0], [1]], -2), ([[0, 2], [1]], -1), ([[], [1]], -1)):
        with pytest.raises(bi.BiError) as e:
            bi.Model(w.n, w.m, w.dep, w.U, 1, A, B, D, bdep=bad)
        assert e.value.code == code, (bad, e.value.code)


# ---- compressed slices for sparse per-agent models ----

@pytest.mark.parametrize("algo", ["vmp", "mmp"])
def test_compressed_slices_give_the_dense_result_bit_for_bit(algo):
    """Per-agent models with 70 % zeros keep their slices as a mask per lane plus the non-floor values;
    the window kernels gather from that form.  Same values, same order of additions: the beliefs equal
    those of a handle made without compression (testing aid BI_TEST_NO_COMPRESS) exactly, and the oracle's
    within tolerance.  A dense per-agent model is left uncompressed."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = make_config(4, N=24, T=7)
    md = bi.model_from_workload(w)
    dense_b, comp_b = md.slice_bytes()
    assert 0 < comp_b < 0.6 * dense_b, (dense_b, comp_b)
    md.set_compressed(True)
    old = os.environ.get("BI_TEST_NO_COMPRESS")
    os.environ["BI_TEST_NO_COMPRESS"] = "1"
    try:
        md_dense = bi.model_from_workload(w)
    finally:
        if old is None:
            del os.environ["BI_TEST_NO_COMPRESS"]
        else:
            os.environ["BI_TEST_NO_COMPRESS"] = old
    assert md_dense.slice_bytes() == (0, 0)
    with pytest.raises(bi.BiError) as e:
        md_dense.set_compressed(True)
    assert e.value.code == -3
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    outs = []
    for m_ in (md, md_dense):
        lq = torch.empty((w.N, w.T, w.S), device="cuda")
        am = torch.empty((w.N, w.T, w.F), dtype=torch.int32, device="cuda")
        q = m_.run(algo, obs, act, w.K, logq_out=lq, argmax_out=am)
        assert m_.last_kernel == f"tile3_{algo}_f64" and m_.status() == 0
        outs.append((q.cpu().numpy(), lq.cpu().numpy(), am.cpu().numpy()))
    for x, y in zip(*outs):
        assert np.array_equal(x, y)
    from parity import compare_conditioned
    print(compare_conditioned(w, algo, *outs[0], oracle.run_workload(w, algo)))
    # filtering on the same handle reads the dense form
    qf = md.bi_filter(obs, act, w.K).cpu().numpy()
    assert np.array_equal(qf, md_dense.bi_filter(obs, act, w.K).cpu().numpy())
    md.close()
    md_dense.close()
    # a dense per-agent model of the same shape: nothing to gain, nothing made
    rng = np.random.default_rng(9)
    A, B, D = make_model(rng, w.n, w.m, w.dep, w.U, 6, sparsity=0.0, d_alpha=1.0)
    md2 = bi.Model(w.n, w.m, w.dep, w.U, 6, [torch.from_numpy(a).cuda() for a in A],
                   [torch.from_numpy(b).cuda() for b in B], [torch.from_numpy(d).cuda() for d in D])
    assert md2.slice_bytes() == (0, 0)
    md2.close()


# ---- the pair filtering kernel (models coupled in at most one pair of factors) ----

PAIR_CASES = {
    "config1": lambda: make_config(1),
    "lanes4_many_agents": lambda: _custom(91, [4, 3], [5, 4, 3], [[0, 1], [1, 0], [1]], [2, 2], N=37, T=6, K=7),
    "lanes8_extra_factors": lambda: _custom(92, [6, 8, 3, 1], [4, 3, 2, 5], [[1, 0], [2], [0], [3]], [2, 1, 3, 1], N=11, T=5, K=6),
    "lanes16_sparse": lambda: _custom(93, [9, 13], [6, 3], [[0, 1], [0, 1]], [3, 2], N=5, T=7, K=8, sparsity=0.7),
    "lanes32": lambda: _custom(94, [32, 31], [3, 4, 2], [[1, 0], [0], [1]], [2, 2], N=3, T=4, K=5),
    "no_pair": lambda: _custom(95, [7, 5, 12], [4, 3, 5, 2], [[0], [2], [2], [0]], [2, 3, 1], N=9, T=6, K=4),
    "per_agent": lambda: _custom(96, [5, 7], [4, 3], [[0, 1], [1]], [2, 2], N=6, T=5, K=6, G=6, sparsity=0.5),
    "one_agent_one_step": lambda: _custom(97, [5, 3], [4], [[0, 1]], [1, 1], N=1, T=1, K=1),
}


@pytest.mark.parametrize("case", sorted(PAIR_CASES))
def test_pair_filter_kernel(case):
    w = PAIR_CASES[case]()
    res = check_workload(w, "filter", conditioned=True)
    print(case, res)
    assert res["kernel"] == "pair_filter_f64", res


@pytest.mark.parametrize("j", [8, 15, 19, 0, 13, 90, 127])
def test_pair_filter_kernel_on_sweep_structures(j):
    w = make_sweep_config(j, N=21, T=7)
    res = check_workload(w, "filter", conditioned=True)
    assert res["kernel"] == "pair_filter_f64", res


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
@pytest.mark.parametrize("case", sorted(PAIR_CASES))
def test_pair_window_kernel(case, algo):
    w = PAIR_CASES[case]()
    res = check_workload(w, algo, conditioned=True)
    print(case, algo, res)
    assert res["kernel"] == f"pair_{algo}_f64", res


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
@pytest.mark.parametrize("j", [8, 15, 19, 0, 13, 90, 127])
def test_pair_window_kernel_on_sweep_structures(j, algo):
    w = make_sweep_config(j, N=21, T=7)
    res = check_workload(w, algo, conditioned=True)
    assert res["kernel"] == f"pair_{algo}_f64", res


RANK2_CASES = {
    "chain": lambda: _custom(191, [6, 9, 5, 3], [4, 3, 5, 2], [[0, 1], [1, 2], [3], [2, 1]], [2, 1, 3, 2], N=9, T=6, K=6),
    "triangle": lambda: _custom(192, [12, 16, 7], [3, 4, 2, 3], [[0, 1], [2, 0], [1, 2], [1]], [2, 2, 2], N=5, T=5, K=5,
                                sparsity=0.5),
    "two_pairs_32_lanes": lambda: _custom(193, [31, 32, 20, 6], [3, 2, 4], [[0, 1], [3, 2], [1, 0]], [1, 2, 2, 3],
                                          N=3, T=4, K=4),
    "per_agent": lambda: _custom(194, [5, 7, 4], [4, 3, 3], [[0, 1], [1, 2], [2]], [2, 2, 1], N=6, T=5, K=6, G=6, sparsity=0.5),
}


@pytest.mark.parametrize("algo", ["vmp", "mmp"])
@pytest.mark.parametrize("case", sorted(RANK2_CASES))
def test_pair_window_kernel_with_several_pairs(case, algo):
    """Models whose groups all span at most two factors, several of them: the window kernel takes every
    group's matrix-vector products from the staged slices."""
    w = RANK2_CASES[case]()
    res = check_workload(w, algo, conditioned=True)
    print(case, algo, res)
    assert res["kernel"] == f"pair_{algo}_f64", res


@pytest.mark.parametrize("j", [1, 2, 4, 17, 30, 62, 78])
def test_pair_window_kernel_on_sweep_structures_with_several_pairs(j):
    w = make_sweep_config(j, N=11, T=6)
    for algo in ("vmp", "mmp"):
        res = check_workload(w, algo, conditioned=True)
        assert res["kernel"] == f"pair_{algo}_f64", res


@pytest.mark.parametrize("case", sorted(RANK2_CASES))
def test_filtering_on_models_with_several_pairs(case):
    """(the same models through bi_filter: the CTA-per-agent filtering kernel's rank-2 path)"""
    w = RANK2_CASES[case]()
    res = check_workload(w, "filter", conditioned=True)
    print(case, res)
    assert res["kernel"] == "cta_filter_f64", res


def test_pair_window_kernel_limits():
    """A window whose steps do not fit one CTA goes to another kernel family; a damped call does not."""
    import torch
    import paper_2607_17855_b200 as bi
    w = _custom(99, [32, 31], [3, 4], [[1, 0], [0]], [2, 2], N=40, T=20, K=3)   # 20 steps x 32 lanes > 512 threads
    res = check_workload(w, "vmp", agents=range(0, 40, 5))
    assert not res["kernel"].startswith("pair_"), res
    w = _custom(98, [6, 8, 3], [4, 3, 2], [[1, 0], [2], [0]], [2, 1, 3], N=11, T=9, K=6)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    md.bi_vmp(obs, act, w.K)
    assert md.last_kernel == "pair_vmp_f64"
    import oracle
    md.set_damping(0.5)
    for algo in ("vmp", "mmp"):
        q = md.run(algo, obs, act, w.K).cpu().numpy()
        assert md.last_kernel == f"pair_{algo}_f64" and md.status() == 0
        assert np.abs(q - oracle.run_workload(w, algo, damping=0.5)[0]).max() <= 1e-5
    md.close()


def test_pair_filter_continued_calls():
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    w = _custom(98, [6, 8, 3], [4, 3, 2], [[1, 0], [2], [0]], [2, 1, 3], N=11, T=9, K=6)
    md = bi.model_from_workload(w)
    obs, act = torch.from_numpy(w.obs).cuda(), torch.from_numpy(w.act).cuda()
    whole = md.bi_filter(obs, act, w.K).cpu().numpy()
    assert md.last_kernel == "pair_filter_f64"
    q, names = _blockwise(md, w, [0, 2, 3, 7, w.T], w.K)
    assert names == {"pair_filter_f64"} and np.array_equal(q, whole)
    head = md.bi_filter(obs[:, :4].contiguous(), act[:, :3].contiguous(), w.K)
    tail = md.bi_filter_from(obs[:, 4:].contiguous(), act[:, 4:].contiguous(), head[:, -1].contiguous(),
                             act[:, 3].contiguous(), w.K).cpu().numpy()
    ref = oracle.run_workload(w, "filter")[0]
    assert np.abs(whole - ref).max() <= 1e-5 and np.abs(tail - ref[:, 4:]).max() <= 1e-5
    # a damped call is this kernel's too, block by block as well
    md.set_damping(0.5)
    damped = md.bi_filter(obs, act, w.K).cpu().numpy()
    assert md.last_kernel == "pair_filter_f64" and md.status() == 0
    q, names = _blockwise(md, w, [0, 2, 3, 7, w.T], w.K)
    assert names == {"pair_filter_f64"} and np.array_equal(q, damped)
    assert np.abs(damped - oracle.run_workload(w, "filter", damping=0.5)[0]).max() <= 1e-5
    md.close()
