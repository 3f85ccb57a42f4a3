"""Random models against the oracle: structures, sizes and batch shapes drawn from a seeded generator,
every call compared element by element (the rules of ``parity.check_workload``).  The named
configurations and the sweep's 128 structures exercise the kernels on the workloads that are timed;
these cases reach the corners between them (one state, one agent, one step, one iteration, ranks 1 to
4 mixed, per-agent models, sparse arrays) on whichever kernel family the dispatcher picks."""
import numpy as np
import pytest

from biwl import Workload, make_model, sample_streams
from parity import check_workload

pytestmark = pytest.mark.gpu


def _draw(seed, large):
    rng = np.random.default_rng(770000 + seed)
    F = int(rng.integers(1, 6))
    wide = rng.random() < 0.3
    n = [int(rng.integers(1, 33 if wide else 13)) for _ in range(F)]
    M = int(rng.integers(1, 6))
    dep, m = [], []
    for _ in range(M):
        d = [int(x) for x in rng.choice(F, size=int(rng.integers(1, min(F, 4) + 1)), replace=False)]
        while np.prod([n[f] for f in d]) * 6 > 60000:
            d = d[:-1]
        dep.append(d)
        m.append(int(rng.integers(1, 7)))
    U = [int(rng.integers(1, 4)) for _ in range(F)]
    N = int(rng.choice([250, 400, 700])) if large else int(rng.choice([1, 3, 17, 40, 70, 300]))
    T = int(rng.choice([9, 12, 16])) if large else int(rng.choice([1, 2, 5, 9, 12]))
    K = int(rng.integers(1, 7))
    G = N if (not large and rng.random() < 0.2 and N <= 40) else 1
    sparsity = float(rng.choice([0.0, 0.0, 0.5, 0.9]))
    A, B, D = make_model(rng, n, m, dep, U, G, sparsity=sparsity, d_alpha=1.0)
    obs, act = sample_streams(rng, n, m, dep, U, G, A, B, D, N, T)
    return Workload(name=f"fuzz{seed}", algo="filter", n=np.asarray(n, np.int32), m=np.asarray(m, np.int32), dep=dep,
                    U=np.asarray(U, np.int32), G=G, A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act)


@pytest.mark.parametrize("block", range(6))
def test_random_models_small_batches(block):
    kernels = {}
    for seed in range(block * 10, block * 10 + 10):
        w = _draw(seed, large=False)
        for algo in ("filter", "vmp", "mmp"):
            res = check_workload(w, algo, agents=range(0, w.N, max(1, w.N // 12)), conditioned=True)
            kernels[res["kernel"]] = kernels.get(res["kernel"], 0) + 1
    print(kernels)


@pytest.mark.parametrize("block", range(3))
def test_random_models_batches_of_thousands_of_units(block):
    kernels = {}
    for seed in range(1000 + block * 8, 1000 + block * 8 + 8):
        w = _draw(seed, large=True)
        for algo in ("filter", "vmp", "mmp"):
            res = check_workload(w, algo, agents=range(0, w.N, max(1, w.N // 12)), conditioned=True)
            kernels[res["kernel"]] = kernels.get(res["kernel"], 0) + 1
    print(kernels)


@pytest.mark.parametrize("block", range(3))
def test_random_models_with_observation_vectors(block):
    """The calls that take categorical vectors: random structures (slices of any padded length, several
    modalities per dependency set, per-agent models), trajectories that end in every block length of the
    slice-forming kernels, float64 (tensor form) and float32 (scalar form) handles."""
    import torch
    import oracle
    import paper_2607_17855_b200 as bi
    kernels = {}
    for case in range(block * 12, block * 12 + 12):
        rng = np.random.default_rng(880000 + case)
        F = int(rng.integers(1, 5))
        n = [int(rng.integers(1, 11)) for _ in range(F)]
        M = int(rng.integers(1, 6))
        dep = [[int(x) for x in rng.choice(F, size=int(rng.integers(1, min(F, 3) + 1)), replace=False)] for _ in range(M)]
        m = [int(rng.integers(1, 8)) for _ in range(M)]
        U = [int(rng.integers(1, 3)) for _ in range(F)]
        N = int(rng.choice([1, 3, 9, 20]))
        algo = ("filter", "vmp", "mmp")[case % 3]
        T = int(rng.choice([1, 2, 7, 9, 17, 25, 33, 41, 66]))
        if algo != "filter":
            T = min(T, 64)   # (the window calls' documented limit)
        K = int(rng.integers(1, 4))
        G = N if rng.random() < 0.3 else 1
        arith = "f64" if case % 4 else "f32"
        A, B, D = make_model(rng, n, m, dep, U, G, sparsity=0.3, d_alpha=1.0)
        obs, act = sample_streams(rng, n, m, dep, U, G, A, B, D, N, T)
        w = Workload(name=f"softfuzz{case}", algo=algo, n=np.asarray(n, np.int32), m=np.asarray(m, np.int32), dep=dep,
                     U=np.asarray(U, np.int32), G=G, A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act)
        off = np.concatenate([[0], np.cumsum(w.m)]).astype(int)
        soft = np.zeros((N, T, int(off[-1])), np.float32)
        for i, mi in enumerate(w.m):
            soft[:, :, off[i]:off[i + 1]] = rng.dirichlet(np.full(int(mi), 0.7), size=(N, T))
        md = bi.model_from_workload(w, arith=arith)
        q = md.run_soft(algo, torch.from_numpy(soft).cuda(), torch.from_numpy(w.act).cuda(), K).cpu().numpy()
        assert md.status() == 0
        kernels[md.last_kernel] = kernels.get(md.last_kernel, 0) + 1
        ref = oracle.run(algo, w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, None, w.act, K, obs_soft=soft)[0]
        err = np.abs(q - ref).max()
        assert err <= (1e-5 if arith == "f64" else 5e-3), (case, algo, arith, md.last_kernel, err)
        md.close()
    print(kernels)


@pytest.mark.parametrize("block", range(2))
def test_random_models_with_several_parents_per_transition(block):
    """Transitions that read up to four factors' previous states, on random structures: filtering (the
    CTA kernel forms the parents' products once per factor and step) and VMP (the window kernel's table
    of parent offsets, its one-, two- and many-parent forms of the future message)."""
    kernels = {}
    for case in range(block * 12, block * 12 + 12):
        rng = np.random.default_rng(990000 + case)
        F = int(rng.integers(1, 5))
        n = [int(rng.integers(1, 9)) for _ in range(F)]
        M = int(rng.integers(1, 4))
        dep = [[int(x) for x in rng.choice(F, size=int(rng.integers(1, min(F, 3) + 1)), replace=False)] for _ in range(M)]
        m = [int(rng.integers(1, 5)) for _ in range(M)]
        U = [int(rng.integers(1, 3)) for _ in range(F)]
        bdep = [[int(x) for x in rng.choice(F, size=int(rng.integers(1, min(F, 4) + 1)), replace=False)] for _ in range(F)]
        N = int(rng.choice([1, 3, 8, 40]))
        T = int(rng.choice([1, 2, 5, 9, 17]))
        K = int(rng.integers(1, 5))
        sparsity, b_sparsity = float(rng.choice([0.0, 0.5])), float(rng.choice([0.0, 0.5]))
        A, B, D = make_model(rng, n, m, dep, U, 1, sparsity=sparsity, d_alpha=1.0, bdep=bdep, b_sparsity=b_sparsity)
        obs, act = sample_streams(rng, n, m, dep, U, 1, A, B, D, N, T, bdep=bdep)
        w = Workload(name=f"bdepfuzz{case}", algo="filter", n=np.asarray(n, np.int32), m=np.asarray(m, np.int32),
                     dep=dep, U=np.asarray(U, np.int32), G=1, A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act, bdep=bdep)
        for algo in ("filter", "vmp"):
            res = check_workload(w, algo, agents=range(0, N, max(1, N // 8)))
            kernels[res["kernel"]] = kernels.get(res["kernel"], 0) + 1
    print(kernels)
