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
