"""Seeded generators for the five benchmark workloads.

Every workload is a pure function of its configuration number and seed.  The
recipe (Section V-A of the paper describes the kind of population; the concrete
sizes are the benchmark's own):

* all probability arrays are drawn in float64 (Dirichlet columns through
  normalised Gamma draws), optionally sparsified, cast once to float32;
* hidden-state trajectories, observations and actions are then sampled from
  that float32 model: ``s_1^f ~ D_f``, ``o_t^i ~ A_i[:, s_t^{dep(i)}]``,
  ``u_t^f ~ Uniform{0..U_f-1}``, ``s_{t+1}^f ~ B_f[:, s_t^f, u_t^f]``.

Array layouts (row-major), matching the library boundary:

* ``A[i]``: ``[G, m_i, n_{dep(i)[0]}, n_{dep(i)[1]}, ...]`` -- a "column" is the
  distribution over the ``m_i`` outcomes for one hidden-state combination;
* ``B[f]``: ``[G, n_f (next), n_f (previous), U_f]``;
* ``D[f]``: ``[G, n_f]``;
* ``obs``: ``[N, T, M]`` int32, ``act``: ``[N, T-1, F]`` int32.

``G`` is 1 when all agents share one model, else ``G == N``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

SWEEP_SIZE = 128
# Largest A_i (outcomes x hidden combinations) allowed in the random sweep.
SWEEP_CAP_ENTRIES = 1 << 18


@dataclass
class Workload:
    name: str
    algo: str  # "filter" | "vmp" | "mmp" | "all"
    n: np.ndarray  # int32 [F]
    m: np.ndarray  # int32 [M]
    dep: List[List[int]]  # per modality, 0-based factor ids in A's axis order
    U: np.ndarray  # int32 [F]
    G: int
    A: List[np.ndarray]
    B: List[np.ndarray]
    D: List[np.ndarray]
    N: int
    T: int
    K: int
    obs: np.ndarray
    act: np.ndarray
    meta: dict = field(default_factory=dict)
    bdep: Optional[List[List[int]]] = None  # B-dependencies (None: every factor depends on itself only)

    @property
    def F(self) -> int:
        return int(len(self.n))

    @property
    def M(self) -> int:
        return int(len(self.m))

    @property
    def S(self) -> int:
        return int(np.sum(self.n))

    @property
    def updates(self) -> int:
        """Belief updates in one call: agents x steps x factors x iterations."""
        return self.N * self.T * self.F * self.K

    def take_agents(self, idx: Sequence[int]) -> "Workload":
        """The same workload restricted to a subset of agents."""
        idx = np.asarray(idx, dtype=np.int64)
        if self.G == 1:
            A, B, D, G = self.A, self.B, self.D, 1
        else:
            A = [np.ascontiguousarray(a[idx]) for a in self.A]
            B = [np.ascontiguousarray(b[idx]) for b in self.B]
            D = [np.ascontiguousarray(d[idx]) for d in self.D]
            G = len(idx)
            if G == 1:
                # G == 1 means "shared"; with a single agent that is the same thing
                pass
        return Workload(
            name=self.name, algo=self.algo, n=self.n, m=self.m, dep=self.dep,
            U=self.U, G=G, A=A, B=B, D=D, N=len(idx), T=self.T, K=self.K,
            obs=np.ascontiguousarray(self.obs[idx]),
            act=np.ascontiguousarray(self.act[idx]), meta=dict(self.meta), bdep=self.bdep)


# --------------------------------------------------------------------------
# drawing probability arrays
# --------------------------------------------------------------------------

def _dirichlet_axis(rng: np.random.Generator, shape, alpha: float, axis: int) -> np.ndarray:
    """Dirichlet(alpha) draws along ``axis`` of an array of the given shape."""
    g = rng.standard_gamma(alpha, size=shape)
    # guard against an all-zero column from underflow at small alpha
    tot = g.sum(axis=axis, keepdims=True)
    bad = tot <= 0.0
    if np.any(bad):
        g = np.where(bad, 1.0, g)
        tot = g.sum(axis=axis, keepdims=True)
    return g / tot


def _sparsify(rng: np.random.Generator, a: np.ndarray, frac: float, axis: int) -> np.ndarray:
    """Zero each entry independently with probability ``frac``; renormalise the
    columns along ``axis``; columns left all-zero become uniform."""
    if frac <= 0.0:
        return a
    keep = rng.random(a.shape) >= frac
    a = a * keep
    tot = a.sum(axis=axis, keepdims=True)
    dead = tot <= 0.0
    a = np.where(dead, 1.0 / a.shape[axis], a / np.where(dead, 1.0, tot))
    return a


def make_model(rng: np.random.Generator, n, m, dep, U, G: int, *,
               a_alpha: float = 1.0, sparsity: float = 0.0,
               b_alpha: float = 1.0, b_diag: float = 0.0,
               d_alpha: Optional[float] = None, chunk: int = 128, bdep=None, b_sparsity: float = 0.0):
    """Draw A, B, D for the given structure.  ``d_alpha=None`` gives uniform D.
    ``bdep`` (per factor, the factors its transition depends on; None = its own previous state)
    gives ``B[f]`` of shape ``[G, n_f, n_bdep..., U_f]``."""
    n = np.asarray(n, dtype=np.int32)
    m = np.asarray(m, dtype=np.int32)
    U = np.asarray(U, dtype=np.int32)
    A = []
    for i, d in enumerate(dep):
        shape_tail = tuple(int(n[f]) for f in d)
        out = np.empty((G, int(m[i])) + shape_tail, dtype=np.float32)
        for g0 in range(0, G, chunk):
            g1 = min(G, g0 + chunk)
            a = _dirichlet_axis(rng, (g1 - g0, int(m[i])) + shape_tail, a_alpha, axis=1)
            a = _sparsify(rng, a, sparsity, axis=1)
            out[g0:g1] = a.astype(np.float32)
        A.append(out)
    B = []
    for f in range(len(n)):
        nf, uf = int(n[f]), int(U[f])
        if bdep is not None:
            par = tuple(int(n[g]) for g in bdep[f])
            b = _dirichlet_axis(rng, (G, nf) + par + (uf,), b_alpha, axis=1)
            b = _sparsify(rng, b, b_sparsity, axis=1)
            B.append(b.astype(np.float32))
            continue
        b = _dirichlet_axis(rng, (G, nf, nf, uf), b_alpha, axis=1)
        if b_diag > 0.0:
            b = b + b_diag * np.eye(nf)[None, :, :, None]
            b = b / b.sum(axis=1, keepdims=True)
        B.append(b.astype(np.float32))
    D = []
    for f in range(len(n)):
        nf = int(n[f])
        if d_alpha is None:
            d = np.full((G, nf), 1.0 / nf)
        else:
            d = _dirichlet_axis(rng, (G, nf), d_alpha, axis=1)
        D.append(d.astype(np.float32))
    return A, B, D


# --------------------------------------------------------------------------
# sampling trajectories from the model
# --------------------------------------------------------------------------

def _categorical(rng: np.random.Generator, p: np.ndarray) -> np.ndarray:
    """One draw per row of ``p`` ([rows, classes], rows need not sum to 1 exactly)."""
    c = np.cumsum(p.astype(np.float64), axis=1)
    u = rng.random(p.shape[0]) * c[:, -1]
    idx = (u[:, None] >= c).sum(axis=1)
    return np.minimum(idx, p.shape[1] - 1).astype(np.int32)


def sample_streams(rng: np.random.Generator, n, m, dep, U, G, A, B, D, N: int, T: int, bdep=None):
    """Sample per-agent observation and action index streams from the model."""
    F, M = len(n), len(m)
    gi = np.zeros(N, dtype=np.int64) if G == 1 else np.arange(N, dtype=np.int64)
    obs = np.empty((N, T, M), dtype=np.int32)
    act = np.empty((N, max(T - 1, 0), F), dtype=np.int32)
    s = np.empty((N, F), dtype=np.int32)
    for f in range(F):
        s[:, f] = _categorical(rng, D[f][gi])
    for t in range(T):
        for i in range(M):
            # A[i][g, :, s_dep...] -> [N, m_i]
            index = (gi, slice(None)) + tuple(s[:, f] for f in dep[i])
            p = A[i][index]
            # advanced indices separated by a slice put the broadcast axis first
            obs[:, t, i] = _categorical(rng, p)
        if t + 1 < T:
            s_prev = s.copy()   # every factor's transition reads the states of step t
            for f in range(F):
                u = rng.integers(0, int(U[f]), size=N).astype(np.int32)
                act[:, t, f] = u
                if bdep is None:
                    p = B[f][gi, :, s_prev[:, f], u]
                else:
                    p = B[f][(gi, slice(None)) + tuple(s_prev[:, g] for g in bdep[f]) + (u,)]
                s[:, f] = _categorical(rng, p)
    return obs, act


def _finish(name, algo, rng, n, m, dep, U, G, A, B, D, N, T, K, meta=None) -> Workload:
    obs, act = sample_streams(rng, n, m, dep, U, G, A, B, D, N, T)
    return Workload(name=name, algo=algo, n=np.asarray(n, np.int32), m=np.asarray(m, np.int32),
                    dep=[list(map(int, d)) for d in dep], U=np.asarray(U, np.int32), G=G,
                    A=A, B=B, D=D, N=N, T=T, K=K, obs=obs, act=act, meta=meta or {})


# --------------------------------------------------------------------------
# the five benchmark configurations
# --------------------------------------------------------------------------

def make_config(c: int, *, N: Optional[int] = None, T: Optional[int] = None,
                K: Optional[int] = None, seed: Optional[int] = None) -> Workload:
    """Configuration ``c`` in 1..4 (5 is a family: see ``make_sweep_config``).

    ``N``, ``T``, ``K`` override the benchmark's sizes (for small parity cases);
    the model structure and value distributions stay those of the configuration.
    """
    rng = np.random.default_rng(1000 + c if seed is None else seed)
    if c == 1:
        n, m, dep, U = [4, 3], [5, 4], [[0, 1], [0, 1]], [2, 2]
        N, T, K = N or 8, T or 10, K or 16
        A, B, D = make_model(rng, n, m, dep, U, 1)
        return _finish("c1_filter_tiny", "filter", rng, n, m, dep, U, 1, A, B, D, N, T, K)
    if c == 2:
        n, m, dep, U = [8, 8, 6], [16, 8, 8], [[0, 1, 2]] * 3, [4, 4, 4]
        N, T, K = N or 4096, T or 50, K or 16
        A, B, D = make_model(rng, n, m, dep, U, 1, b_alpha=0.5, b_diag=0.5)
        return _finish("c2_filter_shared", "filter", rng, n, m, dep, U, 1, A, B, D, N, T, K)
    if c == 3:
        n, m = [10, 10, 8, 6], [20, 16, 12, 8]
        dep, U = [[0, 1], [1, 2], [0, 2, 3], [0, 1, 2, 3]], [3, 3, 3, 3]
        N, T, K = N or 1024, T or 20, K or 16
        A, B, D = make_model(rng, n, m, dep, U, 1, d_alpha=1.0)
        return _finish("c3_vmp_shared", "vmp", rng, n, m, dep, U, 1, A, B, D, N, T, K)
    if c == 4:
        n, m, dep, U = [16, 12, 8], [32, 16], [[0, 1, 2]] * 2, [2, 2, 2]
        N, T, K = N or 2048, T or 20, K or 16
        A, B, D = make_model(rng, n, m, dep, U, N, sparsity=0.7)
        return _finish("c4_mmp_per_agent", "mmp", rng, n, m, dep, U, N, A, B, D, N, T, K)
    raise ValueError("configuration must be 1..4; use make_sweep_config for 5")


def sweep_structure(j: int):
    """Structure (no arrays) of member ``j`` of the randomised sweep."""
    if not 0 <= j < SWEEP_SIZE:
        raise ValueError("sweep member out of range")
    child = np.random.SeedSequence(1005).spawn(SWEEP_SIZE)[j]
    rng = np.random.default_rng(child)
    F = int(rng.integers(1, 6))
    n = rng.integers(2, 33, size=F).astype(np.int32)
    M = int(rng.integers(1, 7))
    m = rng.integers(2, 65, size=M).astype(np.int32)
    dep = []
    for i in range(M):
        chosen = None
        for _ in range(16):
            mask = rng.integers(0, 2, size=F).astype(bool)
            if not mask.any():
                continue
            d = [int(f) for f in np.flatnonzero(mask)]
            if int(m[i]) * int(np.prod(n[d], dtype=np.int64)) <= SWEEP_CAP_ENTRIES:
                chosen = d
                break
        if chosen is None:
            chosen = [int(rng.integers(0, F))]
        dep.append(chosen)
    sparsity = float(rng.choice([0.0, 0.5, 0.9]))
    U = rng.integers(1, 5, size=F).astype(np.int32)
    return rng, n, m, dep, U, sparsity


def make_sweep_config(j: int, *, N: Optional[int] = None, T: Optional[int] = None,
                      K: Optional[int] = None) -> Workload:
    """Member ``j`` (0..127) of configuration 5, run with all three algorithms."""
    rng, n, m, dep, U, sparsity = sweep_structure(j)
    N, T, K = N or 256, T or 10, K or 16
    A, B, D = make_model(rng, n, m, dep, U, 1, sparsity=sparsity, d_alpha=1.0)
    return _finish(f"c5_sweep_{j:03d}", "all", rng, n, m, dep, U, 1, A, B, D, N, T, K,
                   meta={"sparsity": sparsity, "cap_entries": SWEEP_CAP_ENTRIES})
