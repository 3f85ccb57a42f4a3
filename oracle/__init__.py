"""ctypes loader for the CPU oracle (``bi_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Importers: ``tests/``, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA package never imports this module, and
this module imports nothing from the CUDA package.

``build()`` compiles the C file with gcc next to it; ``run()`` marshals numpy
arrays into the C entry point.  No arithmetic of the method lives here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bi_oracle.c")
_LIB = os.path.join(_HERE, "libbi_oracle.so")
_lib = None

ALGOS = {"filter": 0, "vmp": 1, "mmp": 2}


def build(force: bool = False) -> str:
    """Compile the oracle shared library if it is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.bi_ref_run.restype = ctypes.c_int
        lib.bi_ref_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().bi_ref_max_threads())


def _ptr_array(arrs):
    arr_t = ctypes.c_void_p * max(len(arrs), 1)
    return arr_t(*[a.ctypes.data for a in arrs])


def run(algo: str, n: Sequence[int], m: Sequence[int], dep, U: Sequence[int], G: int,
        A, B, D, obs: np.ndarray, act: Optional[np.ndarray], K: int, *,
        q_init: Optional[np.ndarray] = None, threads: int = 0, round32: bool = False,
        q_prev: Optional[np.ndarray] = None, act_prev: Optional[np.ndarray] = None,
        obs_soft: Optional[np.ndarray] = None, damping: float = 1.0, bdep=None):
    """Run ``algo`` ('filter' | 'vmp' | 'mmp') and return ``(q, logq, argmax)``.

    ``obs`` is ``[N, T, M]`` int32, ``act`` ``[N, T-1, F]`` int32 (ignored when
    T == 1); ``q`` and ``logq`` come back as float64 ``[N, T, S]``, ``argmax`` as
    int32 ``[N, T, F]``.  ``q_prev`` ``[N, S]`` with ``act_prev`` ``[N, F]``
    continue a stream: the first step's prior is ``B_u q_prev`` instead of
    ``D`` (for the window algorithms at full weight, like ``D``).  ``obs_soft`` float32 ``[N, T, sum(m)]``
    replaces ``obs`` (pass ``obs=None``): every observation is a categorical
    vector per modality and the log-likelihood is ``log(A_i) . o^i``.
    ``damping`` in (0, 1]: step size of the update on log-beliefs (1 = plain).
    ``bdep`` (a list of factor lists, or None): B-dependencies -- factor f's transition depends on the
    previous states of ``bdep[f]`` and ``B[f]`` is ``[G, n_f, n_bdep..., U_f]``; filtering and VMP only.
    """
    if (q_prev is None) != (act_prev is None):
        raise ValueError("q_prev and act_prev go together")
    lib = _load()
    n = np.ascontiguousarray(n, dtype=np.int32)
    m = np.ascontiguousarray(m, dtype=np.int32)
    U = np.ascontiguousarray(U, dtype=np.int32)
    F, M = len(n), len(m)
    dep_len = np.ascontiguousarray([len(d) for d in dep], dtype=np.int32)
    dep_flat = np.ascontiguousarray([f for d in dep for f in d] or [0], dtype=np.int32)
    A = [np.ascontiguousarray(a, dtype=np.float32) for a in A]
    B = [np.ascontiguousarray(b, dtype=np.float32) for b in B]
    D = [np.ascontiguousarray(d, dtype=np.float32) for d in D]
    if obs_soft is not None:
        assert obs is None and q_init is None and q_prev is None and not round32
        obs_soft = np.ascontiguousarray(obs_soft, dtype=np.float32)
        N, T = int(obs_soft.shape[0]), int(obs_soft.shape[1])
        assert obs_soft.shape == (N, T, int(m.sum()))
    else:
        obs = np.ascontiguousarray(obs, dtype=np.int32)
        N, T = int(obs.shape[0]), int(obs.shape[1])
        assert obs.shape == (N, T, M)
    if T > 1:
        act = np.ascontiguousarray(act, dtype=np.int32)
        assert act.shape == (N, T - 1, F)
        act_p = act.ctypes.data
    else:
        act_p = None
    S = int(n.sum())
    for i, a in enumerate(A):
        assert a.shape == (G, int(m[i])) + tuple(int(n[f]) for f in dep[i]), (i, a.shape)
    for f in range(F):
        par = tuple(int(n[g]) for g in bdep[f]) if bdep is not None else (int(n[f]),)
        assert B[f].shape == (G, int(n[f])) + par + (int(U[f]),), (f, B[f].shape)
        assert D[f].shape == (G, int(n[f]))
    q = np.empty((N, T, S), dtype=np.float64)
    lq = np.empty((N, T, S), dtype=np.float64)
    am = np.empty((N, T, F), dtype=np.int32)
    if q_init is not None:
        q_init = np.ascontiguousarray(q_init, dtype=np.float64)
        assert q_init.shape == (N, T, S)
    Ap, Bp, Dp = _ptr_array(A), _ptr_array(B), _ptr_array(D)
    if bdep is not None:
        assert obs_soft is None and not round32
        bl = np.ascontiguousarray([len(d) for d in bdep], dtype=np.int32)
        bf = np.ascontiguousarray([g for d in bdep for g in d], dtype=np.int32)
        if q_prev is not None:
            q_prev = np.ascontiguousarray(q_prev, dtype=np.float64)
            act_prev = np.ascontiguousarray(act_prev, dtype=np.int32)
            assert q_prev.shape == (N, S) and act_prev.shape == (N, F)
        rc = lib.bi_ref_run_bdep_damped(
            ctypes.c_int(ALGOS[algo]), ctypes.c_int(F), ctypes.c_int(M),
            ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
            ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
            ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
            ctypes.c_void_p(bl.ctypes.data), ctypes.c_void_p(bf.ctypes.data),
            ctypes.c_int(N), ctypes.c_int(T), ctypes.c_void_p(obs.ctypes.data), ctypes.c_void_p(act_p),
            ctypes.c_int(K), ctypes.c_void_p(q_init.ctypes.data if q_init is not None else None),
            ctypes.c_void_p(q_prev.ctypes.data if q_prev is not None else None),
            ctypes.c_void_p(act_prev.ctypes.data if act_prev is not None else None),
            ctypes.c_double(float(damping)),
            ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
            ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads))
        if rc != 0:
            raise ValueError(f"bi_ref_run_bdep rejected its arguments (code {rc})")
        return q, lq, am
    if damping != 1.0:
        if q_prev is not None:
            q_prev = np.ascontiguousarray(q_prev, dtype=np.float64)
            act_prev = np.ascontiguousarray(act_prev, dtype=np.int32)
            assert q_prev.shape == (N, S) and act_prev.shape == (N, F)
        rc = lib.bi_ref_run_opts(
            ctypes.c_int(ALGOS[algo]), ctypes.c_int(F), ctypes.c_int(M),
            ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
            ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
            ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
            ctypes.c_int(N), ctypes.c_int(T),
            ctypes.c_void_p(obs.ctypes.data if obs is not None else None),
            ctypes.c_void_p(obs_soft.ctypes.data if obs_soft is not None else None),
            ctypes.c_void_p(act_p), ctypes.c_int(K),
            ctypes.c_void_p(q_init.ctypes.data if q_init is not None else None),
            ctypes.c_void_p(q_prev.ctypes.data if q_prev is not None else None),
            ctypes.c_void_p(act_prev.ctypes.data if act_prev is not None else None),
            ctypes.c_double(float(damping)),
            ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
            ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads), ctypes.c_int(int(round32)))
        if rc != 0:
            raise ValueError(f"bi_ref_run_opts rejected its arguments (code {rc})")
        return q, lq, am
    if obs_soft is not None:
        rc = lib.bi_ref_run_soft(
            ctypes.c_int(ALGOS[algo]), ctypes.c_int(F), ctypes.c_int(M),
            ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
            ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
            ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
            ctypes.c_int(N), ctypes.c_int(T), ctypes.c_void_p(obs_soft.ctypes.data),
            ctypes.c_void_p(act_p), ctypes.c_int(K),
            ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
            ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads))
        if rc != 0:
            raise ValueError(f"bi_ref_run_soft rejected its arguments (code {rc})")
        return q, lq, am
    if (q_prev is not None or act_prev is not None) and algo != "filter":
        assert not round32
        q_prev = np.ascontiguousarray(q_prev, dtype=np.float64)
        act_prev = np.ascontiguousarray(act_prev, dtype=np.int32)
        assert q_prev.shape == (N, S) and act_prev.shape == (N, F)
        rc = lib.bi_ref_window_from(
            ctypes.c_int(ALGOS[algo]), ctypes.c_int(F), ctypes.c_int(M),
            ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
            ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
            ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
            ctypes.c_int(N), ctypes.c_int(T), ctypes.c_void_p(obs.ctypes.data),
            ctypes.c_void_p(act_p), ctypes.c_int(K),
            ctypes.c_void_p(q_init.ctypes.data if q_init is not None else None),
            ctypes.c_void_p(q_prev.ctypes.data), ctypes.c_void_p(act_prev.ctypes.data),
            ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
            ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads))
        if rc != 0:
            raise ValueError(f"bi_ref_window_from rejected its arguments (code {rc})")
        return q, lq, am
    if q_prev is not None or act_prev is not None:
        assert algo == "filter" and q_init is None and not round32
        q_prev = np.ascontiguousarray(q_prev, dtype=np.float64)
        act_prev = np.ascontiguousarray(act_prev, dtype=np.int32)
        assert q_prev.shape == (N, S) and act_prev.shape == (N, F)
        rc = lib.bi_ref_filter_from(
            ctypes.c_int(F), ctypes.c_int(M),
            ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
            ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
            ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
            ctypes.c_int(N), ctypes.c_int(T), ctypes.c_void_p(obs.ctypes.data),
            ctypes.c_void_p(act_p), ctypes.c_int(K),
            ctypes.c_void_p(q_prev.ctypes.data), ctypes.c_void_p(act_prev.ctypes.data),
            ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
            ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads))
        if rc != 0:
            raise ValueError(f"bi_ref_filter_from rejected its arguments (code {rc})")
        return q, lq, am
    rc = lib.bi_ref_run(
        ctypes.c_int(ALGOS[algo]), ctypes.c_int(F), ctypes.c_int(M),
        ctypes.c_void_p(n.ctypes.data), ctypes.c_void_p(m.ctypes.data),
        ctypes.c_void_p(dep_len.ctypes.data), ctypes.c_void_p(dep_flat.ctypes.data),
        ctypes.c_void_p(U.ctypes.data), ctypes.c_int(G), Ap, Bp, Dp,
        ctypes.c_int(N), ctypes.c_int(T), ctypes.c_void_p(obs.ctypes.data),
        ctypes.c_void_p(act_p), ctypes.c_int(K),
        ctypes.c_void_p(q_init.ctypes.data if q_init is not None else None),
        ctypes.c_void_p(q.ctypes.data), ctypes.c_void_p(lq.ctypes.data),
        ctypes.c_void_p(am.ctypes.data), ctypes.c_int(threads), ctypes.c_int(int(round32)))
    if rc != 0:
        raise ValueError(f"bi_ref_run rejected its arguments (code {rc})")
    return q, lq, am


def run_workload(w, algo: Optional[str] = None, **kw):
    """Convenience: run on an object with the workload generator's field names."""
    if getattr(w, "bdep", None) is not None:
        kw.setdefault("bdep", w.bdep)
    return run(algo or w.algo, w.n, w.m, w.dep, w.U, w.G, w.A, w.B, w.D, w.obs, w.act, w.K, **kw)
