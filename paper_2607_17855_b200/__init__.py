"""Python binding for the ``bi`` CUDA library (B200 / sm_100a).

Argument marshalling only: every step of the belief-update path runs in the
library's kernels.  PyTorch supplies device memory and the current stream.
There is no CPU path; importing works without a GPU (so the build and the
symbol table can be checked), but every compute call needs a CUDA device and
fails loudly without one.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

from .build import LIB, build  # noqa: F401

_lib = None

BI_OK = 0
ERRORS = {0: "BI_OK", -1: "BI_ERR_INVALID_ARG", -2: "BI_ERR_SHAPE", -3: "BI_ERR_UNSUPPORTED",
          -4: "BI_ERR_ALLOC", -5: "BI_ERR_CUDA"}
BI_FLAG_OBS_RANGE = 1
BI_FLAG_ACT_RANGE = 2
BI_FLAG_COPY_TIMEOUT = 4

BI_ARITH_F64 = 0
BI_ARITH_F32 = 1
ARITH = {"f64": BI_ARITH_F64, "f32": BI_ARITH_F32}

EXPORTS = ["bi_model_create", "bi_model_create_arith", "bi_model_create_bdep", "bi_model_slice_bytes", "bi_model_set_compressed", "bi_model_arith", "bi_model_destroy", "bi_filter", "bi_filter_from", "bi_filter_continue", "bi_vmp", "bi_mmp", "bi_vmp_warm", "bi_mmp_warm", "bi_vmp_from", "bi_mmp_from", "bi_filter_soft", "bi_vmp_soft", "bi_mmp_soft", "bi_model_set_damping", "bi_status",
           "bi_last_kernel", "bi_launch_count", "bi_strerror", "bi_filter_static"]
BI_STATIC_SCRATCH_BYTES = 4 << 20


class BiError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)} ({lib().bi_strerror(code).decode()})")


class _Desc(ctypes.Structure):
    _fields_ = [("F", ctypes.c_int32), ("M", ctypes.c_int32),
                ("n", ctypes.c_void_p), ("m", ctypes.c_void_p), ("dep_len", ctypes.c_void_p),
                ("dep", ctypes.c_void_p), ("U", ctypes.c_void_p), ("G", ctypes.c_int32),
                ("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("D", ctypes.c_void_p)]


def lib():
    """Load libbi.so (building it if the sources are newer).  Raises if it cannot be loaded."""
    global _lib
    if _lib is None:
        path = build()
        L = ctypes.CDLL(path)
        L.bi_model_create.restype = ctypes.c_int
        L.bi_model_create.argtypes = [ctypes.POINTER(_Desc), ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)]
        L.bi_model_create_arith.restype = ctypes.c_int
        L.bi_model_create_arith.argtypes = [ctypes.POINTER(_Desc), ctypes.c_int, ctypes.c_void_p,
                                            ctypes.POINTER(ctypes.c_void_p)]
        L.bi_model_create_bdep.restype = ctypes.c_int
        L.bi_model_create_bdep.argtypes = [ctypes.POINTER(_Desc), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                           ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)]
        L.bi_model_set_compressed.restype = ctypes.c_int
        L.bi_model_set_compressed.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.bi_model_slice_bytes.restype = ctypes.c_int
        L.bi_model_slice_bytes.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
        L.bi_model_arith.restype = ctypes.c_int
        L.bi_model_arith.argtypes = [ctypes.c_void_p]
        L.bi_model_destroy.restype = ctypes.c_int
        L.bi_model_destroy.argtypes = [ctypes.c_void_p]
        for name in ("bi_filter", "bi_vmp", "bi_mmp", "bi_filter_soft", "bi_vmp_soft", "bi_mmp_soft"):
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.bi_filter_from.restype = ctypes.c_int
        L.bi_filter_from.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        for name in ("bi_vmp_warm", "bi_mmp_warm", "bi_filter_continue"):   # (handle, N, T, obs, act, one pointer, iters, outputs)
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_void_p]
        for name in ("bi_vmp_from", "bi_mmp_from"):
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.bi_model_set_damping.restype = ctypes.c_int
        L.bi_model_set_damping.argtypes = [ctypes.c_void_p, ctypes.c_double]
        L.bi_status.restype = ctypes.c_int
        L.bi_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        L.bi_last_kernel.restype = ctypes.c_char_p
        L.bi_last_kernel.argtypes = [ctypes.c_void_p]
        L.bi_launch_count.restype = ctypes.c_int64
        L.bi_launch_count.argtypes = [ctypes.c_void_p]
        L.bi_strerror.restype = ctypes.c_char_p
        L.bi_strerror.argtypes = [ctypes.c_int]
        L.bi_filter_static.restype = ctypes.c_int
        L.bi_filter_static.argtypes = [ctypes.POINTER(_Desc), ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def _i32(vals):
    arr = (ctypes.c_int32 * max(len(vals), 1))(*[int(v) for v in vals])
    return arr


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class Model:
    """A packed generative model on the current CUDA device (``bi_model_create``).

    ``A[i]``, ``B[f]``, ``D[f]`` are float32 CUDA tensors laid out as the
    header documents: ``A[i]: [G, m_i, n_dep...]``, ``B[f]: [G, n, n, U]``,
    ``D[f]: [G, n]``.  ``arith`` selects the kernels' arithmetic: ``"f64"``
    (default; reproduces a float64 evaluation to 1e-5) or ``"f32"`` (fast).
    ``bdep`` (per factor, the factors its transition depends on) makes a model
    with non-trivial B-dependencies (``bi_model_create_bdep``): ``B[f]`` is then
    ``[G, n_f, n_bdep..., U_f]``.
    """

    def __init__(self, n: Sequence[int], m: Sequence[int], dep: Sequence[Sequence[int]], U: Sequence[int],
                 G: int, A: List, B: List, D: List, stream=None, arith: str = "f64", bdep=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("bi needs a CUDA device: there is no CPU path")
        L = lib()
        self.n, self.m, self.U = [int(v) for v in n], [int(v) for v in m], [int(v) for v in U]
        self.dep = [[int(f) for f in d] for d in dep]
        self.G, self.F, self.M, self.S = int(G), len(self.n), len(self.m), sum(self.n)
        for t in list(A) + list(B) + list(D):
            if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
                raise ValueError("model arrays must be contiguous float32 CUDA tensors")
        d = _Desc()
        d.F, d.M, d.G = self.F, self.M, self.G
        keep = [_i32(self.n), _i32(self.m), _i32([len(x) for x in self.dep]),
                _i32([f for x in self.dep for f in x]), _i32(self.U)]
        d.n, d.m, d.dep_len, d.dep, d.U = [ctypes.cast(k, ctypes.c_void_p) for k in keep]
        pa = (ctypes.c_void_p * max(self.M, 1))(*[a.data_ptr() for a in A])
        pb = (ctypes.c_void_p * self.F)(*[b.data_ptr() for b in B])
        pd = (ctypes.c_void_p * self.F)(*[x.data_ptr() for x in D])
        d.A, d.B, d.D = [ctypes.cast(p, ctypes.c_void_p) for p in (pa, pb, pd)]
        h = ctypes.c_void_p()
        self.bdep = [[int(g) for g in x] for x in bdep] if bdep is not None else None
        if self.bdep is not None:
            bl, bf = _i32([len(x) for x in self.bdep]), _i32([g for x in self.bdep for g in x])
            rc = L.bi_model_create_bdep(ctypes.byref(d), ctypes.cast(bl, ctypes.c_void_p), ctypes.cast(bf, ctypes.c_void_p),
                                        ARITH[arith], _stream_ptr(stream), ctypes.byref(h))
        elif arith == "f64":
            rc = L.bi_model_create(ctypes.byref(d), _stream_ptr(stream), ctypes.byref(h))
        else:
            rc = L.bi_model_create_arith(ctypes.byref(d), ARITH[arith], _stream_ptr(stream), ctypes.byref(h))
        if rc != BI_OK:
            raise BiError(rc, "bi_model_create")
        self._h = h
        self.arith = arith
        assert L.bi_model_arith(h) == ARITH[arith]

    def close(self):
        if getattr(self, "_h", None):
            lib().bi_model_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- inference -----------------------------------------------------------
    def _run(self, name, obs, act, iters, q_out, logq_out, argmax_out, stream):
        import torch
        N, T = int(obs.shape[0]), int(obs.shape[1])
        if q_out is None:
            q_out = torch.empty((N, T, self.S), dtype=torch.float32, device=obs.device)
        fn = getattr(lib(), name)
        rc = fn(self._h, N, T, ctypes.c_void_p(obs.data_ptr()),
                ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                int(iters), ctypes.c_void_p(q_out.data_ptr()),
                ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                _stream_ptr(stream))
        if rc != BI_OK:
            raise BiError(rc, name)
        return q_out

    def bi_filter(self, obs, act, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """Variational filtering; ``obs`` int32 ``[N,T,M]``, ``act`` int32 ``[N,T-1,F]`` (CUDA)."""
        return self._run("bi_filter", obs, act, iters, q_out, logq_out, argmax_out, stream)

    def bi_filter_from(self, obs, act, q_prev, act_prev, iters, q_out=None, logq_out=None, argmax_out=None,
                       stream=None):
        """Filtering continued from ``q_prev`` float32 ``[N,S]`` (the belief of the step before
        this window) and ``act_prev`` int32 ``[N,F]`` (the action taken there)."""
        import torch
        N, T = int(obs.shape[0]), int(obs.shape[1])
        if q_out is None:
            q_out = torch.empty((N, T, self.S), dtype=torch.float32, device=obs.device)
        rc = lib().bi_filter_from(self._h, N, T, ctypes.c_void_p(obs.data_ptr()),
                                  ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                                  ctypes.c_void_p(q_prev.data_ptr()), ctypes.c_void_p(act_prev.data_ptr()),
                                  int(iters), ctypes.c_void_p(q_out.data_ptr()),
                                  ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                                  ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                                  _stream_ptr(stream))
        if rc != BI_OK:
            raise BiError(rc, "bi_filter_from")
        return q_out

    def bi_filter_continue(self, obs, act, act_prev, iters, q_out=None, logq_out=None, argmax_out=None,
                           stream=None):
        """Filtering continued from the belief this handle kept from its previous filtering call
        (full precision: consecutive blocks equal the single call bit for bit); ``act_prev`` int32
        ``[N,F]`` is the action taken at that call's last step."""
        import torch
        N, T = int(obs.shape[0]), int(obs.shape[1])
        if q_out is None:
            q_out = torch.empty((N, T, self.S), dtype=torch.float32, device=obs.device)
        rc = lib().bi_filter_continue(self._h, N, T, ctypes.c_void_p(obs.data_ptr()),
                                      ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                                      ctypes.c_void_p(act_prev.data_ptr()), int(iters),
                                      ctypes.c_void_p(q_out.data_ptr()),
                                      ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                                      ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                                      _stream_ptr(stream))
        if rc != BI_OK:
            raise BiError(rc, "bi_filter_continue")
        return q_out

    def bi_vmp(self, obs, act, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """Variational message passing over one window."""
        return self._run("bi_vmp", obs, act, iters, q_out, logq_out, argmax_out, stream)

    def bi_mmp(self, obs, act, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """Marginal message passing over one window."""
        return self._run("bi_mmp", obs, act, iters, q_out, logq_out, argmax_out, stream)

    def _run_warm(self, name, obs, act, q_init, iters, q_out, logq_out, argmax_out, stream):
        import torch
        N, T = int(obs.shape[0]), int(obs.shape[1])
        if q_out is None:
            q_out = torch.empty((N, T, self.S), dtype=torch.float32, device=obs.device)
        rc = getattr(lib(), name)(self._h, N, T, ctypes.c_void_p(obs.data_ptr()),
                                  ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                                  ctypes.c_void_p(q_init.data_ptr()), int(iters), ctypes.c_void_p(q_out.data_ptr()),
                                  ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                                  ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                                  _stream_ptr(stream))
        if rc != BI_OK:
            raise BiError(rc, name)
        return q_out

    def bi_vmp_warm(self, obs, act, q_init, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """``bi_vmp`` started from ``q_init`` float32 ``[N,T,S]`` instead of uniform beliefs."""
        return self._run_warm("bi_vmp_warm", obs, act, q_init, iters, q_out, logq_out, argmax_out, stream)

    def bi_mmp_warm(self, obs, act, q_init, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """``bi_mmp`` started from ``q_init`` float32 ``[N,T,S]`` instead of uniform beliefs."""
        return self._run_warm("bi_mmp_warm", obs, act, q_init, iters, q_out, logq_out, argmax_out, stream)

    def run_from(self, algo, obs, act, q_prev, act_prev, iters, q_init=None, q_out=None, logq_out=None,
                 argmax_out=None, stream=None):
        """``bi_filter_from`` / ``bi_vmp_from`` / ``bi_mmp_from``: the call continues a stream from
        ``q_prev`` float32 ``[N,S]`` and ``act_prev`` int32 ``[N,F]``."""
        if algo == "filter":
            return self.bi_filter_from(obs, act, q_prev, act_prev, iters, q_out, logq_out, argmax_out, stream)
        import torch
        N, T = int(obs.shape[0]), int(obs.shape[1])
        if q_out is None:
            q_out = torch.empty((N, T, self.S), dtype=torch.float32, device=obs.device)
        name = "bi_vmp_from" if algo == "vmp" else "bi_mmp_from"
        rc = getattr(lib(), name)(self._h, N, T, ctypes.c_void_p(obs.data_ptr()),
                                  ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                                  ctypes.c_void_p(q_prev.data_ptr()), ctypes.c_void_p(act_prev.data_ptr()),
                                  ctypes.c_void_p(q_init.data_ptr() if q_init is not None else None), int(iters),
                                  ctypes.c_void_p(q_out.data_ptr()),
                                  ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                                  ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                                  _stream_ptr(stream))
        if rc != BI_OK:
            raise BiError(rc, name)
        return q_out

    def run_soft(self, algo, obs_soft, act, iters, q_out=None, logq_out=None, argmax_out=None, stream=None):
        """``bi_filter_soft`` / ``bi_vmp_soft`` / ``bi_mmp_soft``: observations as categorical vectors,
        ``obs_soft`` float32 ``[N,T,sum(m)]`` (CUDA)."""
        return self._run({"filter": "bi_filter_soft", "vmp": "bi_vmp_soft", "mmp": "bi_mmp_soft"}[algo], obs_soft,
                         act, iters, q_out, logq_out, argmax_out, stream)

    def run(self, algo, *a, **k):
        return {"filter": self.bi_filter, "vmp": self.bi_vmp, "mmp": self.bi_mmp}[algo](*a, **k)

    def set_damping(self, lam: float):
        """Step size of the update on log-beliefs for every later call (1 = the plain update)."""
        rc = lib().bi_model_set_damping(self._h, float(lam))
        if rc != BI_OK:
            raise BiError(rc, "bi_model_set_damping")

    def status(self, stream=None) -> int:
        v = ctypes.c_uint32(0)
        rc = lib().bi_status(self._h, _stream_ptr(stream), ctypes.byref(v))
        if rc != BI_OK:
            raise BiError(rc, "bi_status")
        return int(v.value)

    def set_compressed(self, on: bool):
        """Window calls gather from the compressed slices (``bi_model_set_compressed``)."""
        rc = lib().bi_model_set_compressed(self._h, int(bool(on)))
        if rc != BI_OK:
            raise BiError(rc, "bi_model_set_compressed")

    def slice_bytes(self):
        """(dense, compressed) bytes of a per-agent model's slices as the window kernels gather them
        (``bi_model_slice_bytes``); (0, 0) when the handle keeps no compressed form."""
        a, b = ctypes.c_int64(0), ctypes.c_int64(0)
        rc = lib().bi_model_slice_bytes(self._h, ctypes.byref(a), ctypes.byref(b))
        if rc != BI_OK:
            raise BiError(rc, "bi_model_slice_bytes")
        return int(a.value), int(b.value)

    @property
    def last_kernel(self) -> str:
        return lib().bi_last_kernel(self._h).decode()

    @property
    def launch_count(self) -> int:
        return int(lib().bi_launch_count(self._h))


def bi_filter_static(n, m, dep, U, A, B, D, obs, act, iters, q_out, logq_out=None, argmax_out=None, stream=None):
    """Filtering for callers that must not allocate (``bi_filter_static``).

    The library packs the shared model ``A``, ``B``, ``D`` (float32 CUDA
    tensors laid out as for :class:`Model`, ``G == 1``) into its own fixed
    scratch array on every call instead of using a handle, so no device memory
    is obtained anywhere on this path; the caller supplies every output
    tensor.  Calls share that one array: do not let two of them overlap on the
    GPU.  The model must pack into ``BI_STATIC_SCRATCH_BYTES``.
    """
    L = lib()
    n, m, U = [int(v) for v in n], [int(v) for v in m], [int(v) for v in U]
    dep = [[int(f) for f in d] for d in dep]
    d = _Desc()
    d.F, d.M, d.G = len(n), len(m), 1
    keep = [_i32(n), _i32(m), _i32([len(x) for x in dep]), _i32([f for x in dep for f in x]), _i32(U)]
    d.n, d.m, d.dep_len, d.dep, d.U = [ctypes.cast(k, ctypes.c_void_p) for k in keep]
    pa = (ctypes.c_void_p * max(len(m), 1))(*[a.data_ptr() for a in A])
    pb = (ctypes.c_void_p * len(n))(*[b.data_ptr() for b in B])
    pd = (ctypes.c_void_p * len(n))(*[x.data_ptr() for x in D])
    d.A, d.B, d.D = [ctypes.cast(p, ctypes.c_void_p) for p in (pa, pb, pd)]
    N, T = int(obs.shape[0]), int(obs.shape[1])
    rc = L.bi_filter_static(ctypes.byref(d), N, T, ctypes.c_void_p(obs.data_ptr()),
                            ctypes.c_void_p(act.data_ptr() if act is not None and act.numel() > 0 else None),
                            int(iters), ctypes.c_void_p(q_out.data_ptr()),
                            ctypes.c_void_p(logq_out.data_ptr() if logq_out is not None else None),
                            ctypes.c_void_p(argmax_out.data_ptr() if argmax_out is not None else None),
                            _stream_ptr(stream))
    if rc != BI_OK:
        raise BiError(rc, "bi_filter_static")
    return q_out


def model_from_workload(w, device="cuda", stream=None, arith: str = "f64") -> Model:
    """Upload a workload's arrays (numpy) and pack them."""
    import torch
    A = [torch.from_numpy(a).to(device) for a in w.A]
    B = [torch.from_numpy(b).to(device) for b in w.B]
    D = [torch.from_numpy(d).to(device) for d in w.D]
    md = Model(w.n, w.m, w.dep, w.U, w.G, A, B, D, stream=stream, arith=arith, bdep=getattr(w, "bdep", None))
    torch.cuda.synchronize()
    return md
