"""Thin ctypes binding of libflashgmm (see include/flashgmm.h): argument marshalling only.

torch supplies device memory and the stream; every numerical step runs in the library's CUDA kernels.  Importing
this module loads ``libflashgmm.so`` from the package directory and raises if it is missing -- there is no CPU or
PyTorch fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np
import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libflashgmm.so"

GMM_OK = 0
GMM_EINVAL, GMM_EALIGN, GMM_ENOMEM, GMM_ECUDA, GMM_ENUMERIC, GMM_ETIMEOUT, GMM_EUNSUPPORTED = -1, -2, -3, -4, -5, -6, -7
GMM_PATH_AUTO, GMM_PATH_FP32, GMM_PATH_TENSOR = 0, 1, 2
GMM_MAX_TOPM = 8
GMM_COV_DIAG, GMM_COV_ISOTROPIC = 0, 1

EXPORTS = {
    # name: (restype, argtypes)
    "gmm_create": (ctypes.c_int, [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, ctypes.c_void_p]),
    "gmm_destroy": (ctypes.c_int, [ctypes.c_void_p]),
    "gmm_set_path": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "gmm_last_path": (ctypes.c_int, [ctypes.c_void_p]),
    "gmm_last_exact_count": (ctypes.c_int, [ctypes.c_void_p]),
    "gmm_last_exact_pairs": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                                            ctypes.POINTER(ctypes.c_int)]),
    "gmm_tensor_path_supports": (ctypes.c_int, [ctypes.c_int, ctypes.c_int]),
    "gmm_auto_path": (ctypes.c_int, [ctypes.c_int, ctypes.c_int]),
    "gmm_em_step": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                   ctypes.POINTER(ctypes.c_double)]),
    "gmm_em_step_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.POINTER(ctypes.c_double)]),
    "gmm_finalize": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "gmm_finalize_isotropic": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                              ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "gmm_set_covariance": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "gmm_fit": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                               ctypes.c_int, ctypes.c_float, ctypes.c_double,
                               ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int)]),
    "gmm_assign_topm": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p]),
    "gmm_build_posting_lists": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_float, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double)]),
    "gmm_kmeans_step": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.POINTER(ctypes.c_double)]),
    "gmm_score_samples": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.POINTER(ctypes.c_double)]),
    "gmm_fisher_vectors": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.POINTER(ctypes.c_double)]),
    "gmm_em_step_static": (ctypes.c_int, [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.POINTER(ctypes.c_double)]),
    "gmm_sync_status": (ctypes.c_int, [ctypes.c_void_p]),
    "gmm_update_counts": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]),
    "gmm_scratch_bytes": (ctypes.c_size_t, [ctypes.c_int, ctypes.c_int]),
    "gmm_launch_count": (ctypes.c_int64, [ctypes.c_void_p]),
    "gmm_set_profiling": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "gmm_kernel_time": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_int64)]),
    "gmm_reset_counters": (ctypes.c_int, [ctypes.c_void_p]),
    "gmm_probe_rates": (ctypes.c_int, [ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]),
    "gmm_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "gmm_last_error": (ctypes.c_char_p, [ctypes.c_void_p]),
    "gmm_version": (ctypes.c_char_p, []),
}


def _load() -> ctypes.CDLL:
    if not LIB_PATH.exists():
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2606_10896_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(str(LIB_PATH))
    for name, (restype, argtypes) in EXPORTS.items():
        fn = getattr(lib, name)
        fn.restype = restype
        fn.argtypes = argtypes
    return lib


lib = _load()


class GmmError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"libflashgmm error {code} ({lib.gmm_strerror(code).decode()}): {message}")
        self.code = code


def tensor_path_supports(D: int, K: int) -> bool:
    return bool(lib.gmm_tensor_path_supports(int(D), int(K)))


def gmm_auto_path(D: int, K: int) -> int:
    return int(lib.gmm_auto_path(int(D), int(K)))


def gmm_probe_rates(device: int = 0):
    """(fp32 FMA flop/s, ex2 results/s) measured on the device by two short micro-benchmarks."""
    a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = lib.gmm_probe_rates(int(device), ctypes.byref(a), ctypes.byref(b))
    if rc != GMM_OK:
        raise GmmError(rc, "gmm_probe_rates failed")
    return a.value, b.value


def gmm_scratch_bytes(D: int, K: int) -> int:
    return int(lib.gmm_scratch_bytes(D, K))


def _dev(t: torch.Tensor, dtype, shape, name: str):
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous {dtype} of shape {tuple(shape)}, got {t.dtype} {tuple(t.shape)}")
    return ctypes.c_void_p(t.data_ptr())


def _host(a: np.ndarray, dtype, shape, name: str):
    if not isinstance(a, np.ndarray) or a.dtype != dtype or tuple(a.shape) != tuple(shape) or not a.flags.c_contiguous:
        raise TypeError(f"{name} must be a C-contiguous numpy {np.dtype(dtype).name} array of shape {tuple(shape)}")
    return ctypes.c_void_p(a.ctypes.data)


def gmm_em_step_static(X, pi, mu, var, out, stream: torch.cuda.Stream | None = None):
    """gmm_em_step for callers that may not allocate device memory: no context, scratch in the library's own
    static device array (K <= 1024, K * D <= 32768).  ``out`` = (Nk, S1, S2) preallocated float64 CUDA tensors --
    this wrapper allocates nothing on the device either.  Returns the log-likelihood.  Calls that overlap on one
    GPU race on the shared scratch; the first call on a device should precede any stream capture."""
    N, D = X.shape
    K = pi.shape[0]
    Nk, S1, S2 = out
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    ll = ctypes.c_double(0.0)
    rc = lib.gmm_em_step_static(X.device.index or 0, ctypes.c_void_p(st.cuda_stream),
                                _dev(X, torch.float32, (N, D), "X"), N, D, K,
                                _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                                _dev(var, torch.float32, (K, D), "var"),
                                _dev(Nk, torch.float64, (K,), "Nk"), _dev(S1, torch.float64, (K, D), "S1"),
                                _dev(S2, torch.float64, (K, D), "S2"), ctypes.byref(ll))
    if rc != GMM_OK:
        raise GmmError(rc, "gmm_em_step_static failed")
    return ll.value


class Context:
    """One libflashgmm context bound to a device and to the torch stream current at construction (or ``stream``)."""

    def __init__(self, device: int | torch.device = 0, stream: torch.cuda.Stream | None = None):
        dev = torch.device(device if not isinstance(device, int) else f"cuda:{device}")
        self.device = dev
        torch.cuda.init()
        with torch.cuda.device(dev):
            torch.zeros(1, device=dev)          # make sure the primary context exists
            self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self._h = ctypes.c_void_p()
        rc = lib.gmm_create(ctypes.byref(self._h), dev.index or 0, ctypes.c_void_p(self.stream.cuda_stream))
        if rc != GMM_OK:
            raise GmmError(rc, "gmm_create failed")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            lib.gmm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _check(self, rc: int):
        if rc != GMM_OK:
            raise GmmError(rc, lib.gmm_last_error(self._h).decode())

    # ---- options / instrumentation ----
    def gmm_set_path(self, path: int):
        self._check(lib.gmm_set_path(self._h, path))

    def gmm_last_path(self) -> int:
        return int(lib.gmm_last_path(self._h))

    def gmm_last_exact_count(self) -> int:
        return int(lib.gmm_last_exact_count(self._h))

    def gmm_last_exact_pairs(self):
        """(marked, kept, dense_pieces) of the most recent wide tensor-path step: see include/flashgmm.h."""
        a, b, c = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int(0)
        self._check(lib.gmm_last_exact_pairs(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return int(a.value), int(b.value), int(c.value)

    def gmm_launch_count(self) -> int:
        return int(lib.gmm_launch_count(self._h))

    def gmm_set_profiling(self, on: bool):
        self._check(lib.gmm_set_profiling(self._h, int(bool(on))))

    def gmm_kernel_time(self):
        ms, n = ctypes.c_double(0), ctypes.c_int64(0)
        self._check(lib.gmm_kernel_time(self._h, ctypes.byref(ms), ctypes.byref(n)))
        return ms.value, n.value

    def gmm_reset_counters(self):
        self._check(lib.gmm_reset_counters(self._h))

    def gmm_sync_status(self):
        """Waits for the stream; raises GmmError if an earlier asynchronous call recorded an error on the device."""
        self._check(lib.gmm_sync_status(self._h))

    def gmm_update_counts(self):
        """(variance entries raised to the floor, components left unchanged as empty) of the last parameter update."""
        fl, em = ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(lib.gmm_update_counts(self._h, ctypes.byref(fl), ctypes.byref(em)))
        return int(fl.value), int(em.value)

    # ---- compute ----
    def gmm_em_step(self, X, pi, mu, var, out=None):
        """(Nk [K], S1 [K, D], S2 [K, D]) as float64 CUDA tensors and the log-likelihood (float)."""
        N, D = X.shape
        K = pi.shape[0]
        if out is None:
            Nk = torch.empty(K, dtype=torch.float64, device=X.device)
            S1 = torch.empty((K, D), dtype=torch.float64, device=X.device)
            S2 = torch.empty((K, D), dtype=torch.float64, device=X.device)
        else:
            Nk, S1, S2 = out
        ll = ctypes.c_double(0.0)
        rc = lib.gmm_em_step(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K,
                             _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                             _dev(var, torch.float32, (K, D), "var"),
                             _dev(Nk, torch.float64, (K,), "Nk"), _dev(S1, torch.float64, (K, D), "S1"),
                             _dev(S2, torch.float64, (K, D), "S2"), ctypes.byref(ll))
        self._check(rc)
        return Nk, S1, S2, ll.value

    def gmm_em_step_host(self, X, pi, mu, var, out=None):
        """Same statistics with every array a host numpy array (X may live in pinned memory)."""
        N, D = X.shape
        K = pi.shape[0]
        if out is None:
            Nk = np.empty(K, np.float64)
            S1 = np.empty((K, D), np.float64)
            S2 = np.empty((K, D), np.float64)
        else:
            Nk, S1, S2 = out
        ll = ctypes.c_double(0.0)
        rc = lib.gmm_em_step_host(self._h, _host(X, np.float32, (N, D), "X"), N, D, K,
                                  _host(pi, np.float32, (K,), "pi"), _host(mu, np.float32, (K, D), "mu"),
                                  _host(var, np.float32, (K, D), "var"),
                                  _host(Nk, np.float64, (K,), "Nk"), _host(S1, np.float64, (K, D), "S1"),
                                  _host(S2, np.float64, (K, D), "S2"), ctypes.byref(ll))
        self._check(rc)
        return Nk, S1, S2, ll.value

    def gmm_finalize(self, N, Nk, S1, S2, var_floor, pi, mu, var):
        """In-place parameter update of the CUDA tensors pi, mu, var from the statistics."""
        K, D = mu.shape
        rc = lib.gmm_finalize(self._h, int(N), D, K, _dev(Nk, torch.float64, (K,), "Nk"),
                              _dev(S1, torch.float64, (K, D), "S1"), _dev(S2, torch.float64, (K, D), "S2"),
                              float(var_floor), _dev(pi, torch.float32, (K,), "pi"),
                              _dev(mu, torch.float32, (K, D), "mu"), _dev(var, torch.float32, (K, D), "var"))
        self._check(rc)

    def gmm_finalize_isotropic(self, N, Nk, S1, S2, var_floor, pi, mu, var):
        """In-place update for the paper's isotropic model (one variance per component, replicated over d)."""
        K, D = mu.shape
        rc = lib.gmm_finalize_isotropic(self._h, int(N), D, K, _dev(Nk, torch.float64, (K,), "Nk"),
                                        _dev(S1, torch.float64, (K, D), "S1"), _dev(S2, torch.float64, (K, D), "S2"),
                                        float(var_floor), _dev(pi, torch.float32, (K,), "pi"),
                                        _dev(mu, torch.float32, (K, D), "mu"), _dev(var, torch.float32, (K, D), "var"))
        self._check(rc)

    def gmm_set_covariance(self, covariance: int):
        self._check(lib.gmm_set_covariance(self._h, int(covariance)))

    def gmm_fit(self, X, pi, mu, var, iters, var_floor=1e-6, tol=0.0):
        """Runs EM in place on pi, mu, var; returns (loglik_trace float64 numpy [iters_done], iters_done)."""
        N, D = X.shape
        K = pi.shape[0]
        trace = np.zeros(int(iters), np.float64)
        done = ctypes.c_int(0)
        rc = lib.gmm_fit(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K,
                         _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                         _dev(var, torch.float32, (K, D), "var"), int(iters), float(var_floor), float(tol),
                         trace.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), ctypes.byref(done))
        self._check(rc)
        return trace[: done.value].copy(), done.value

    def gmm_assign_topm(self, X, pi, mu, var, m, out=None, indices_only=False):
        """(idx int32 [N, m], resp float32 [N, m]) CUDA tensors; asynchronous on the context's stream.
        indices_only: resp is not computed (returned as None; ``out`` is then (idx, None))."""
        N, D = X.shape
        K = pi.shape[0]
        if out is None:
            idx = torch.empty((N, m), dtype=torch.int32, device=X.device)
            resp = None if indices_only else torch.empty((N, m), dtype=torch.float32, device=X.device)
        else:
            idx, resp = out
        if resp is None:
            rc = lib.gmm_assign_topm(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K,
                                     _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                                     _dev(var, torch.float32, (K, D), "var"), int(m),
                                     _dev(idx, torch.int32, (N, m), "idx"), None)
            self._check(rc)
            return idx, None
        rc = lib.gmm_assign_topm(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K,
                                 _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                                 _dev(var, torch.float32, (K, D), "var"), int(m),
                                 _dev(idx, torch.int32, (N, m), "idx"), _dev(resp, torch.float32, (N, m), "resp"))
        self._check(rc)
        return idx, resp

    def gmm_build_posting_lists(self, idx, resp, K, tau=None, max_lists=2, out=None):
        """Posting lists from a top-m assignment: (offsets int64 [K + 1], items int32 [N * max_lists], total, mean lists
        per vector); list k is items[offsets[k]:offsets[k + 1]], ascending.  tau None selects 1 / K."""
        N, m = idx.shape
        if out is None:
            offsets = torch.empty(int(K) + 1 if K >= 0 else 1, dtype=torch.int64, device=idx.device)
            items = torch.empty(max(1, N * max(1, int(max_lists))), dtype=torch.int32, device=idx.device)
        else:
            offsets, items = out
        total, mean = ctypes.c_int64(0), ctypes.c_double(0.0)
        rc = lib.gmm_build_posting_lists(self._h, _dev(idx, torch.int32, (N, m), "idx"), _dev(resp, torch.float32, (N, m), "resp"),
                                         N, m, int(K), float(tau) if tau is not None else 0.0, int(max_lists),
                                         ctypes.c_void_p(offsets.data_ptr()), ctypes.c_void_p(items.data_ptr()),
                                         ctypes.byref(total), ctypes.byref(mean))
        self._check(rc)
        return offsets, items, int(total.value), float(mean.value)

    def gmm_score_samples(self, X, pi, mu, var, out=None):
        """Per-point log-density: (logp float32 [N], their float64 sum)."""
        N, D = X.shape
        K = mu.shape[0]
        logp = out if out is not None else torch.empty(N, dtype=torch.float32, device=X.device)
        ll = ctypes.c_double(0.0)
        rc = lib.gmm_score_samples(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K, _dev(pi, torch.float32, (K,), "pi"),
                                   _dev(mu, torch.float32, (K, D), "mu"), _dev(var, torch.float32, (K, D), "var"),
                                   _dev(logp, torch.float32, (N,), "logp"), ctypes.byref(ll))
        self._check(rc)
        return logp, float(ll.value)

    def gmm_fisher_vectors(self, X, offsets, pi, mu, var, out=None):
        """Fisher vectors of the groups of consecutive rows given by ``offsets`` (host int64 [G + 1]):
        (fv float32 [G, 2, K, D], total log-likelihood)."""
        N, D = X.shape
        K = mu.shape[0]
        offsets = np.ascontiguousarray(offsets, dtype=np.int64)
        if offsets.ndim != 1 or offsets.shape[0] < 2:
            raise ValueError("offsets must hold G + 1 >= 2 entries")
        G = offsets.shape[0] - 1
        fv = out if out is not None else torch.empty((G, 2, K, D), dtype=torch.float32, device=X.device)
        ll = ctypes.c_double(0.0)
        rc = lib.gmm_fisher_vectors(self._h, _dev(X, torch.float32, (N, D), "X"), N, _host(offsets, np.int64, (G + 1,), "offsets"),
                                    G, D, K, _dev(pi, torch.float32, (K,), "pi"), _dev(mu, torch.float32, (K, D), "mu"),
                                    _dev(var, torch.float32, (K, D), "var"), _dev(fv, torch.float32, (G, 2, K, D), "fv"),
                                    ctypes.byref(ll))
        self._check(rc)
        return fv, float(ll.value)

    def gmm_kmeans_step(self, X, centroids, out=None, work=None):
        """One Lloyd iteration: (assign int32 [N], new centroids float32 [K, D], counts int64 [K], inertia)."""
        N, D = X.shape
        K = centroids.shape[0]
        if out is None:
            assign = torch.empty(N, dtype=torch.int32, device=X.device)
            new = torch.empty((K, D), dtype=torch.float32, device=X.device)
            counts = torch.empty(K, dtype=torch.int64, device=X.device)
        else:
            assign, new, counts = out
        if work is None:
            work = torch.empty(2 * N, dtype=torch.int32, device=X.device)
        inertia = ctypes.c_double(0.0)
        rc = lib.gmm_kmeans_step(self._h, _dev(X, torch.float32, (N, D), "X"), N, D, K,
                                 _dev(centroids, torch.float32, (K, D), "centroids"), _dev(assign, torch.int32, (N,), "assign"),
                                 _dev(work, torch.int32, (2 * N,), "work"), _dev(new, torch.float32, (K, D), "centroids_out"),
                                 ctypes.c_void_p(counts.data_ptr()), ctypes.byref(inertia))
        self._check(rc)
        return assign, new, counts, float(inertia.value)
