"""ctypes front end of the float64 CPU oracle (``gmm_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline / reference legs call this;
the product package never imports it.  It compiles the C++ file with g++ on first use (a couple of seconds), in two
flavours chosen from the host's CPU flags, so a library built on one machine is never run on a CPU that lacks its
instructions.  No arithmetic of the method lives in this file: it only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gmm_oracle.cpp"
_LIB = None


def _cpu_has(*flags: str) -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    have = set(line.split(":", 1)[1].split())
                    return all(fl in have for fl in flags)
    except OSError:
        pass
    return False


def _flavours():
    return {"v3": ["-march=x86-64-v3"], "base": []}


def lib_path(flavour: str) -> Path:
    return _HERE / f"libgmm_oracle_{flavour}.so"


def build(force: bool = False) -> None:
    """Compile every flavour of the oracle library next to its source."""
    for flavour, march in _flavours().items():
        out = lib_path(flavour)
        if not force and out.exists() and out.stat().st_mtime >= _SRC.stat().st_mtime:
            continue
        cmd = ["g++", "-O3", "-std=c++17", "-fopenmp", "-fPIC", "-shared", *march, str(_SRC), "-o", str(out)]
        subprocess.run(cmd, check=True)


def _load():
    global _LIB
    if _LIB is not None:
        return _LIB
    build()
    flavour = "v3" if _cpu_has("avx2", "fma", "bmi2") else "base"
    lib = ctypes.CDLL(str(lib_path(flavour)))
    c_fp = ctypes.POINTER(ctypes.c_float)
    c_dp = ctypes.POINTER(ctypes.c_double)
    c_ip = ctypes.POINTER(ctypes.c_int32)
    i64, ci = ctypes.c_int64, ctypes.c_int
    sig = {
        "oracle_num_threads": ([], ci),
        "oracle_log_joint": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, c_dp], ci),
        "oracle_responsibilities": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, c_dp, c_dp], ci),
        "oracle_brute_force": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, c_dp, c_dp], ci),
        "oracle_em_step": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, c_dp, c_dp, c_dp, c_dp, ci], ci),
        "oracle_finalize_moments": ([i64, ci, ci, c_dp, c_dp, c_dp, ctypes.c_double, c_dp, c_dp, c_dp], ci),
        "oracle_em_iteration": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, ctypes.c_double, c_dp, c_dp, c_dp, ci], ci),
        "oracle_em_iteration_isotropic": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, ctypes.c_double, c_dp, ci], ci),
        "oracle_fit": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, ci, ctypes.c_double, ctypes.c_double, c_dp,
                        ctypes.POINTER(ci), c_dp, ci], ci),
        "oracle_topm": ([c_fp, i64, ci, ci, c_dp, c_dp, c_dp, ci, c_ip, c_dp, c_dp, ci], ci),
    }
    for name, (argtypes, restype) in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = restype
    _LIB = lib
    return lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _fp(a):
    return _p(a, ctypes.c_float)


def _dp(a):
    return _p(a, ctypes.c_double) if a is not None else None


def _shapes(X, mu):
    X = _f32(X)
    if X.ndim != 2:
        raise ValueError("X must be [N, D]")
    mu = _f64(mu)
    if mu.ndim != 2 or mu.shape[1] != X.shape[1]:
        raise ValueError("mu must be [K, D]")
    return X, mu, X.shape[0], X.shape[1], mu.shape[0]


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def log_joint(X, pi, mu, var):
    """ell[i, k] = log(pi_k N(x_i | mu_k, diag var_k)) as float64 [N, K]."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, var = _f64(pi), _f64(var)
    out = np.empty((N, K), np.float64)
    _check(_load().oracle_log_joint(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), _dp(out)), "oracle_log_joint")
    return out


def responsibilities(X, pi, mu, var):
    """(R [N, K], logZ [N]) by the log-space definition."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, var = _f64(pi), _f64(var)
    R = np.empty((N, K), np.float64)
    lz = np.empty(N, np.float64)
    _check(_load().oracle_responsibilities(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), _dp(R), _dp(lz)),
           "oracle_responsibilities")
    return R, lz


def brute_force(X, pi, mu, var):
    """(R [N, K], p [N]) from linear-space products of univariate pdfs; tiny inputs only."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, var = _f64(pi), _f64(var)
    R = np.empty((N, K), np.float64)
    p = np.empty(N, np.float64)
    _check(_load().oracle_brute_force(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), _dp(R), _dp(p)),
           "oracle_brute_force")
    return R, p


def em_step(X, pi, mu, var, nthreads: int = 0):
    """(Nk [K], S1 [K, D], S2 [K, D], loglik) under the given parameters."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, var = _f64(pi), _f64(var)
    Nk = np.empty(K, np.float64)
    S1 = np.empty((K, D), np.float64)
    S2 = np.empty((K, D), np.float64)
    L = ctypes.c_double(0.0)
    rc = _load().oracle_em_step(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), _dp(Nk), _dp(S1), _dp(S2),
                                ctypes.byref(L), nthreads)
    _check(rc, "oracle_em_step")
    return Nk, S1, S2, L.value


def finalize_moments(N, Nk, S1, S2, var_floor, mu_old, var_old):
    """(pi, mu, var) from the moments: mu = S1/Nk, var = max(S2/Nk - mu^2, floor); empty components keep mu, var."""
    Nk, S1, S2 = _f64(Nk), _f64(S1), _f64(S2)
    K, D = S1.shape
    pi = np.empty(K, np.float64)
    mu = _f64(mu_old).copy()
    var = _f64(var_old).copy()
    _check(_load().oracle_finalize_moments(int(N), D, K, _dp(Nk), _dp(S1), _dp(S2), float(var_floor), _dp(pi),
                                           _dp(mu), _dp(var)), "oracle_finalize_moments")
    return pi, mu, var


def em_iteration(X, pi, mu, var, var_floor: float = 0.0, nthreads: int = 0):
    """One EM iteration by the definition (centred variance with the new mean).

    Returns (pi_new, mu_new, var_new, loglik_under_old_params, Nk, S1)."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, mu, var = _f64(pi).copy(), mu.copy(), _f64(var).copy()
    Nk = np.empty(K, np.float64)
    S1 = np.empty((K, D), np.float64)
    L = ctypes.c_double(0.0)
    rc = _load().oracle_em_iteration(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), float(var_floor), ctypes.byref(L),
                                     _dp(Nk), _dp(S1), nthreads)
    _check(rc, "oracle_em_iteration")
    return pi, mu, var, L.value, Nk, S1


def em_iteration_isotropic(X, pi, mu, var, var_floor: float = 0.0, nthreads: int = 0):
    """One EM iteration of the paper's isotropic model (Eq. 1-3 as printed).  ``var`` is [K, D] with each row constant.

    Returns (pi_new, mu_new, var_new [K, D] with constant rows, loglik_under_old_params)."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, mu, var = _f64(pi).copy(), mu.copy(), _f64(var).copy()
    L = ctypes.c_double(0.0)
    rc = _load().oracle_em_iteration_isotropic(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), float(var_floor),
                                               ctypes.byref(L), nthreads)
    _check(rc, "oracle_em_iteration_isotropic")
    return pi, mu, var, L.value


def fit(X, pi, mu, var, iters: int, var_floor: float = 0.0, tol: float = 0.0, keep_params: bool = False,
        nthreads: int = 0):
    """Run EM.  Returns dict(pi, mu, var, trace[iters_done], iters_done, params=[(pi, mu, var) per iteration + final])."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, mu, var = _f64(pi).copy(), mu.copy(), _f64(var).copy()
    trace = np.zeros(iters, np.float64)
    done = ctypes.c_int(0)
    P = K + 2 * K * D
    ptrace = np.zeros((iters + 1, P), np.float64) if keep_params else None
    rc = _load().oracle_fit(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), int(iters), float(var_floor), float(tol),
                            _dp(trace), ctypes.byref(done), _dp(ptrace), nthreads)
    _check(rc, "oracle_fit")
    out = dict(pi=pi, mu=mu, var=var, trace=trace[: done.value].copy(), iters_done=done.value)
    if keep_params:
        out["params"] = [
            (ptrace[t, :K].copy(), ptrace[t, K:K + K * D].reshape(K, D).copy(),
             ptrace[t, K + K * D:].reshape(K, D).copy())
            for t in range(done.value + 1)
        ]
    return out


def topm(X, pi, mu, var, m: int, nthreads: int = 0):
    """(idx int32 [N, m], resp float64 [N, m], next_resp float64 [N]): the m largest responsibilities per point,
    descending, ties to the smaller component index; next_resp is the (m+1)-th largest (0 when m == K)."""
    X, mu, N, D, K = _shapes(X, mu)
    pi, var = _f64(pi), _f64(var)
    idx = np.empty((N, m), np.int32)
    resp = np.empty((N, m), np.float64)
    nxt = np.empty(N, np.float64)
    rc = _load().oracle_topm(_fp(X), N, D, K, _dp(pi), _dp(mu), _dp(var), int(m), _p(idx, ctypes.c_int32), _dp(resp),
                             _dp(nxt), nthreads)
    _check(rc, "oracle_topm")
    return idx, resp, nxt
