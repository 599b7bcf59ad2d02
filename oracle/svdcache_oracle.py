"""ctypes front-end of the fp64 CPU oracle (``svdcache_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this module.  It shares nothing with the CUDA library and never imports
it.  Arguments and results are numpy float64 arrays, row-major.

The shared object is compiled with gcc on first use (and again when the C file is newer).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "svdcache_oracle.c")
_LIB = os.path.join(_HERE, "libsvdcache_oracle.so")
_lock = threading.Lock()
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object beside it; returns its path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i64, ci, cd = ctypes.c_int64, ctypes.c_int, ctypes.c_double
            lib.oracle_gram.argtypes = [_dp, i64, ci, _dp]
            lib.oracle_gram.restype = None
            lib.oracle_eigh_desc.argtypes = [_dp, ci, _dp, _dp]
            lib.oracle_eigh_desc.restype = ci
            lib.oracle_calibrate.argtypes = [_dp, i64, ci, ci, _dp, _dp, _dp, _dp]
            lib.oracle_calibrate.restype = ci
            lib.oracle_jacobi_svd.argtypes = [_dp, ci, ci, _dp, _dp]
            lib.oracle_jacobi_svd.restype = ci
            lib.oracle_rank_for_energy.argtypes = [_dp, ci, cd, cd]
            lib.oracle_rank_for_energy.restype = ci
            lib.oracle_full_step.argtypes = [_dp, i64, ci, _dp, ci, cd, ci, _dp, _dp, _dp]
            lib.oracle_full_step.restype = None
            lib.oracle_cached_step.argtypes = [_dp, _dp, _dp, i64, ci, ci, _dp]
            lib.oracle_cached_step.restype = None
            lib.oracle_full_step_residual_ema.argtypes = [_dp, i64, ci, _dp, ci, cd, cd, ci, _dp, _dp, _dp]
            lib.oracle_full_step_residual_ema.restype = None
            lib.oracle_forecast.argtypes = [ctypes.POINTER(_dp), ci, i64, cd, ci, _dp]
            lib.oracle_forecast.restype = None
            lib.oracle_left_factors.argtypes = [_dp, _dp, i64, ci, _dp]
            lib.oracle_left_factors.restype = None
            lib.oracle_threads.restype = ci
            lib.oracle_set_threads.argtypes = [ci]
            _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


def threads() -> int:
    return int(_load().oracle_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def gram(F) -> np.ndarray:
    """G = F^T F of a row-stack F (M x D); Eq. 4 through sigma_i^2 = eig_i(G)."""
    F = _f64(F)
    M, D = F.shape
    G = np.empty((D, D))
    _load().oracle_gram(_p(F), M, D, _p(G))
    return G


def eigh_desc(A):
    """Eigenvalues (descending) and eigenvectors (columns) of a symmetric matrix."""
    A = _f64(A).copy()
    n = A.shape[0]
    w = np.empty(n)
    Z = np.empty((n, n))
    rc = _load().oracle_eigh_desc(_p(A), n, _p(w), _p(Z))
    if rc != 0:
        raise RuntimeError("oracle_eigh_desc: QR sweeps did not converge")
    return w, Z


def calibrate(Fstack, k: int, all_eigenvalues: bool = False):
    """Top-k right singular basis of the stack: (V_k [D x k], lambda [k], trace)."""
    F = _f64(Fstack)
    M, D = F.shape
    if not (1 <= k <= D):
        raise ValueError("need 1 <= k <= D")
    Vk = np.empty((D, k))
    lam = np.empty(k)
    tr = ctypes.c_double(0.0)
    lam_all = np.empty(D) if all_eigenvalues else None
    rc = _load().oracle_calibrate(_p(F), M, D, k, _p(Vk), _p(lam), ctypes.byref(tr),
                                  _p(lam_all) if all_eigenvalues else None)
    if rc != 0:
        raise RuntimeError("oracle_calibrate: eigen-solver did not converge")
    if all_eigenvalues:
        return Vk, lam, tr.value, lam_all
    return Vk, lam, tr.value


def jacobi_svd(A):
    """One-sided Jacobi SVD: (sigma [n] descending, V [n x n]) of A (m x n)."""
    A = _f64(A)
    m, n = A.shape
    s = np.empty(n)
    V = np.empty((n, n))
    _load().oracle_jacobi_svd(_p(A), m, n, _p(s), _p(V))
    return s, V


def rank_for_energy(lam, trace: float, tau: float) -> int:
    """Smallest k with sum_{i<=k} lambda_i / trace >= tau (Eq. 6)."""
    lam = _f64(lam)
    return int(_load().oracle_rank_for_energy(_p(lam), lam.shape[0], float(trace), float(tau)))


def full_step(F, Vk, beta: float, Chat_prev=None):
    """One full step.  Returns (C, R, Chat).  ``Chat_prev is None`` marks the first one."""
    F = _f64(F)
    Vk = _f64(Vk)
    N, D = F.shape
    k = Vk.shape[1]
    assert Vk.shape[0] == D
    first = Chat_prev is None
    Chat = np.zeros((N, k)) if first else _f64(Chat_prev).copy()
    assert Chat.shape == (N, k)
    R = np.empty((N, D))
    C = np.empty((N, k))
    _load().oracle_full_step(_p(F), N, D, _p(Vk), k, float(beta), int(first), _p(Chat), _p(R), _p(C))
    return C, R, Chat


def cached_step(Chat, Vk, R) -> np.ndarray:
    """Fhat = Chat V_k^T + R."""
    Chat = _f64(Chat)
    Vk = _f64(Vk)
    R = _f64(R)
    N, D = R.shape
    k = Vk.shape[1]
    assert Chat.shape == (N, k) and Vk.shape[0] == D
    Fhat = np.empty((N, D))
    _load().oracle_cached_step(_p(Chat), _p(Vk), _p(R), N, D, k, _p(Fhat))
    return Fhat


def full_step_residual_ema(F, Vk, beta: float, beta_r: float, Chat_prev=None, Rhat_prev=None):
    """Full step whose stored residual is an EMA of the residuals (ablation, Fig. 4(c)).
    Returns (C, Rhat, Chat); ``Chat_prev is None`` marks the first one."""
    F = _f64(F)
    Vk = _f64(Vk)
    N, D = F.shape
    k = Vk.shape[1]
    first = Chat_prev is None
    Chat = np.zeros((N, k)) if first else _f64(Chat_prev).copy()
    Rhat = np.zeros((N, D)) if first else _f64(Rhat_prev).copy()
    C = np.empty((N, k))
    _load().oracle_full_step_residual_ema(_p(F), N, D, _p(Vk), k, float(beta), float(beta_r), int(first),
                                          _p(Chat), _p(Rhat), _p(C))
    return C, Rhat, Chat


FORECAST_KINDS = {"taylor": 1, "newton": 2}


def forecast(history, u: float, kind: str = "taylor") -> np.ndarray:
    """Forecast of the coefficients ``u`` intervals past the newest full step from the list
    ``history`` (newest first; its length - 1 is the order)."""
    hist = [_f64(h) for h in history]
    order = len(hist) - 1
    if not 0 <= order <= 7:
        raise ValueError("order must be in 0..7")
    n = hist[0].size
    assert all(h.shape == hist[0].shape for h in hist)
    ptrs = (_dp * (order + 1))(*[_p(h) for h in hist])
    out = np.empty_like(hist[0])
    _load().oracle_forecast(ptrs, order, n, float(u), FORECAST_KINDS[kind], _p(out))
    return out


def left_factors(C, sigma) -> np.ndarray:
    """U = C diag(sigma)^-1 (Eq. 8)."""
    C = _f64(C)
    sigma = _f64(sigma)
    N, k = C.shape
    U = np.empty((N, k))
    _load().oracle_left_factors(_p(C), _p(sigma), N, k, _p(U))
    return U


def basis_similarity(VA, lamA, VB, lamB):
    """Stability of a decomposition across two calibrations (Fig. 1(b)): similarity = cosine
    similarity x magnitude similarity (smaller norm / larger norm).  Returns (that of the singular
    values sigma = sqrt(lambda), the mean over the columns of that of the right singular vectors,
    the per-column values).  Singular vectors are sign-free, so their cosine enters in magnitude."""
    VA, VB = _f64(VA), _f64(VB)
    sa, sb = np.sqrt(np.maximum(_f64(lamA), 0.0)), np.sqrt(np.maximum(_f64(lamB), 0.0))

    def sim(a, b, signed=True):
        na, nb = np.linalg.norm(a), np.linalg.norm(b)
        if na == 0.0 or nb == 0.0:
            return 0.0
        c = float(a @ b) / (na * nb)
        return (c if signed else abs(c)) * min(na, nb) / max(na, nb)

    cols = np.array([sim(VA[:, j], VB[:, j], signed=False) for j in range(VA.shape[1])])
    return sim(sa, sb), float(cols.mean()), cols
