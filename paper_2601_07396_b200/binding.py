"""Thin ctypes binding of ``libsvdcache.so``: same names as ``include/svdcache.h``,
argument marshalling only (tensor -> raw pointer, current stream -> void*).  Every step
of the path runs in the library's CUDA kernels; nothing here computes, and there is no
fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

F32, BF16 = 0, 1
_DTYPES = {torch.float32: F32, torch.bfloat16: BF16}

_HERE = os.path.dirname(os.path.abspath(__file__))
# SVDCACHE_LIBRARY names another build of the same library (e.g. one made with different
# compiler flags); by default the in-tree build next to this file is loaded.
LIB_PATH = os.environ.get("SVDCACHE_LIBRARY") or os.path.join(_HERE, "libsvdcache.so")
_lib = None

_vp, _i64, _ci, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
_szp = ctypes.POINTER(ctypes.c_size_t)

# name -> (restype, argtypes); mirrors include/svdcache.h declaration by declaration
SIGNATURES = {
    "svdcache_status_string": (ctypes.c_char_p, [_ci]),
    "svdcache_last_cuda_error": (ctypes.c_char_p, []),
    "svdcache_calibrate_workspace_bytes": (_ci, [_ci, _ci, _szp]),
    "svdcache_calibrate_begin": (_ci, [_ci, _ci, _vp, _sz, _vp]),
    "svdcache_calibrate_accumulate": (_ci, [_vp, _i64, _ci, _i64, _ci, _vp, _sz, _vp]),
    "svdcache_calibrate_finish": (_ci, [_ci, _ci, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "svdcache_calibrate": (_ci, [_vp, _i64, _ci, _i64, _ci, _ci, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "svdcache_calibrate_noalloc": (_ci, [_vp, _i64, _ci, _i64, _ci, _ci, _vp, _vp, _vp, _vp, _vp]),
    "svdcache_rank_for_energy": (_ci, [_vp, _ci, ctypes.c_double, ctypes.c_double, ctypes.POINTER(_ci)]),
    "svdcache_basis_bytes": (_ci, [_ci, _ci, _ci, _szp]),
    "svdcache_basis_layout": (_ci, [_ci, _ci, _ci, _szp, _szp, _szp, _szp]),
    "svdcache_basis_prepare": (_ci, [_vp, _ci, _ci, _ci, _vp, _sz, _vp]),
    "svdcache_state_bytes": (_ci, [_i64, _ci, _ci, _ci, _szp]),
    "svdcache_state_layout": (_ci, [_i64, _ci, _ci, _ci, _szp, _szp]),
    "svdcache_state_reset": (_ci, [_vp, _i64, _ci, _ci, _ci, _vp]),
    "svdcache_state_query": (_ci, [_vp, _vp, ctypes.POINTER(_i64), ctypes.POINTER(_ci)]),
    "svdcache_full_step": (_ci, [_vp, _i64, _vp, _vp, _vp, _i64, _ci, _ci, _ci, ctypes.c_float, _vp]),
    "svdcache_cached_step": (_ci, [_vp, _vp, _vp, _i64, _i64, _ci, _ci, _ci, _ci, _vp]),
    "svdcache_full_step_batched": (_ci, [_ci, _vp, _i64, _sz, _vp, _sz, _vp, _sz, _vp, _sz, _i64, _ci, _ci,
                                         _ci, ctypes.c_float, _vp]),
    "svdcache_cached_step_batched": (_ci, [_ci, _vp, _sz, _vp, _sz, _vp, _i64, _sz, _i64, _ci, _ci, _ci,
                                           _ci, _vp]),
    "svdcache_kernel_launches": (ctypes.c_uint64, []),
    "svdcache_set_path": (_ci, [_ci]),
    "svdcache_last_path": (_ci, []),
    "svdcache_selftest_wait_timeout": (_ci, [_vp, _i64, _vp]),
    "svdcache_full_step_ranked_batched": (_ci, [_ci, _vp, _i64, _sz, _vp, _sz, _vp, _sz, _vp, _sz, _i64, _ci,
                                                ctypes.POINTER(_ci), _ci, ctypes.c_float, _vp]),
    "svdcache_cached_step_ranked_batched": (_ci, [_ci, _vp, _sz, _vp, _sz, _vp, _i64, _sz, _i64, _ci,
                                                  ctypes.POINTER(_ci), _ci, _ci, _vp]),
    "svdcache_forecast_weights": (_ci, [_ci, _ci, _ci, _ci, ctypes.POINTER(ctypes.c_double)]),
    "svdcache_forecast_bytes": (_ci, [_i64, _ci, _szp]),
    "svdcache_cached_step_forecast_batched": (_ci, [_ci, _vp, _sz, _vp, _sz, _vp, _i64, _sz, _i64, _ci, _ci, _ci,
                                                    ctypes.POINTER(_vp), _sz, _ci, _ci, _ci, _ci, _vp, _sz, _vp]),
    "svdcache_full_step_residual_ema_batched": (_ci, [_ci, _vp, _i64, _sz, _vp, _sz, _vp, _sz, _vp, _sz, _i64, _ci,
                                                      _ci, _ci, ctypes.c_float, ctypes.c_float, _vp]),
    "svdcache_calibrate_gram_region": (_ci, [_ci, _szp, _szp]),
    "svdcache_basis_similarity": (_ci, [_vp, _vp, _vp, _vp, _ci, _ci, _vp, ctypes.POINTER(ctypes.c_double), _vp]),
    "svdcache_singular_values": (_ci, [_vp, _ci, _vp, _vp]),
    "svdcache_left_factors": (_ci, [_vp, _vp, _i64, _ci, _vp, _vp]),
}


class SvdCacheError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        text = lib().svdcache_status_string(code).decode()
        extra = ""
        if code == -7:
            extra = " [" + lib().svdcache_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {text} ({code}){extra}")


def lib():
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2601_07396_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != 0:
        raise SvdCacheError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensor expected")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dt(t_or_dtype) -> int:
    d = t_or_dtype.dtype if isinstance(t_or_dtype, torch.Tensor) else t_or_dtype
    return _DTYPES[d]


def _bytes_buffer(nbytes: int, device) -> torch.Tensor:
    # torch's caching allocator hands out 512-byte aligned blocks
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


# ------------------------------------------------------------------ size queries ---

def svdcache_calibrate_workspace_bytes(D: int, k: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().svdcache_calibrate_workspace_bytes(D, k, ctypes.byref(out)), "calibrate_workspace_bytes")
    return out.value


def svdcache_basis_bytes(D: int, k: int, dtype: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().svdcache_basis_bytes(D, k, dtype, ctypes.byref(out)), "basis_bytes")
    return out.value


def svdcache_basis_layout(D: int, k: int, dtype: int) -> Tuple[int, int, int, int]:
    o = [ctypes.c_size_t(0) for _ in range(4)]
    _check(lib().svdcache_basis_layout(D, k, dtype, *[ctypes.byref(x) for x in o]), "basis_layout")
    return tuple(x.value for x in o)


def svdcache_state_bytes(N: int, D: int, k: int, dtype: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().svdcache_state_bytes(N, D, k, dtype, ctypes.byref(out)), "state_bytes")
    return out.value


def svdcache_state_layout(N: int, D: int, k: int, dtype: int) -> Tuple[int, int]:
    a, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().svdcache_state_layout(N, D, k, dtype, ctypes.byref(a), ctypes.byref(b)), "state_layout")
    return a.value, b.value


# ------------------------------------------------------------------- calibration ---

def svdcache_calibrate_begin(D: int, k: int, workspace: torch.Tensor, stream=None) -> None:
    _check(lib().svdcache_calibrate_begin(D, k, _ptr(workspace), workspace.numel(), _stream(stream)),
           "calibrate_begin")


def svdcache_calibrate_accumulate(F: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    M, D = F.shape
    assert F.stride(1) == 1
    _check(lib().svdcache_calibrate_accumulate(_ptr(F), M, D, F.stride(0), _dt(F), _ptr(workspace),
                                               workspace.numel(), _stream(stream)), "calibrate_accumulate")


def svdcache_calibrate_finish(D: int, k: int, workspace: torch.Tensor, stream=None, strict: bool = True):
    """Returns (Vk [D x k] fp32, lambda [k] fp64, trace [1] fp64, info list) on the device."""
    dev = workspace.device
    Vk = torch.empty(D, k, dtype=torch.float32, device=dev)
    lam = torch.empty(k, dtype=torch.float64, device=dev)
    tr = torch.empty(1, dtype=torch.float64, device=dev)
    info = (ctypes.c_double * 4)()
    rc = lib().svdcache_calibrate_finish(D, k, _ptr(Vk), _ptr(lam), _ptr(tr), ctypes.cast(info, _vp),
                                         _ptr(workspace), workspace.numel(), _stream(stream))
    if rc != 0 and (strict or rc != -8):
        raise SvdCacheError(rc, "calibrate_finish")
    return Vk, lam, tr, list(info)


def svdcache_calibrate(Fstack: torch.Tensor, k: int, workspace: Optional[torch.Tensor] = None,
                       stream=None, strict: bool = True):
    """One-shot calibration of a device stack (M x D).  Returns (Vk, lambda, trace, info)."""
    M, D = Fstack.shape
    assert Fstack.stride(1) == 1
    if workspace is None:
        workspace = _bytes_buffer(svdcache_calibrate_workspace_bytes(D, k), Fstack.device)
    dev = Fstack.device
    Vk = torch.empty(D, k, dtype=torch.float32, device=dev)
    lam = torch.empty(k, dtype=torch.float64, device=dev)
    tr = torch.empty(1, dtype=torch.float64, device=dev)
    info = (ctypes.c_double * 4)()
    rc = lib().svdcache_calibrate(_ptr(Fstack), M, D, Fstack.stride(0), _dt(Fstack), k, _ptr(Vk), _ptr(lam),
                                  _ptr(tr), ctypes.cast(info, _vp), _ptr(workspace), workspace.numel(),
                                  _stream(stream))
    if rc != 0 and (strict or rc != -8):
        raise SvdCacheError(rc, "calibrate")
    return Vk, lam, tr, list(info)


BUILTIN_SCRATCH_BYTES = 4 << 20


def svdcache_calibrate_noalloc(Fstack: torch.Tensor, k: int, Vk: torch.Tensor, lam: torch.Tensor,
                               tr: torch.Tensor, stream=None, strict: bool = True):
    """Calibration on the library's built-in scratch, for callers that may not allocate
    device memory: the outputs (Vk [D x k] fp32, lam [k] fp64, tr [1] fp64) are passed in,
    and neither this wrapper nor the call behind it allocates anything on the device.
    Returns the info list."""
    M, D = Fstack.shape
    assert Fstack.stride(1) == 1 and Vk.shape == (D, k) and Vk.dtype == torch.float32 and Vk.is_contiguous()
    info = (ctypes.c_double * 4)()
    rc = lib().svdcache_calibrate_noalloc(_ptr(Fstack), M, D, Fstack.stride(0), _dt(Fstack), k, _ptr(Vk),
                                          _ptr(lam), _ptr(tr), ctypes.cast(info, _vp), _stream(stream))
    if rc != 0 and (strict or rc != -8):
        raise SvdCacheError(rc, "calibrate_noalloc")
    return list(info)


def svdcache_rank_for_energy(lam, trace: float, tau: float) -> int:
    arr = (ctypes.c_double * len(lam))(*[float(x) for x in lam])
    out = ctypes.c_int(0)
    _check(lib().svdcache_rank_for_energy(ctypes.cast(arr, _vp), len(lam), float(trace), float(tau),
                                          ctypes.byref(out)), "rank_for_energy")
    return out.value


# ------------------------------------------------------------------ basis, state ---

def svdcache_basis_prepare(Vk: torch.Tensor, dtype: int, basis: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    D, k = Vk.shape
    assert Vk.dtype == torch.float32 and Vk.is_contiguous()
    if basis is None:
        basis = _bytes_buffer(svdcache_basis_bytes(D, k, dtype), Vk.device)
    _check(lib().svdcache_basis_prepare(_ptr(Vk), D, k, dtype, _ptr(basis), basis.numel(), _stream(stream)),
           "basis_prepare")
    return basis


def svdcache_state_reset(state: torch.Tensor, N: int, D: int, k: int, dtype: int, stream=None) -> None:
    _check(lib().svdcache_state_reset(_ptr(state), N, D, k, dtype, _stream(stream)), "state_reset")


def svdcache_state_query(state: torch.Tensor, stream=None) -> Tuple[int, int]:
    steps, status = ctypes.c_int64(0), ctypes.c_int(0)
    _check(lib().svdcache_state_query(_ptr(state), _stream(stream), ctypes.byref(steps), ctypes.byref(status)),
           "state_query")
    return steps.value, status.value


# ------------------------------------------------------------------------- steps ---

def svdcache_full_step(F: torch.Tensor, basis: torch.Tensor, state: torch.Tensor, k: int, beta: float,
                       C_out: Optional[torch.Tensor] = None, stream=None) -> None:
    N, D = F.shape
    assert F.stride(1) == 1
    _check(lib().svdcache_full_step(_ptr(F), F.stride(0), _ptr(basis), _ptr(state), _ptr(C_out), N, D, k,
                                    _dt(F), float(beta), _stream(stream)), "full_step")


def svdcache_cached_step(state: torch.Tensor, basis: torch.Tensor, Fhat: torch.Tensor, k: int,
                         steps_since_full: int = 1, stream=None) -> None:
    N, D = Fhat.shape
    assert Fhat.stride(1) == 1
    _check(lib().svdcache_cached_step(_ptr(state), _ptr(basis), _ptr(Fhat), Fhat.stride(0), N, D, k,
                                      _dt(Fhat), int(steps_since_full), _stream(stream)), "cached_step")


def svdcache_full_step_batched(F: torch.Tensor, basis: torch.Tensor, state: torch.Tensor, k: int,
                               beta: float, C_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """F: [blocks, N, D]; basis, state: [blocks, bytes] uint8; C_out: [blocks, N, k] or None."""
    nb, N, D = F.shape
    assert F.stride(2) == 1
    eb = F.element_size()
    _check(lib().svdcache_full_step_batched(
        nb, _ptr(F), F.stride(1), F.stride(0) * eb, _ptr(basis), basis.stride(0), _ptr(state),
        state.stride(0), _ptr(C_out), 0 if C_out is None else C_out.stride(0) * 4, N, D, k, _dt(F),
        float(beta), _stream(stream)), "full_step_batched")


def svdcache_cached_step_batched(state: torch.Tensor, basis: torch.Tensor, Fhat: torch.Tensor, k: int,
                                 steps_since_full: int = 1, stream=None) -> None:
    nb, N, D = Fhat.shape
    assert Fhat.stride(2) == 1
    eb = Fhat.element_size()
    _check(lib().svdcache_cached_step_batched(
        nb, _ptr(state), state.stride(0), _ptr(basis), basis.stride(0), _ptr(Fhat), Fhat.stride(1),
        Fhat.stride(0) * eb, N, D, k, _dt(Fhat), int(steps_since_full), _stream(stream)), "cached_step_batched")


def svdcache_kernel_launches() -> int:
    return int(lib().svdcache_kernel_launches())


def svdcache_set_path(path: int) -> int:
    return int(lib().svdcache_set_path(path))


def svdcache_last_path() -> int:
    return int(lib().svdcache_last_path())


def svdcache_selftest_wait_timeout(state: torch.Tensor, limit_cycles: int, stream=None) -> None:
    _check(lib().svdcache_selftest_wait_timeout(_ptr(state), int(limit_cycles), _stream(stream)), "selftest_wait_timeout")


PREDICT_EMA, PREDICT_TAYLOR, PREDICT_NEWTON = 0, 1, 2


def svdcache_forecast_weights(predictor: int, order: int, steps_since_full: int, interval: int):
    w = (ctypes.c_double * (order + 1))()
    _check(lib().svdcache_forecast_weights(predictor, order, steps_since_full, interval, w), "forecast_weights")
    return list(w)


def svdcache_forecast_bytes(N: int, k: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().svdcache_forecast_bytes(N, k, ctypes.byref(out)), "forecast_bytes")
    return int(out.value)


def svdcache_cached_step_forecast_batched(state: torch.Tensor, basis: torch.Tensor, Fhat: torch.Tensor, k: int, history,
                                  predictor: int, steps_since_full: int, interval: int, forecast=None, stream=None):
    """Cached step with the coefficients forecast from `history` (list of N x k fp32 device tensors --
    or [blocks, N, k] for a batched Fhat [blocks, N, D] -- newest first; its length - 1 is the order).
    Returns the forecast buffer (allocated here unless given)."""
    batched = Fhat.dim() == 3
    nb = Fhat.shape[0] if batched else 1
    N, D = Fhat.shape[-2:]
    assert Fhat.stride(-1) == 1
    order = len(history) - 1
    fbytes = svdcache_forecast_bytes(N, k)
    if forecast is None:
        forecast = torch.empty(nb, fbytes, dtype=torch.uint8, device=Fhat.device) if batched else _bytes_buffer(fbytes, Fhat.device)
    ptrs = (_vp * (order + 1))(*[_ptr(h) for h in history])
    eb = Fhat.element_size()
    _check(lib().svdcache_cached_step_forecast_batched(
        nb, _ptr(state), state.stride(0) if batched else 0, _ptr(basis), basis.stride(0) if batched else 0, _ptr(Fhat),
        Fhat.stride(-2), Fhat.stride(0) * eb if batched else 0, N, D, k, _dt(Fhat), ptrs,
        history[0].stride(0) * 4 if batched else 0, predictor, order, int(steps_since_full), int(interval), _ptr(forecast),
        forecast.stride(0) if batched else 0, _stream(stream)), "cached_step_forecast")
    return forecast


def svdcache_full_step_residual_ema_batched(F: torch.Tensor, basis: torch.Tensor, state: torch.Tensor, k: int, beta: float,
                                    beta_r: float, C_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """Full step whose stored residual is an EMA of the residuals (ablation); F is [N, D] or [blocks, N, D]."""
    batched = F.dim() == 3
    nb = F.shape[0] if batched else 1
    N, D = F.shape[-2:]
    eb = F.element_size()
    _check(lib().svdcache_full_step_residual_ema_batched(
        nb, _ptr(F), F.stride(-2), F.stride(0) * eb if batched else 0, _ptr(basis), basis.stride(0) if batched else 0,
        _ptr(state), state.stride(0) if batched else 0, _ptr(C_out) if C_out is not None else None,
        C_out.stride(0) * 4 if (batched and C_out is not None) else 0, N, D, k, _dt(F), float(beta), float(beta_r),
        _stream(stream)), "full_step_residual_ema")


def svdcache_full_step_ranked_batched(F: torch.Tensor, bases: torch.Tensor, states: torch.Tensor, ranks, beta: float,
                              C_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """Batched full step over blocks of different rank: F [blocks, N, D], bases / states [blocks, bytes]
    (each block's buffer laid out for its own rank), C_out [blocks, N, kmax] (row b*... holds N x k_b dense)."""
    nb, N, D = F.shape
    arr = (_ci * nb)(*[int(r) for r in ranks])
    _check(lib().svdcache_full_step_ranked_batched(
        nb, _ptr(F), F.stride(1), F.stride(0) * F.element_size(), _ptr(bases), bases.stride(0), _ptr(states),
        states.stride(0), _ptr(C_out) if C_out is not None else None, C_out.stride(0) * 4 if C_out is not None else 0,
        N, D, arr, _dt(F), float(beta), _stream(stream)), "full_step_ranked")


def svdcache_cached_step_ranked_batched(states: torch.Tensor, bases: torch.Tensor, Fhat: torch.Tensor, ranks,
                                steps_since_full: int = 1, stream=None) -> None:
    nb, N, D = Fhat.shape
    arr = (_ci * nb)(*[int(r) for r in ranks])
    _check(lib().svdcache_cached_step_ranked_batched(
        nb, _ptr(states), states.stride(0), _ptr(bases), bases.stride(0), _ptr(Fhat), Fhat.stride(1),
        Fhat.stride(0) * Fhat.element_size(), N, D, arr, _dt(Fhat), int(steps_since_full), _stream(stream)),
        "cached_step_ranked")


def svdcache_calibrate_gram_region(D: int):
    off, nbytes = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().svdcache_calibrate_gram_region(D, ctypes.byref(off), ctypes.byref(nbytes)), "calibrate_gram_region")
    return int(off.value), int(nbytes.value)


def svdcache_basis_similarity(VkA: torch.Tensor, lamA: torch.Tensor, VkB: torch.Tensor, lamB: torch.Tensor, stream=None):
    """(similarity of the singular values, mean similarity of the right singular vectors, per-column |cos|)."""
    D, k = VkA.shape
    assert VkB.shape == (D, k) and VkA.is_contiguous() and VkB.is_contiguous()
    cols = torch.empty(k, dtype=torch.float64, device=VkA.device)
    out = (ctypes.c_double * 2)()
    _check(lib().svdcache_basis_similarity(_ptr(VkA), _ptr(lamA), _ptr(VkB), _ptr(lamB), D, k, _ptr(cols), out,
                                           _stream(stream)), "basis_similarity")
    return float(out[0]), float(out[1]), cols


def svdcache_singular_values(lam: torch.Tensor, stream=None) -> torch.Tensor:
    sigma = torch.empty_like(lam)
    _check(lib().svdcache_singular_values(_ptr(lam), lam.numel(), _ptr(sigma), _stream(stream)), "singular_values")
    return sigma


def svdcache_left_factors(C: torch.Tensor, sigma: torch.Tensor, stream=None) -> torch.Tensor:
    N, k = C.shape
    assert C.is_contiguous() and C.dtype == torch.float32 and sigma.dtype == torch.float64
    U = torch.empty_like(C)
    _check(lib().svdcache_left_factors(_ptr(C), _ptr(sigma), N, k, _ptr(U), _stream(stream)), "left_factors")
    return U


# ---------------------------------------------------------- views for tests/tools ---

def new_state(N: int, D: int, k: int, dtype: int, device="cuda", blocks: int = 0) -> torch.Tensor:
    """Allocate (torch) and reset a state buffer; ``blocks`` > 0 gives [blocks, bytes]."""
    nbytes = svdcache_state_bytes(N, D, k, dtype)
    if blocks:
        st = torch.empty(blocks, nbytes, dtype=torch.uint8, device=device)
        for b in range(blocks):
            svdcache_state_reset(st[b], N, D, k, dtype)
        return st
    st = _bytes_buffer(nbytes, device)
    svdcache_state_reset(st, N, D, k, dtype)
    return st


def state_views(state: torch.Tensor, N: int, D: int, k: int, dtype: int):
    """(Chat [N x k] fp32, R [N x D]) views into one block's state buffer."""
    co, ro = svdcache_state_layout(N, D, k, dtype)
    tdt = torch.float32 if dtype == F32 else torch.bfloat16
    eb = 4 if dtype == F32 else 2
    chat = state[co:co + N * k * 4].view(torch.float32).view(N, k)
    r = state[ro:ro + N * D * eb].view(tdt).view(N, D)
    return chat, r


def basis_views(basis: torch.Tensor, D: int, k: int, dtype: int):
    """(V fp32, V^T fp32, V bf16 | None, V^T bf16 | None) views into a basis buffer."""
    a, b, c, d = svdcache_basis_layout(D, k, dtype)
    v32 = basis[a:a + D * k * 4].view(torch.float32).view(D, k)
    vt32 = basis[b:b + D * k * 4].view(torch.float32).view(k, D)
    if dtype == BF16:
        v16 = basis[c:c + D * k * 2].view(torch.bfloat16).view(D, k)
        vt16 = basis[d:d + D * k * 2].view(torch.bfloat16).view(k, D)
        return v32, vt32, v16, vt16
    return v32, vt32, None, None
