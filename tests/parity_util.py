"""Helpers shared by the GPU parity tests: error measures, tolerances, and a driver that
plays a schedule of full and cached steps through the C ABI and through the oracle on
the same inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import svdcache_oracle as oracle
from paper_2601_07396_b200 import binding as sc

# Tolerances of the comparison with the fp64 oracle, per output array (C, Chat, R, Fhat):
#   fp32 I/O: relative Frobenius error <= 1e-5
#   bf16 I/O: relative Frobenius error <= 5e-3 and max-abs error <= 2e-2 * rms(F) (one bf16 ulp of
#             the reference value where that is larger: see check_close)
TOL = {sc.F32: dict(rel=1e-5, maxabs=None), sc.BF16: dict(rel=5e-3, maxabs=2e-2)}


def rel_fro(x: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref)
    num = np.linalg.norm(x.astype(np.float64) - ref)
    return float(num / den) if den > 0 else float(num)


def check_close(name, got, ref, dtype, rms_f, coeff=0):
    """Assert `got` (torch tensor or ndarray) against the oracle's `ref`; `coeff` = D for the
    fp32 coefficient arrays (see below), 0 for arrays in the I/O dtype."""
    if isinstance(got, torch.Tensor):
        got = got.detach().double().cpu().numpy()
    tol = TOL[dtype]
    rel = rel_fro(got, ref)
    # Coefficient arrays (C, Chat) are fp32 in both modes and never rounded to bf16.  `coeff` is
    # the width D they were reduced over: bf16 products are exact in fp32, and the tensor cores
    # truncate the fp32 running sum once per 16 columns, a one-sided error of at most
    # 2^-24 * D / 4 = 4e-9 * D relative (D = 1024: 1.3e-6 measured; D = 8192: 1.8e-5), so the
    # bound is the fp32 one up to D = 2500 and 4e-9 * D beyond; fp32 I/O accumulates in fp64.
    bound = (1e-5 if dtype == sc.F32 else max(1e-5, 4e-9 * float(coeff))) if coeff else tol["rel"]
    assert rel <= bound, f"{name}: relative Frobenius error {rel:.3e} > {bound:.1e}"
    if tol["maxabs"] is not None:
        # Element-wise bound of the bf16 mode: 2e-2 * rms(F) -- or one bf16 ulp of the reference
        # value where that is larger.  An output stored in bf16 is off by up to half an ulp
        # (2^-9 |x|) however it was computed, which passes 2e-2 * rms(F) once |x| > 10 rms(F);
        # among the 1e8 elements sampled at the full FLUX size a few are that large.
        err = np.abs(got - ref)
        ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7.0)   # bf16: 8 significant bits
        bound_el = np.maximum(tol["maxabs"] * rms_f, ulp)
        worst = int(np.argmax(err - bound_el))
        assert (err <= bound_el).all(), (f"{name}: element error {err.flat[worst]:.3e} > "
                                        f"max({tol['maxabs']}*rms(F)={tol['maxabs'] * rms_f:.3e}, ulp(ref)={ulp.flat[worst]:.3e})")
    return rel


def basis_as_consumed(basis: torch.Tensor, D: int, k: int, dtype: int) -> np.ndarray:
    """V_k exactly as the kernels multiply with it (fp32 copy, or the bf16-rounded copy)."""
    v32, _, v16, _ = sc.basis_views(basis, D, k, dtype)
    v = v32 if dtype == sc.F32 else v16
    return v.double().cpu().numpy()


def orthonormal_basis(D: int, k: int, seed: int, device="cuda") -> torch.Tensor:
    g = torch.Generator().manual_seed(seed)
    Q, _ = torch.linalg.qr(torch.randn(D, k, generator=g, dtype=torch.float64))
    return Q.float().contiguous().to(device)


class OracleTrack:
    """The oracle's state for a set of rows of one block (fp64, never rounded)."""

    def __init__(self, V: np.ndarray, beta: float):
        self.V = V
        self.beta = float(np.float32(beta))
        self.chat = None
        self.R = None
        self.C = None

    def full(self, F_rows: np.ndarray):
        self.C, self.R, self.chat = oracle.full_step(F_rows, self.V, self.beta, self.chat)

    def cached(self) -> np.ndarray:
        return oracle.cached_step(self.chat, self.V, self.R)
