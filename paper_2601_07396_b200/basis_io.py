"""Calibrated bases on disk: the paper's one-time SVD is done offline and its result -- V_k and
the singular values (Eq. 7) -- is what every later run loads.  One small binary file per block:

    magic "SVCBAS1\\0" | D, k (int32) | trace (float64) | lambda [k] float64 | V_k [D x k] float32

little-endian, row-major.  Host-side helpers only; `svdcache_basis_prepare` turns the loaded V_k
into the device buffer the step kernels read.
"""
from __future__ import annotations

import struct
from typing import Tuple

import numpy as np
import torch

MAGIC = b"SVCBAS1\0"


def save_basis(path: str, Vk: torch.Tensor, lam: torch.Tensor, trace: float) -> None:
    V = Vk.detach().to("cpu", torch.float32).contiguous().numpy()
    l = lam.detach().to("cpu", torch.float64).contiguous().numpy()
    D, k = V.shape
    if l.shape != (k,):
        raise ValueError("lambda must have one entry per column of V_k")
    with open(path, "wb") as fh:
        fh.write(MAGIC)
        fh.write(struct.pack("<iid", D, k, float(trace)))
        fh.write(l.astype("<f8").tobytes())
        fh.write(V.astype("<f4").tobytes())


def load_basis(path: str, device="cpu") -> Tuple[torch.Tensor, torch.Tensor, float]:
    """Returns (V_k [D x k] fp32, lambda [k] fp64, trace)."""
    with open(path, "rb") as fh:
        if fh.read(8) != MAGIC:
            raise ValueError(f"{path}: not a basis file")
        D, k, trace = struct.unpack("<iid", fh.read(16))
        if not (1 <= k <= D <= 1 << 20):
            raise ValueError(f"{path}: implausible shape {D} x {k}")
        l = np.frombuffer(fh.read(8 * k), dtype="<f8")
        V = np.frombuffer(fh.read(4 * D * k), dtype="<f4")
        if l.size != k or V.size != D * k:
            raise ValueError(f"{path}: truncated")
    return (torch.from_numpy(V.reshape(D, k).copy()).to(device), torch.from_numpy(l.copy()).to(device), float(trace))
