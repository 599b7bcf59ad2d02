"""Seeded synthetic feature streams with the shapes of the paper's workloads.

This module holds input generators only: none of the method's arithmetic lives here, so
both the CUDA library's tests/benchmark and the CPU oracle's tests may draw from it.

Real DiT hidden features need model weights and prompt sets; these streams stand in for
them and imitate the structure the paper describes for them (Fig. 1): a smooth,
high-energy low-rank part in a basis shared by all "prompts", plus a low-energy residual
whose sign flips from one timestep to the next.

For block ``b`` and trajectory ("prompt") ``j``::

    F_t = U_t diag(s) V_gen^T + (-1)^t E            (N x D, then rounded to the I/O dtype)
    V_gen        D x rank, orthonormal (Q of the QR of a Gaussian matrix; seed = block)
    s_i          amp * i^(-power), i = 1..rank
    U_t[n, i]    sin(omega[n, i] * t + phi[n, i] + psi[frame(n)])
    omega        ~ U[0.05, 0.3],  phi ~ U[0, 2 pi)  per (row, component); seed = (block, j)
    psi          ~ U[0, 2 pi) per video frame (HunyuanVideo shape only), else 0
    E            noise_std * Gaussian, fixed per trajectory

V_gen and s depend on the block only, which is the prompt invariance the paper reports
for the right singular vectors and singular values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class StreamSpec:
    name: str
    blocks: int          # DiT blocks carrying a cache each
    rows: int            # N: tokens x batch
    D: int               # hidden width
    dtype: str           # "f32" | "bf16": storage type of F, R and Fhat
    k: int               # rank of the principal subspace
    T: int               # sampling timesteps
    interval: int        # a full step every `interval` timesteps (t % interval == 0)
    rank: int            # generator rank
    amp: float
    power: float
    noise_std: float
    beta: float = 0.9    # EMA weight the paper uses in all experiments
    frame_rows: int = 0  # rows per video frame (0: no per-frame phase offsets)
    calib_trajectories: Tuple[int, ...] = (1,)
    calib_timesteps: Tuple[int, ...] = (0,)

    @property
    def torch_dtype(self) -> torch.dtype:
        return {"f32": torch.float32, "bf16": torch.bfloat16}[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return {"f32": 4, "bf16": 2}[self.dtype]

    def full_timesteps(self) -> List[int]:
        return [t for t in range(self.T) if t % self.interval == 0]

    def calib_rows(self) -> int:
        return len(self.calib_trajectories) * len(self.calib_timesteps) * self.rows


# The five configurations.  Calibration stacks: where the configuration text leaves the
# stack open, it is chosen here (tiny, HunyuanVideo).
TINY = StreamSpec("tiny", blocks=1, rows=256, D=1152, dtype="f32", k=32, T=10, interval=3,
                  rank=64, amp=100.0, power=1.2, noise_std=0.05,
                  calib_trajectories=(1, 2, 3, 4), calib_timesteps=(0, 3, 6, 9))
DIT_XL = StreamSpec("dit_xl", blocks=28, rows=8 * 256, D=1152, dtype="bf16", k=64, T=50,
                    interval=4, rank=128, amp=50.0, power=1.0, noise_std=0.02,
                    calib_trajectories=tuple(range(1, 17)), calib_timesteps=(0, 16, 32, 48))
FLUX = StreamSpec("flux", blocks=57, rows=4608, D=3072, dtype="bf16", k=64, T=50, interval=6,
                  rank=256, amp=200.0, power=1.1, noise_std=0.01,
                  calib_trajectories=tuple(range(1, 9)),
                  calib_timesteps=(0, 7, 14, 21, 28, 35, 42, 49))
HUNYUAN = StreamSpec("hunyuan", blocks=60, rows=118800, D=3072, dtype="bf16", k=128, T=50,
                     interval=6, rank=512, amp=300.0, power=1.1, noise_std=0.01,
                     frame_rows=3600, calib_trajectories=(1,), calib_timesteps=(0, 25))

SPECS = {s.name: s for s in (TINY, DIT_XL, FLUX, HUNYUAN)}
SWEEP_RANKS = (16, 32, 64, 128, 256)
SWEEP_CALIB_ROWS = (4608, 73728, 294912)


def _gen(device, *words: int) -> torch.Generator:
    seed = 0x9E3779B97F4A7C15
    for w in words:
        seed = ((seed ^ (int(w) + 0x632BE59BD9B4E019)) * 0xBF58476D1CE4E5B9) & ((1 << 63) - 1)
        seed ^= seed >> 29
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


class BlockStream:
    """Feature stream of one block and one trajectory.  ``rows`` may shrink the spec's N
    (the rows are independent draws, so a prefix of the rows is a valid smaller stream)."""

    def __init__(self, spec: StreamSpec, block: int, trajectory: int = 0,
                 device: str | torch.device = "cpu", rows: Optional[int] = None):
        self.spec = spec
        self.block = int(block)
        self.trajectory = int(trajectory)
        self.device = torch.device(device)
        self.rows = int(spec.rows if rows is None else rows)
        dev = self.device
        # basis and spectrum: block only
        gb = _gen(dev, 1, self.block)
        A = torch.randn(spec.D, spec.rank, generator=gb, device=dev, dtype=torch.float64)
        Q, _ = torch.linalg.qr(A)
        self.V_gen = Q.contiguous()                                   # D x rank, fp64
        i = torch.arange(1, spec.rank + 1, device=dev, dtype=torch.float64)
        self.s = spec.amp * i.pow(-spec.power)                        # rank
        self._VsT = (self.V_gen * self.s).t().contiguous().float()    # rank x D
        # trajectory-dependent left factors
        gt = _gen(dev, 2, self.block, self.trajectory)
        self.omega = 0.05 + 0.25 * torch.rand(self.rows, spec.rank, generator=gt, device=dev)
        self.phi = (2.0 * math.pi) * torch.rand(self.rows, spec.rank, generator=gt, device=dev)
        if spec.frame_rows > 0:
            frames = (spec.rows + spec.frame_rows - 1) // spec.frame_rows
            psi = (2.0 * math.pi) * torch.rand(frames, generator=gt, device=dev)
            frame_of_row = torch.arange(self.rows, device=dev) // spec.frame_rows
            self.phi = self.phi + psi[frame_of_row].unsqueeze(1)

    def _noise(self) -> torch.Tensor:
        ge = _gen(self.device, 3, self.block, self.trajectory)
        return self.spec.noise_std * torch.randn(self.rows, self.spec.D, generator=ge,
                                                 device=self.device)

    def features(self, t: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """F_t as an N x D tensor in the spec's I/O dtype."""
        U = torch.sin(self.omega * float(t) + self.phi)
        prev = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = False
        try:
            F = U @ self._VsT
        finally:
            torch.backends.cuda.matmul.allow_tf32 = prev
        E = self._noise()
        F.add_(E, alpha=(-1.0 if (t % 2) else 1.0))
        if out is None:
            return F.to(self.spec.torch_dtype)
        out.copy_(F)
        return out


def calibration_stack(spec: StreamSpec, block: int, device="cpu", rows_per_snapshot=None,
                      trajectories: Optional[Sequence[int]] = None,
                      timesteps: Optional[Sequence[int]] = None) -> torch.Tensor:
    """Row-stack of feature snapshots from the calibration trajectories of one block,
    (snapshots * rows) x D in the spec's I/O dtype."""
    trajectories = spec.calib_trajectories if trajectories is None else tuple(trajectories)
    timesteps = spec.calib_timesteps if timesteps is None else tuple(timesteps)
    n = spec.rows if rows_per_snapshot is None else int(rows_per_snapshot)
    out = torch.empty(len(trajectories) * len(timesteps) * n, spec.D,
                      dtype=spec.torch_dtype, device=device)
    at = 0
    for j in trajectories:
        stream = BlockStream(spec, block, trajectory=j, device=device, rows=n)
        for t in timesteps:
            stream.features(t, out=out[at:at + n])
            at += n
    return out


def sample_rows(n_rows: int, count: int, tile: int = 128, extra: Sequence[int] = (),
                seed: int = 0) -> torch.Tensor:
    """Row indices for sampled parity checks: the first and last rows, the rows around
    tile boundaries near both ends, any ``extra`` rows, then seeded random rows."""
    must = {0, 1, n_rows - 1, n_rows - 2, tile - 1, tile, n_rows - (n_rows % tile) - 1,
            n_rows - (n_rows % tile)}
    must.update(int(e) for e in extra)
    must = {r for r in must if 0 <= r < n_rows}
    g = torch.Generator().manual_seed(seed)
    want = max(0, min(count, n_rows) - len(must))
    perm = torch.randperm(n_rows, generator=g)[: want + len(must)].tolist()
    rows = list(must)
    for r in perm:
        if len(rows) >= min(count, n_rows):
            break
        if r not in must:
            rows.append(r)
    return torch.tensor(sorted(set(rows)), dtype=torch.long)
