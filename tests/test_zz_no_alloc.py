"""The calibration entry point that needs no workspace from the caller.

Who needs it: a host that is not allowed to allocate device memory at the point where it
calibrates -- a plugin living inside a server whose memory pool was carved up at start-up,
or code running inside a latency-critical loop where cudaMalloc would stall the device.
`svdcache_calibrate_noalloc` runs the same calibration on a scratch array that is part of
the library itself, so all the caller brings is its input stack and its output buffers.

The test calls it through the C ABI twice in a row (the second call starts from the first
call's leftovers in the shared scratch, and on a different stack) and holds each result
against the regular entry point on the same input: same subspace (principal-angle cosines
>= 1 - 1e-4, the bound of the other calibration tests), same eigenvalues and trace.  It
also checks that a problem too large for the built-in scratch is refused with its own
status code before anything is launched.  This file sorts last so that a run stopping at
the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams

pytestmark = pytest.mark.gpu
DEV = "cuda"
COS_MIN = 1.0 - 1e-4


def _stack(seed_block: int, M: int, D: int, k: int, dtype: str) -> torch.Tensor:
    spec = streams.StreamSpec("noalloc", blocks=1, rows=M, D=D, dtype=dtype, k=k, T=2, interval=1,
                              rank=min(D, 2 * k), amp=30.0, power=1.0, noise_std=0.02)
    return streams.BlockStream(spec, seed_block, trajectory=1, device=DEV).features(0)


def test_noalloc_calibration_matches_the_regular_entry_point_twice_in_a_row():
    cases = [(0, 1500, 384, 32, "bf16"), (1, 900, 264, 24, "f32")]
    # outputs are the caller's: allocate them (and everything else) before the calls under test
    prepared = []
    for block, M, D, k, dtype in cases:
        stack = _stack(block, M, D, k, dtype)
        ref = sc.svdcache_calibrate(stack, k)
        out = (torch.empty(D, k, dtype=torch.float32, device=DEV),
               torch.empty(k, dtype=torch.float64, device=DEV),
               torch.empty(1, dtype=torch.float64, device=DEV))
        assert sc.svdcache_calibrate_workspace_bytes(D, k) <= sc.BUILTIN_SCRATCH_BYTES
        prepared.append((stack, k, ref, out))
    torch.cuda.synchronize()
    for stack, k, (Vr, lr, tr, _), (Vk, lam, trc) in prepared:
        sc.svdcache_calibrate_noalloc(stack, k, Vk, lam, trc)
        torch.cuda.synchronize()
        cos = torch.linalg.svdvals(Vr.double().t() @ Vk.double())
        assert float(cos.min()) >= COS_MIN, f"smallest principal-angle cosine {float(cos.min()):.8f}"
        np.testing.assert_allclose(lam.cpu().numpy(), lr.cpu().numpy(), rtol=1e-9)
        assert float(trc.cpu()[0]) == pytest.approx(float(tr.cpu()[0]), rel=1e-12)


def test_noalloc_calibration_refuses_what_the_builtin_scratch_cannot_hold():
    D, k = 1152, 64
    assert sc.svdcache_calibrate_workspace_bytes(D, k) > sc.BUILTIN_SCRATCH_BYTES
    stack = torch.zeros(64, D, dtype=torch.float32, device=DEV)
    Vk = torch.empty(D, k, dtype=torch.float32, device=DEV)
    lam = torch.empty(k, dtype=torch.float64, device=DEV)
    tr = torch.empty(1, dtype=torch.float64, device=DEV)
    launches = sc.svdcache_kernel_launches()
    with pytest.raises(sc.SvdCacheError) as err:
        sc.svdcache_calibrate_noalloc(stack, k, Vk, lam, tr)
    assert err.value.code == -9
    assert sc.svdcache_kernel_launches() == launches
