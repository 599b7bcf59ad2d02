"""GPU parity of the calibration path (Gram matrix + top-k eigenvectors, Eq. 4 - Eq. 7)
against the fp64 oracle on the same seeded stacks, through the C ABI.

Several bases are correct for one stack (signs, and rotations inside near-degenerate
eigenvalue clusters), so the basis is compared through what is unique: the principal
angles between the two k-dimensional subspaces, the eigenvalues and the trace."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import svdcache_oracle as oracle
from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams

pytestmark = pytest.mark.gpu
DEV = "cuda"
COS_MIN = 1.0 - 1e-4


def _compare(stack: torch.Tensor, k: int, Vk, lam, tr, check_gap=True):
    Fh = stack.double().cpu().numpy()
    Vo, lo, to, lall = oracle.calibrate(Fh, k, all_eigenvalues=True)
    V = Vk.double().cpu().numpy()
    lam = lam.cpu().numpy()
    # orthonormal (fp32 storage), ordered, signed
    np.testing.assert_allclose(V.T @ V, np.eye(k), atol=5e-6)
    assert np.all(np.diff(lam) <= 1e-12 * lam[0])
    assert np.all(V[np.argmax(np.abs(V), axis=0), np.arange(k)] > 0)
    # eigenvalues and trace.  The fp64 Gram reproduces them to ~1e-10.  The tensor-core Gram
    # (bf16 stacks of >= 2048 rows whose width is a multiple of 128) sums each chunk of 2048
    # rows in fp32 before it adds the chunk to the fp64 total, and the tensor cores truncate
    # that running sum: G comes out smaller by a few 1e-6, almost uniformly -- which moves the
    # eigenvalues by that much and the eigenvectors (what the method uses) hardly at all.
    M, D = stack.shape
    tensor_gram = stack.dtype == torch.bfloat16 and D >= 256 and D % 128 == 0 and M >= 2048
    # (a perturbation of G of relative size e moves every eigenvalue by at most e * lambda_1)
    rtol_l, atol_l, rel_t = (2e-5, 5e-6, 2e-5) if tensor_gram else (1e-9, 1e-12, 1e-12)
    np.testing.assert_allclose(lam, lo, rtol=rtol_l, atol=atol_l * lo[0])
    assert float(tr.cpu()[0]) == pytest.approx(to, rel=rel_t)
    # the subspace is well defined only if lambda_k is separated from lambda_{k+1}
    if check_gap and k < len(lall):
        gap = (lall[k - 1] - lall[k]) / lall[k - 1]
        assert gap > 1e-3, f"oracle eigen-gap at k too small to grade angles: {gap:.2e}"
    cos = np.linalg.svd(Vo.T @ V, compute_uv=False)
    assert cos.min() >= COS_MIN, f"smallest principal-angle cosine {cos.min():.8f}"
    return cos.min()


def test_tiny_config_calibration():
    spec = streams.TINY
    stack = streams.calibration_stack(spec, 0, device=DEV)
    assert stack.shape == (4096, 1152) and stack.dtype == torch.float32
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare(stack, spec.k, Vk, lam, tr)
    assert info[1] <= 1e-12


@pytest.mark.parametrize("block", [0, 27])
def test_dit_xl_config_calibration(block):
    spec = streams.DIT_XL
    # 16 calibration trajectories x 4 timesteps x 256 tokens (batch 1) = 16,384 rows
    stack = streams.calibration_stack(spec, block, device=DEV, rows_per_snapshot=256)
    assert stack.shape == (16384, 1152) and stack.dtype == torch.bfloat16
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare(stack, spec.k, Vk, lam, tr)


def test_flux_width_calibration_single_snapshot():
    """FLUX width (D = 3072) on one snapshot of 4608 rows (the smallest stack of the
    calibration sweep); the full 294,912-row stack differs only in the Gram loop length."""
    spec = streams.FLUX
    stack = streams.calibration_stack(spec, 0, device=DEV, trajectories=(1,), timesteps=(0,))
    assert stack.shape == (4608, 3072)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare(stack, spec.k, Vk, lam, tr)


def _compare_large(stack: torch.Tensor, k: int, Vk, lam, tr, min_gap=1e-7):
    """The same comparison for stacks whose fp64 copy would not fit comfortably on the host: the
    oracle's Gram routine is called snapshot by snapshot (the sum of the partial Gram matrices is
    the definition, Eq. 4), then the oracle's eigen-solver on the total."""
    M, D = stack.shape
    G = np.zeros((D, D))
    for lo in range(0, M, 4608):
        G += oracle.gram(stack[lo:lo + 4608].double().cpu().numpy())
    w, Z = oracle.eigh_desc(G)
    V = Vk.double().cpu().numpy()
    gap = (w[k - 1] - w[k]) / w[0]
    assert gap > min_gap, f"eigen-gap at k too small to grade angles: {gap:.2e}"
    cos = np.linalg.svd(Z[:, :k].T @ V, compute_uv=False)
    assert cos.min() >= COS_MIN, f"smallest principal-angle cosine {cos.min():.8f} (gap {gap:.2e})"
    # eigenvalues and trace on the tensor-core path: see _compare
    np.testing.assert_allclose(lam.cpu().numpy(), w[:k], rtol=2e-5, atol=5e-6 * w[0])
    assert float(tr.cpu()[0]) == pytest.approx(float(np.trace(G)), rel=2e-5)
    np.testing.assert_allclose(V.T @ V, np.eye(k), atol=5e-6)
    return cos.min(), gap


def test_flux_stack_of_73728_rows():
    """The middle stack of the calibration sweep: 16 snapshots of the FLUX-shaped stream
    (73,728 x 3072, bf16, k = 64) against the oracle.  The eigen-gap at k of this spectrum is only
    a few 1e-6 of lambda_1, so this is where an fp32 sum over the whole stack would lose the
    subspace."""
    spec = streams.FLUX
    stack = streams.calibration_stack(spec, 0, device=DEV, trajectories=(1, 2), timesteps=spec.calib_timesteps)
    assert stack.shape == (73728, 3072)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare_large(stack, spec.k, Vk, lam, tr)


def test_flux_configured_stack_of_294912_rows():
    """The FLUX configuration's own calibration stack: 8 trajectories x 8 timesteps x 4608 rows =
    294,912 x 3072 (the stack the calibration timing is quoted on), against the oracle."""
    spec = streams.FLUX
    stack = streams.calibration_stack(spec, 5, device=DEV)
    assert stack.shape == (294912, 3072)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare_large(stack, spec.k, Vk, lam, tr)


def test_hunyuan_configuration_rank_and_width():
    """The HunyuanVideo configuration's calibration: k = 128 at D = 3072 (the Ritz problem of 160
    columns no longer fits shared memory and runs its Jacobi sweeps from global memory), on two
    snapshots of 8192 rows, which takes the tensor-core Gram."""
    spec = streams.HUNYUAN
    stack = streams.calibration_stack(spec, 2, device=DEV, rows_per_snapshot=8192)
    assert stack.shape == (16384, 3072) and stack.dtype == torch.bfloat16
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    _compare_large(stack, spec.k, Vk, lam, tr)


def test_finish_refuses_a_workspace_begun_for_another_shape():
    """svdcache_calibrate_finish (and _accumulate) against what svdcache_calibrate_begin laid out."""
    L = sc.lib()
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    ws = torch.empty(sc.svdcache_calibrate_workspace_bytes(512, 64), dtype=torch.uint8, device=DEV)
    spec = streams.StreamSpec("cal", blocks=1, rows=300, D=256, dtype="f32", k=8, T=2, interval=1,
                              rank=48, amp=40.0, power=1.0, noise_std=0.02)
    F = streams.BlockStream(spec, 0, device=DEV).features(1)
    Vk = torch.empty(512, 64, device=DEV)
    sc.svdcache_calibrate_begin(256, 16, ws)
    sc.svdcache_calibrate_accumulate(F, ws)
    # another width, and a larger rank than the workspace was begun for
    assert L.svdcache_calibrate_finish(512, 16, p(Vk), None, None, None, p(ws), ws.numel(), s) == -5
    assert L.svdcache_calibrate_finish(256, 32, p(Vk), None, None, None, p(ws), ws.numel(), s) == -5
    # a chunk of another width poisons the accumulation
    F2 = torch.randn(300, 128, device=DEV)
    assert L.svdcache_calibrate_accumulate(p(F2), 300, 128, 128, 0, p(ws), ws.numel(), s) == 0
    assert L.svdcache_calibrate_finish(256, 16, p(Vk), None, None, None, p(ws), ws.numel(), s) == -5
    # begun again, the same workspace works, also for a smaller rank than begun
    sc.svdcache_calibrate_begin(256, 16, ws)
    sc.svdcache_calibrate_accumulate(F, ws)
    V8, lam, tr, info = sc.svdcache_calibrate_finish(256, 8, ws, strict=False)
    _compare(F, 8, V8, lam, tr)


@pytest.mark.parametrize("M,D,k,dtype", [(100, 64, 8, "f32"), (1000, 264, 24, "bf16"), (37, 128, 16, "f32"),
                                         (5000, 512, 256, "bf16"), (3001, 1000, 128, "bf16")])
def test_ragged_shapes(M, D, k, dtype):
    spec = streams.StreamSpec("cal", blocks=1, rows=M, D=D, dtype=dtype, k=k, T=2, interval=1,
                              rank=min(D, max(2 * k, 48)), amp=40.0, power=1.0, noise_std=0.02)
    stack = streams.BlockStream(spec, 0, device=DEV).features(1)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, k)
    _compare(stack, k, Vk, lam, tr, check_gap=(M > k))


def test_streaming_accumulation_matches_one_shot():
    spec = streams.StreamSpec("cal", blocks=1, rows=3000, D=384, dtype="bf16", k=32, T=2, interval=1,
                              rank=96, amp=40.0, power=1.1, noise_std=0.02)
    stack = streams.BlockStream(spec, 0, device=DEV).features(0)
    ws = torch.empty(sc.svdcache_calibrate_workspace_bytes(384, 32), dtype=torch.uint8, device=DEV)
    sc.svdcache_calibrate_begin(384, 32, ws)
    for lo, hi in ((0, 1), (1, 1000), (1000, 1000), (1000, 2999), (2999, 3000)):
        sc.svdcache_calibrate_accumulate(stack[lo:hi], ws)
    Vk, lam, tr, info = sc.svdcache_calibrate_finish(384, 32, ws)
    _compare(stack, 32, Vk, lam, tr)
    # and the run is reproducible bit for bit
    sc.svdcache_calibrate_begin(384, 32, ws)
    for lo, hi in ((0, 1), (1, 1000), (1000, 1000), (1000, 2999), (2999, 3000)):
        sc.svdcache_calibrate_accumulate(stack[lo:hi], ws)
    Vk2, lam2, tr2, _ = sc.svdcache_calibrate_finish(384, 32, ws)
    assert torch.equal(Vk, Vk2) and torch.equal(lam, lam2) and torch.equal(tr, tr2)


def test_noise_free_stack_recovers_the_generator_basis():
    spec = streams.StreamSpec("cal", blocks=1, rows=2000, D=256, dtype="f32", k=16, T=2, interval=1,
                              rank=16, amp=10.0, power=0.5, noise_std=0.0)
    st = streams.BlockStream(spec, 0, device=DEV)
    stack = st.features(0)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, 16, strict=False)
    cos = torch.linalg.svdvals(st.V_gen.t() @ Vk.double())
    assert float(cos.min()) >= 1 - 1e-6
    assert float(lam.sum()) == pytest.approx(float(tr[0]), rel=1e-6)   # all the energy is in rank 16


def test_steep_spectrum_takes_the_one_product_iteration():
    """A stack whose k-th eigenvalue lies 7 decades under the first: the degree-2 filter would lift
    the leading direction 1e14 over the k-th one per iteration, so the solver has to fall back to
    shifted power steps (one product with G per iteration) -- same subspace, same eigenvalues."""
    M, D, k, r = 3000, 1152, 32, 64
    g = torch.Generator(device="cpu").manual_seed(1234)
    A = torch.linalg.qr(torch.randn(M, r, generator=g, dtype=torch.float64))[0]
    B = torch.linalg.qr(torch.randn(D, r, generator=g, dtype=torch.float64))[0]
    sv = 10.0 ** (-0.12 * torch.arange(r, dtype=torch.float64))
    stack = ((A * sv) @ B.t() * 50.0).float().to(DEV)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, k)
    assert info[1] <= 1e-12
    assert float(lam[0] / lam[k - 1]) > 1e7
    _compare(stack, k, Vk, lam, tr)


def test_rank_selection_by_energy_threshold():
    """Eq. 6 on the calibrated spectrum, against the oracle's rule."""
    spec = streams.TINY
    stack = streams.calibration_stack(spec, 0, device=DEV)
    Vk, lam, tr, _ = sc.svdcache_calibrate(stack, 64)
    lam_h, tr_h = lam.cpu().numpy(), float(tr.cpu()[0])
    for tau in (0.5, 0.85, 0.9, 0.99):
        assert sc.svdcache_rank_for_energy(lam_h, tr_h, tau) == oracle.rank_for_energy(lam_h, tr_h, tau)
    assert 1 <= sc.svdcache_rank_for_energy(lam_h, tr_h, 0.85) < 64


def test_calibration_argument_errors():
    L = sc.lib()
    ws = torch.empty(sc.svdcache_calibrate_workspace_bytes(64, 8), dtype=torch.uint8, device=DEV)
    F = torch.zeros(16, 64, device=DEV)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert L.svdcache_calibrate_begin(64, 8, p(ws), 100, s) == -5
    assert L.svdcache_calibrate_begin(64, 9, p(ws), ws.numel(), s) == -2
    assert L.svdcache_calibrate_begin(64, 8, None, ws.numel(), s) == -1
    assert L.svdcache_calibrate_begin(64, 8, ctypes.c_void_p(ws.data_ptr() + 16), ws.numel() - 16, s) == -3
    assert L.svdcache_calibrate_accumulate(p(F), 16, 64, 60, 0, p(ws), ws.numel(), s) == -2
    assert L.svdcache_calibrate_accumulate(p(F), 16, 64, 64, 3, p(ws), ws.numel(), s) == -1
    assert L.svdcache_calibrate(p(F), 0, 64, 64, 0, 8, p(F), None, None, None, p(ws), ws.numel(), s) == -2
    torch.cuda.synchronize()
