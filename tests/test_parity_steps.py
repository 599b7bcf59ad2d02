"""GPU parity of the fused full step and cached step against the fp64 oracle, through the
C ABI, on the same seeded inputs (Eq. 8 - Eq. 11, Sec. 3.5)."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams
from tests.parity_util import (OracleTrack, basis_as_consumed, check_close, orthonormal_basis)

pytestmark = pytest.mark.gpu
DEV = "cuda"
TD = {sc.F32: torch.float32, sc.BF16: torch.bfloat16}


def _np(t):
    return t.detach().double().cpu().numpy()


def _rms(x):
    return float(np.sqrt(np.mean(np.square(x))))


def _play(spec, block, Vk, timesteps, rows=None, sample=None, path=0, ld_pad=0, poison=False):
    """Run the schedule `timesteps` (full when t % interval == 0) for one block through the
    library and the oracle; compare every output of every step on `sample` rows (all rows
    if None).  `poison` fills Chat and R of the fresh state with NaN first: the first full
    step must not read either."""
    prev = sc.svdcache_set_path(path)
    try:
        st = streams.BlockStream(spec, block, device=DEV, rows=rows)
        if Vk is None:   # the generator's own leading directions: a well calibrated basis
            Vk = st.V_gen[:, :spec.k].float().contiguous()
        N, D, k = st.rows, spec.D, Vk.shape[1]
        dt = sc.F32 if spec.dtype == "f32" else sc.BF16
        basis = sc.svdcache_basis_prepare(Vk, dt)
        state = sc.new_state(N, D, k, dt, DEV)
        chat_v, r_v = sc.state_views(state, N, D, k, dt)
        if poison:
            chat_v.fill_(float("nan"))
            r_v.fill_(float("nan"))
        idx = torch.arange(N) if sample is None else sample
        idx_d = idx.to(DEV)
        track = OracleTrack(basis_as_consumed(basis, D, k, dt), spec.beta)
        C_out = torch.empty(N, k, dtype=torch.float32, device=DEV)
        Fbuf = torch.empty(N, D + ld_pad, dtype=TD[dt], device=DEV)[:, :D]
        Fhat = torch.full((N, D + ld_pad), float("nan"), dtype=TD[dt], device=DEV)[:, :D]
        worst = {}
        rms_f = 1.0
        for t in timesteps:
            if t % spec.interval == 0:
                Fbuf.copy_(st.features(t))
                sc.svdcache_full_step(Fbuf, basis, state, k, spec.beta, C_out=C_out)
                F_rows = _np(Fbuf[idx_d])
                rms_f = _rms(F_rows)
                track.full(F_rows)
                for name, got, ref, coeff in (("C", C_out[idx_d], track.C, D),
                                              ("Chat", chat_v[idx_d], track.chat, D),
                                              ("R", r_v[idx_d], track.R, 0)):
                    e = check_close(f"{name}@t={t}", got, ref, dt, rms_f, coeff=coeff)
                    worst[name] = max(worst.get(name, 0.0), e)
            else:
                sc.svdcache_cached_step(state, basis, Fhat, k, steps_since_full=t % spec.interval)
                e = check_close(f"Fhat@t={t}", Fhat[idx_d], track.cached(), dt, rms_f)
                worst["Fhat"] = max(worst.get("Fhat", 0.0), e)
        steps, status = sc.svdcache_state_query(state)
        assert status == 0
        assert steps == sum(1 for t in timesteps if t % spec.interval == 0)
        return worst
    finally:
        sc.svdcache_set_path(prev)


def _calibrated_basis(spec, block, rows_per_snapshot=None):
    stack = streams.calibration_stack(spec, block, device=DEV, rows_per_snapshot=rows_per_snapshot)
    Vk, lam, tr, info = sc.svdcache_calibrate(stack, spec.k)
    return Vk


def test_tiny_config_whole_trajectory():
    spec = streams.TINY
    Vk = _calibrated_basis(spec, 0)
    worst = _play(spec, 0, Vk, range(spec.T))
    assert set(worst) == {"C", "Chat", "R", "Fhat"}


@pytest.mark.parametrize("block", [0, 13, 27])
def test_dit_xl_config_blocks(block):
    spec = streams.DIT_XL
    # calibration on a quarter of the configured stack keeps the test short; the basis is
    # the same for both sides, so the step parity does not depend on its quality
    Vk = _calibrated_basis(spec, block, rows_per_snapshot=64)
    _play(spec, block, Vk, range(spec.T))


SHAPES = [
    # N, D, k, dtype, ld_pad
    (1, 8, 8, "f32", 0),
    (7, 64, 16, "f32", 4),
    (129, 264, 24, "f32", 0),
    (300, 1152, 64, "f32", 0),
    (1, 64, 64, "bf16", 0),
    (127, 256, 64, "bf16", 8),
    (129, 512, 64, "bf16", 0),
    (300, 1152, 64, "bf16", 0),
    (257, 3072, 128, "bf16", 0),
    (1000, 512, 256, "bf16", 0),
    (200, 768, 192, "bf16", 0),     # three K blocks: operand in tensor memory, previous Chat fetched per block
    (515, 1024, 16, "bf16", 0),
    (384, 2048, 32, "bf16", 64),
    (40, 8192, 64, "bf16", 0),
]


@pytest.mark.parametrize("N,D,k,dtype,ld_pad", SHAPES)
def test_shapes_and_ragged_tails(N, D, k, dtype, ld_pad):
    spec = streams.StreamSpec("shape", blocks=1, rows=N, D=D, dtype=dtype, k=k, T=5, interval=2,
                              rank=min(D, 2 * k), amp=30.0, power=1.0, noise_std=0.02)
    # f32: an arbitrary orthonormal basis (large residual); bf16: the generator's leading
    # directions, as a calibrated basis gives -- the max-abs bound of the bf16 mode presumes
    # the stored residual is small against F (its bf16 rounding alone is 2^-9 |R|)
    Vk = orthonormal_basis(D, k, seed=D + k) if dtype == "f32" else None
    _play(spec, 0, Vk, range(5), ld_pad=ld_pad)


def _random_shapes(n, seed=20260131):
    """Seeded draw of bf16 shapes the tensor-core kernels take: every rank class (operand in shared
    memory, in tensor memory with two buffers or one), widths that are not a multiple of the group
    width, row counts with ragged last tiles, padded leading dimensions."""
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        k = int(rng.choice([16, 32, 64, 128, 192, 256]))
        D = int(rng.integers(max(k, 64) // 8, 2600 // 8)) * 8
        N = int(rng.integers(1, 1500))
        ld_pad = int(rng.choice([0, 8, 64]))
        out.append((N, D, k, ld_pad))
    return out


@pytest.mark.parametrize("N,D,k,ld_pad", _random_shapes(18))
def test_random_bf16_shapes(N, D, k, ld_pad):
    spec = streams.StreamSpec("rand", blocks=1, rows=N, D=D, dtype="bf16", k=k, T=4, interval=2,
                              rank=min(D, 2 * k), amp=30.0, power=1.0, noise_std=0.02)
    _play(spec, 0, None, range(4), ld_pad=ld_pad)


@pytest.mark.parametrize("D", [256, 448, 704])
def test_first_full_step_never_reads_the_old_state(D):
    """Narrow blocks with many row tiles: a tile takes fewer chunks than the load ring has slots,
    so nothing but the kernel's own ordering keeps the first-step branch of Eq. 11 apart from the
    step count.  The state starts as NaN; every output of the first step must be finite and right."""
    spec = streams.StreamSpec("narrow", blocks=1, rows=20000, D=D, dtype="bf16", k=64, T=3, interval=1,
                              rank=128, amp=30.0, power=1.0, noise_std=0.02)
    _play(spec, 0, None, range(3), path=2, poison=True, sample=streams.sample_rows(20000, 4096, tile=128))


@pytest.mark.parametrize("path,rows,D,k", [(0, 200, 512, 64), (2, 200, 512, 64), (2, 700, 3072, 64),
                                          (2, 700, 3072, 128), (2, 300, 1024, 256)])
def test_batched_equals_per_block_and_oracle(path, rows, D, k):
    """One batched launch over three blocks (tiles run across block boundaries) against three
    per-block launches (bitwise) and the oracle."""
    prev = sc.svdcache_set_path(path)
    try:
        _batched_case(rows, D, k)
    finally:
        sc.svdcache_set_path(prev)


def _batched_case(rows, D, k=64):
    spec = streams.StreamSpec("batch", blocks=3, rows=rows, D=D, dtype="bf16", k=k, T=4, interval=2,
                              rank=2 * k, amp=30.0, power=1.0, noise_std=0.02)
    nb, N, D, k, dt = 3, spec.rows, spec.D, spec.k, sc.BF16
    bases = torch.stack([sc.svdcache_basis_prepare(
        streams.BlockStream(spec, b, device=DEV).V_gen[:, :k].float().contiguous(), dt) for b in range(nb)])
    st_b = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    st_s = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    F = torch.stack([streams.BlockStream(spec, b, device=DEV).features(0) for b in range(nb)])
    F2 = torch.stack([streams.BlockStream(spec, b, device=DEV).features(2) for b in range(nb)])
    Cb = torch.empty(nb, N, k, dtype=torch.float32, device=DEV)
    out_b = torch.empty(nb, N, D, dtype=torch.bfloat16, device=DEV)
    out_s = torch.empty_like(out_b)
    for Fi in (F, F2):
        sc.svdcache_full_step_batched(Fi, bases, st_b, k, 0.9, C_out=Cb)
        for b in range(nb):
            sc.svdcache_full_step(Fi[b], bases[b], st_s[b], k, 0.9)
    sc.svdcache_cached_step_batched(st_b, bases, out_b, k)
    for b in range(nb):
        sc.svdcache_cached_step(st_s[b], bases[b], out_s[b], k)
    torch.cuda.synchronize()
    for b in range(nb):   # compare the defined parts of the state (padding is never written)
        for x, y in zip(sc.state_views(st_b[b], N, D, k, dt), sc.state_views(st_s[b], N, D, k, dt)):
            assert torch.equal(x, y)
    assert torch.equal(out_b, out_s)
    for b in range(nb):
        tr = OracleTrack(basis_as_consumed(bases[b], D, k, dt), 0.9)
        tr.full(_np(F[b]))
        tr.full(_np(F2[b]))
        rms = _rms(_np(F2[b]))
        check_close("C", Cb[b], tr.C, dt, rms, coeff=D)
        check_close("Fhat", out_b[b], tr.cached(), dt, rms)
        assert sc.svdcache_state_query(st_b[b]) == (2, 0)


def test_flux_shape_full_size_sampled_rows(path=2):
    """All 57 blocks of the FLUX-shaped stream at full size in one batched launch per step --
    the launch the benchmark times: 2052 row tiles, every CTA runs about 14 units -- three full
    steps (first-step branch, then the EMA twice) each
    followed by a cached step; the oracle checks 512 sampled rows of every block one by one."""
    spec = streams.FLUX
    nb, N, D, k, dt = spec.blocks, spec.rows, spec.D, spec.k, sc.BF16
    prev = sc.svdcache_set_path(path)
    try:
        strs = [streams.BlockStream(spec, b, device=DEV) for b in range(nb)]
        bases = torch.stack([sc.svdcache_basis_prepare(s.V_gen[:, :k].float().contiguous(), dt) for s in strs])
        state = sc.new_state(N, D, k, dt, DEV, blocks=nb)
        F = torch.empty(nb, N, D, dtype=torch.bfloat16, device=DEV)
        Fhat = torch.empty_like(F)
        C = torch.empty(nb, N, k, dtype=torch.float32, device=DEV)
        rows = streams.sample_rows(N, 512, tile=128, extra=(4095, 4096))
        rows_d = rows.to(DEV)
        tracks = [OracleTrack(basis_as_consumed(bases[b], D, k, dt), spec.beta) for b in range(nb)]
        for t in (0, 6, 12):
            for b in range(nb):
                strs[b].features(t, out=F[b])
            sc.svdcache_full_step_batched(F, bases, state, k, spec.beta, C_out=C)
            sc.svdcache_cached_step_batched(state, bases, Fhat, k)
            assert sc.svdcache_last_path() == path
            for b in range(nb):
                Fr = _np(F[b][rows_d])
                tracks[b].full(Fr)
                rms = _rms(Fr)
                chat_v, r_v = sc.state_views(state[b], N, D, k, dt)
                check_close(f"C[{b}]", C[b][rows_d], tracks[b].C, dt, rms, coeff=D)
                check_close(f"Chat[{b}]", chat_v[rows_d], tracks[b].chat, dt, rms, coeff=D)
                check_close(f"R[{b}]", r_v[rows_d], tracks[b].R, dt, rms)
                check_close(f"Fhat[{b}]", Fhat[b][rows_d], tracks[b].cached(), dt, rms)
        for b in range(nb):
            assert sc.svdcache_state_query(state[b]) == (3, 0)
    finally:
        sc.svdcache_set_path(prev)


def test_hunyuan_shape_full_size_sampled_rows(path=2):
    """One block of the HunyuanVideo-shaped stream at full N = 118,800 and k = 128 (929 row
    tiles: several units per CTA)."""
    spec = streams.HUNYUAN
    prev = sc.svdcache_set_path(path)
    try:
        _hunyuan_case(spec)
        assert sc.svdcache_last_path() == path
    finally:
        sc.svdcache_set_path(prev)


def _hunyuan_case(spec):
    N, D, k, dt = spec.rows, spec.D, spec.k, sc.BF16
    st = streams.BlockStream(spec, 3, device=DEV)
    basis = sc.svdcache_basis_prepare(st.V_gen[:, :k].float().contiguous(), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    F = torch.empty(N, D, dtype=torch.bfloat16, device=DEV)
    Fhat = torch.empty_like(F)
    rows = streams.sample_rows(N, 1024, tile=128, extra=(3599, 3600, 7199, 7200, 118783, 118784))
    rows_d = rows.to(DEV)
    track = OracleTrack(basis_as_consumed(basis, D, k, dt), spec.beta)
    chat_v, r_v = sc.state_views(state, N, D, k, dt)
    for t in (0, 6):
        st.features(t, out=F)
        sc.svdcache_full_step(F, basis, state, k, spec.beta)
        sc.svdcache_cached_step(state, basis, Fhat, k)
        Fr = _np(F[rows_d])
        track.full(Fr)
        rms = _rms(Fr)
        check_close("Chat", chat_v[rows_d], track.chat, dt, rms, coeff=D)
        check_close("R", r_v[rows_d], track.R, dt, rms)
        check_close("Fhat", Fhat[rows_d], track.cached(), dt, rms)
    # properties that hold at any size: the stored residual has no component along V_k
    Vb = sc.basis_views(basis, D, k, dt)[2].float()
    leak = (r_v.float() @ Vb).norm() / r_v.float().norm()
    assert float(leak) < 2e-2   # bf16 rounding of R only


@pytest.mark.parametrize("k", streams.SWEEP_RANKS)
def test_rank_sweep_on_flux_width(k):
    spec = streams.StreamSpec("sweep", blocks=1, rows=640, D=3072, dtype="bf16", k=k, T=3, interval=2,
                              rank=256, amp=200.0, power=1.1, noise_std=0.01)
    Vk = streams.BlockStream(spec, 0, device=DEV).V_gen[:, :k].float().contiguous()
    _play(spec, 0, Vk, range(3))


def test_cached_step_before_any_full_step_is_reported_not_computed():
    N, D, k, dt = 64, 256, 16, sc.BF16
    basis = sc.svdcache_basis_prepare(orthonormal_basis(D, k, 1), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    out = torch.full((N, D), 7.0, dtype=torch.bfloat16, device=DEV)
    sc.svdcache_cached_step(state, basis, out, k)
    steps, status = sc.svdcache_state_query(state)
    assert (steps, status) == (0, -4)
    assert bool((out == 7.0).all())
    # reset clears the sticky status
    sc.svdcache_state_reset(state, N, D, k, dt)
    assert sc.svdcache_state_query(state) == (0, 0)


@pytest.mark.parametrize("k", [64, 128, 256])
def test_batched_cached_step_skips_blocks_without_a_full_step(k):
    """A batch in which only some blocks have seen a full step: those are reconstructed exactly as
    by a call of their own, the others are reported (status -4) and their output is left alone --
    at every rank the operand reaches the tensor cores by a different route."""
    N, D, dt, nb = 900, 1024, sc.BF16, 4
    spec = streams.StreamSpec("mixed", blocks=nb, rows=N, D=D, dtype="bf16", k=k, T=2, interval=1,
                              rank=2 * k, amp=30.0, power=1.0, noise_std=0.02)
    bases = torch.stack([sc.svdcache_basis_prepare(
        streams.BlockStream(spec, b, device=DEV).V_gen[:, :k].float().contiguous(), dt) for b in range(nb)])
    state = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    live = (0, 2)
    for b in live:
        sc.svdcache_full_step(streams.BlockStream(spec, b, device=DEV).features(0), bases[b], state[b], k, 0.9)
    out = torch.full((nb, N, D), 7.0, dtype=torch.bfloat16, device=DEV)
    sc.svdcache_cached_step_batched(state, bases, out, k)
    ref = torch.empty(N, D, dtype=torch.bfloat16, device=DEV)
    for b in range(nb):
        if b in live:
            sc.svdcache_cached_step(state[b], bases[b], ref, k)
            assert torch.equal(out[b], ref)
            assert sc.svdcache_state_query(state[b]) == (1, 0)
        else:
            assert bool((out[b] == 7.0).all())
            assert sc.svdcache_state_query(state[b]) == (0, -4)


def test_beta_zero_returns_the_last_full_feature():
    """beta = 0: the forecast is the latest coefficients, so Fhat = F_k + R = F up to the
    bf16 rounding of R and Fhat (the reuse baseline, Eq. 3)."""
    N, D, k, dt = 256, 1024, 64, sc.BF16
    spec = streams.StreamSpec("b0", blocks=1, rows=N, D=D, dtype="bf16", k=k, T=4, interval=1, rank=128,
                              amp=30.0, power=1.0, noise_std=0.02)
    st = streams.BlockStream(spec, 0, device=DEV)
    basis = sc.svdcache_basis_prepare(st.V_gen[:, :k].float().contiguous(), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    out = torch.empty(N, D, dtype=torch.bfloat16, device=DEV)
    for t in range(3):
        F = st.features(t)
        sc.svdcache_full_step(F, basis, state, k, 0.0)
        sc.svdcache_cached_step(state, basis, out, k)
        err = (out.float() - F.float()).norm() / F.float().norm()
        assert float(err) < 5e-3


def test_nan_and_inf_propagate_per_row():
    N, D, k, dt = 40, 128, 16, sc.F32
    F = torch.randn(N, D, device=DEV)
    F[3, 5] = float("nan")
    F[9, 0] = float("inf")
    basis = sc.svdcache_basis_prepare(orthonormal_basis(D, k, 2), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    out = torch.empty(N, D, device=DEV)
    sc.svdcache_full_step(F, basis, state, k, 0.9)
    sc.svdcache_cached_step(state, basis, out, k)
    bad = ~torch.isfinite(out).all(dim=1)
    assert bad[3] and bad[9] and int(bad.sum()) == 2
    assert sc.svdcache_state_query(state) == (1, 0)


def test_results_are_bitwise_reproducible():
    N, D, k, dt = 333, 1152, 64, sc.BF16
    F = (torch.randn(N, D, device=DEV) * 3).bfloat16()
    basis = sc.svdcache_basis_prepare(orthonormal_basis(D, k, 3), dt)
    outs = []
    for _ in range(2):
        state = sc.new_state(N, D, k, dt, DEV)
        out = torch.empty(N, D, dtype=torch.bfloat16, device=DEV)
        sc.svdcache_full_step(F, basis, state, k, 0.9)
        sc.svdcache_full_step(F * 2, basis, state, k, 0.9)
        sc.svdcache_cached_step(state, basis, out, k)
        torch.cuda.synchronize()
        chat_v, r_v = sc.state_views(state, N, D, k, dt)
        outs.append((chat_v.clone(), r_v.clone(), out.clone()))
    assert all(torch.equal(x, y) for x, y in zip(outs[0], outs[1]))


def test_argument_errors_are_refused_before_launch():
    L = sc.lib()
    N, D, k, dt = 64, 256, 16, sc.BF16
    basis = sc.svdcache_basis_prepare(orthonormal_basis(D, k, 1), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    F = torch.zeros(N, D + 8, dtype=torch.bfloat16, device=DEV)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    before = sc.svdcache_kernel_launches()
    assert L.svdcache_full_step(None, D, p(basis), p(state), None, N, D, k, dt, 0.9, s) == -1
    assert L.svdcache_full_step(p(F), D, p(basis), p(state), None, N, D, 12, dt, 0.9, s) == -2   # k % 8
    assert L.svdcache_full_step(p(F), D, p(basis), p(state), None, N, D, 512, dt, 0.9, s) == -2  # k > 256
    assert L.svdcache_full_step(p(F), D - 8, p(basis), p(state), None, N, D, k, dt, 0.9, s) == -2  # ld < D
    assert L.svdcache_full_step(p(F), D + 1, p(basis), p(state), None, N, D, k, dt, 0.9, s) == -3  # pitch
    assert L.svdcache_full_step(ctypes.c_void_p(F.data_ptr() + 2), D + 8, p(basis), p(state), None, N, D, k,
                                dt, 0.9, s) == -3
    assert L.svdcache_full_step(p(F), D + 8, p(basis), p(state), None, N, D, k, 5, 0.9, s) == -1  # dtype
    assert L.svdcache_full_step(p(F), D + 8, p(basis), p(state), None, N, D, k, dt, 1.5, s) == -1  # beta
    assert L.svdcache_cached_step(p(state), p(basis), None, D, N, D, k, dt, 1, s) == -1
    assert L.svdcache_full_step(p(F), D + 8, p(basis), p(state), None, 0, D, k, dt, 0.9, s) == -2  # N = 0
    assert sc.svdcache_kernel_launches() == before
    torch.cuda.synchronize()
