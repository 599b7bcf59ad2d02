"""GPU parity, through the C ABI, of what lies beyond the method's own two kernels: forecasts of
the principal coefficients by other predictors (Sec. 5.3, Fig. 4(b)), the residual EMA of the
ablation (Sec. 4.5, Fig. 4(c)), per-block ranks (Eq. 6), singular values and left factors
(Eq. 7, Eq. 8) -- each against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import svdcache_oracle as oracle
from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams
from tests.parity_util import basis_as_consumed, check_close

DEV = "cuda"
KIND = {sc.PREDICT_TAYLOR: "taylor", sc.PREDICT_NEWTON: "newton"}


def _np(t):
    return t.detach().double().cpu().numpy()


def _rms(x):
    return float(np.sqrt(np.mean(np.square(x))))


@pytest.mark.parametrize("predictor", [sc.PREDICT_TAYLOR, sc.PREDICT_NEWTON])
@pytest.mark.parametrize("order", [0, 1, 2, 3])
def test_forecast_weights_reproduce_the_oracle_forecast(predictor, order):
    """Host-only: the weights the library applies to the history against the oracle's
    difference-table evaluation of the same predictor."""
    rng = np.random.default_rng(order)
    hist = [rng.standard_normal((5, 7)) for _ in range(order + 1)]
    for s, interval in ((0, 4), (1, 6), (3, 6), (5, 6), (7, 7), (9, 4)):
        w = sc.svdcache_forecast_weights(predictor, order, s, interval)
        got = sum(wj * h for wj, h in zip(w, hist))
        np.testing.assert_allclose(got, oracle.forecast(hist, s / interval, KIND[predictor]), rtol=1e-12, atol=1e-12)
        assert sum(w) == pytest.approx(1.0, abs=1e-12)
    L = sc.lib()
    import ctypes
    buf = (ctypes.c_double * 9)()
    assert L.svdcache_forecast_weights(predictor, 8, 1, 4, buf) == -1      # order > 7
    assert L.svdcache_forecast_weights(0, 1, 1, 4, buf) == -1              # the EMA has no history weights
    assert L.svdcache_forecast_weights(predictor, 1, 1, 0, buf) == -1      # interval < 1


def _forecast_case(spec, block, rows, sample, orders=(1, 2)):
    st = streams.BlockStream(spec, block, device=DEV, rows=rows)
    N, D, k = st.rows, spec.D, spec.k
    dt = sc.F32 if spec.dtype == "f32" else sc.BF16
    basis = sc.svdcache_basis_prepare(st.V_gen[:, :k].float().contiguous(), dt)
    V = basis_as_consumed(basis, D, k, dt)
    state = sc.new_state(N, D, k, dt, DEV)
    idx = torch.arange(N) if sample is None else sample
    idx_d = idx.to(DEV)
    Fhat = torch.empty(N, D, dtype=spec.torch_dtype, device=DEV)
    hist_dev, hist_ref = [], []
    chat = R = None
    interval = spec.interval
    max_order = max(orders)
    for n_full in range(max_order + 2):
        t = n_full * interval
        F = st.features(t)
        C = torch.empty(N, k, dtype=torch.float32, device=DEV)
        sc.svdcache_full_step(F, basis, state, k, spec.beta, C_out=C)
        Fr = _np(F[idx_d])
        Cr, R, chat = oracle.full_step(Fr, V, float(np.float32(spec.beta)), chat)
        hist_dev.insert(0, C)
        hist_ref.insert(0, Cr)
        rms = _rms(Fr)
        for order in orders:
            if len(hist_dev) < order + 1:
                continue
            for predictor in (sc.PREDICT_TAYLOR, sc.PREDICT_NEWTON):
                for s in sorted({1, interval - 1}):
                    buf = sc.svdcache_cached_step_forecast_batched(state, basis, Fhat, k, hist_dev[:order + 1], predictor, s, interval)
                    pred = oracle.forecast(hist_ref[:order + 1], s / interval, KIND[predictor])
                    name = f"{KIND[predictor]} order {order} s={s} after {n_full + 1} full steps"
                    got_pred = buf[:N * k * 4].view(torch.float32).view(N, k)[idx_d]
                    # the weights (up to ~3 in magnitude at order 2) amplify the rounding of the history
                    e = np.linalg.norm(_np(got_pred) - pred) / np.linalg.norm(pred)
                    assert e <= 5 * max(1e-5, 4e-9 * D), f"forecast {name}: {e:.3e}"
                    check_close("Fhat " + name, Fhat[idx_d], oracle.cached_step(pred, V, R), dt, rms)
    # the EMA predictor through the same entry point is the plain cached step
    sc.svdcache_cached_step_forecast_batched(state, basis, Fhat, k, hist_dev[:1], sc.PREDICT_EMA, 1, interval)
    ref = torch.empty_like(Fhat)
    sc.svdcache_cached_step(state, basis, ref, k)
    assert torch.equal(Fhat, ref)
    assert sc.svdcache_state_query(state) == (max_order + 2, 0)


@pytest.mark.gpu
def test_forecast_predictors_tiny_config():
    _forecast_case(streams.TINY, 0, None, None)


@pytest.mark.gpu
def test_forecast_predictors_dit_xl_block():
    _forecast_case(streams.DIT_XL, 5, None, None)


@pytest.mark.gpu
def test_forecast_predictors_flux_block_sampled_rows():
    _forecast_case(streams.FLUX, 18, None, streams.sample_rows(streams.FLUX.rows, 512, tile=128), orders=(1, 2))


@pytest.mark.gpu
def test_forecast_batched_equals_per_block():
    spec = streams.StreamSpec("fc", blocks=3, rows=300, D=1024, dtype="bf16", k=64, T=9, interval=4, rank=128,
                              amp=30.0, power=1.0, noise_std=0.02)
    nb, N, D, k, dt = 3, spec.rows, spec.D, spec.k, sc.BF16
    strs = [streams.BlockStream(spec, b, device=DEV) for b in range(nb)]
    bases = torch.stack([sc.svdcache_basis_prepare(s.V_gen[:, :k].float().contiguous(), dt) for s in strs])
    state = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    hist = []
    for t in (0, 4, 8):
        F = torch.stack([s.features(t) for s in strs])
        C = torch.empty(nb, N, k, dtype=torch.float32, device=DEV)
        sc.svdcache_full_step_batched(F, bases, state, k, 0.9, C_out=C)
        hist.insert(0, C)
    out_b = torch.empty(nb, N, D, dtype=torch.bfloat16, device=DEV)
    out_s = torch.empty_like(out_b)
    sc.svdcache_cached_step_forecast_batched(state, bases, out_b, k, hist, sc.PREDICT_NEWTON, 3, 4)
    for b in range(nb):
        sc.svdcache_cached_step_forecast_batched(state[b], bases[b], out_s[b], k, [h[b] for h in hist], sc.PREDICT_NEWTON, 3, 4)
    assert torch.equal(out_b, out_s)


@pytest.mark.gpu
@pytest.mark.parametrize("N,D,k,dtype", [(256, 1152, 32, "f32"), (300, 1024, 64, "bf16"), (129, 3072, 128, "bf16"),
                                         (515, 1000, 32, "bf16"), (2000, 512, 16, "bf16")])
def test_residual_ema_full_step(N, D, k, dtype):
    """The ablation's full step: Chat as in the method, the stored residual an EMA of the residuals;
    then the cached step on that state."""
    spec = streams.StreamSpec("abl", blocks=1, rows=N, D=D, dtype=dtype, k=k, T=5, interval=1,
                              rank=min(D, 2 * k), amp=30.0, power=1.0, noise_std=0.05)
    st = streams.BlockStream(spec, 0, device=DEV)
    dt = sc.F32 if dtype == "f32" else sc.BF16
    basis = sc.svdcache_basis_prepare(st.V_gen[:, :k].float().contiguous(), dt)
    V = basis_as_consumed(basis, D, k, dt)
    state = sc.new_state(N, D, k, dt, DEV)
    chat_v, r_v = sc.state_views(state, N, D, k, dt)
    Fhat = torch.empty(N, D, dtype=spec.torch_dtype, device=DEV)
    chat = rhat = None
    beta, beta_r = 0.9, 0.5
    for t in range(4):
        F = st.features(t)
        C = torch.empty(N, k, dtype=torch.float32, device=DEV)
        sc.svdcache_full_step_residual_ema_batched(F, basis, state, k, beta, beta_r, C_out=C)
        assert sc.svdcache_last_path() == (1 if dtype == "f32" else 2)   # bf16: the tensor-core full step blends in its epilogue
        sc.svdcache_cached_step(state, basis, Fhat, k)
        Fh = _np(F)
        Cr, rhat, chat = oracle.full_step_residual_ema(Fh, V, float(np.float32(beta)), float(np.float32(beta_r)), chat, rhat)
        rms = _rms(Fh)
        check_close(f"C@{t}", C, Cr, dt, rms, coeff=D)
        check_close(f"Chat@{t}", chat_v, chat, dt, rms, coeff=D)
        # the stored residual is rounded to the I/O dtype at every step and fed back: t roundings pile up
        check_close(f"Rhat@{t}", r_v, rhat, dt, rms)
        check_close(f"Fhat@{t}", Fhat, oracle.cached_step(chat, V, rhat), dt, rms)
    assert sc.svdcache_state_query(state) == (4, 0)
    # beta_r = 0 is the method's own step, bit for bit
    s1, s2 = sc.new_state(N, D, k, dt, DEV), sc.new_state(N, D, k, dt, DEV)
    for t in range(2):
        F = st.features(t)
        sc.svdcache_full_step_residual_ema_batched(F, basis, s1, k, beta, 0.0)
        sc.svdcache_full_step(F, basis, s2, k, beta)
    for x, y in zip(sc.state_views(s1, N, D, k, dt), sc.state_views(s2, N, D, k, dt)):
        assert torch.equal(x, y)


@pytest.mark.gpu
@pytest.mark.parametrize("k", [64, 128])
def test_residual_ema_batch_with_blocks_at_their_first_step(k):
    """One batched launch in which some blocks blend with a stored residual and others are at their
    first full step (nothing to blend, nothing fetched): bitwise the per-block calls.  Enough row
    tiles that every CTA meets both kinds, in either order."""
    N, D, dt, nb = 5000, 1024, sc.BF16, 5
    spec = streams.StreamSpec("ablmix", blocks=nb, rows=N, D=D, dtype="bf16", k=k, T=3, interval=1,
                              rank=2 * k, amp=30.0, power=1.0, noise_std=0.05)
    st = [streams.BlockStream(spec, b, device=DEV) for b in range(nb)]
    bases = torch.stack([sc.svdcache_basis_prepare(st[b].V_gen[:, :k].float().contiguous(), dt) for b in range(nb)])
    s_b = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    s_s = sc.new_state(N, D, k, dt, DEV, blocks=nb)
    seasoned = (0, 2, 3)
    for b in seasoned:   # these blocks have a stored residual before the batched call
        for s_ in (s_b, s_s):
            sc.svdcache_full_step_residual_ema_batched(st[b].features(0), bases[b], s_[b], k, 0.9, 0.5)
    for t in (1, 2):
        F = torch.stack([st[b].features(t) for b in range(nb)])
        sc.svdcache_full_step_residual_ema_batched(F, bases, s_b, k, 0.9, 0.5)
        for b in range(nb):
            sc.svdcache_full_step_residual_ema_batched(F[b], bases[b], s_s[b], k, 0.9, 0.5)
        torch.cuda.synchronize()
        for b in range(nb):
            for x, y in zip(sc.state_views(s_b[b], N, D, k, dt), sc.state_views(s_s[b], N, D, k, dt)):
                assert torch.equal(x, y)
            assert sc.svdcache_state_query(s_b[b]) == ((t + 1) if b in seasoned else t, 0)


@pytest.mark.gpu
def test_blocks_of_different_rank_in_one_call():
    """Ranks picked per block from its own spectrum (Eq. 6 at tau = 0.85, rounded up to what the
    kernels take), one ranked call over all blocks against per-block calls (bitwise) and the oracle."""
    nb, N, D, dt = 5, 300, 1024, sc.BF16
    specs = [streams.StreamSpec("rk", blocks=nb, rows=N, D=D, dtype="bf16", k=64, T=3, interval=2, rank=128,
                                amp=30.0, power=p, noise_std=0.02) for p in (0.6, 0.6, 1.6, 1.6, 0.6)]
    strs = [streams.BlockStream(specs[b], b, device=DEV) for b in range(nb)]
    ranks = []
    for b in range(nb):
        stack = streams.BlockStream(specs[b], b, trajectory=1, device=DEV).features(0)
        Vk, lam, tr, _ = sc.svdcache_calibrate(stack, 64, strict=False)
        k_tau = sc.svdcache_rank_for_energy(lam.cpu().numpy(), float(tr.cpu()[0]), 0.85)
        assert k_tau == oracle.rank_for_energy(lam.cpu().numpy(), float(tr.cpu()[0]), 0.85)
        ranks.append(16 if k_tau <= 16 else 32 if k_tau <= 32 else 64)
    assert len(set(ranks)) > 1, ranks           # the steep spectra need a smaller rank than the flat ones
    kmax = max(ranks)
    bb = max(sc.svdcache_basis_bytes(D, r, dt) for r in ranks)
    sb = max(sc.svdcache_state_bytes(N, D, r, dt) for r in ranks)
    bb, sb = (bb + 255) // 256 * 256, (sb + 255) // 256 * 256
    bases = torch.zeros(nb, bb, dtype=torch.uint8, device=DEV)
    st_r = torch.zeros(nb, sb, dtype=torch.uint8, device=DEV)
    st_s = torch.zeros(nb, sb, dtype=torch.uint8, device=DEV)
    for b in range(nb):
        sc.svdcache_basis_prepare(strs[b].V_gen[:, :ranks[b]].float().contiguous(), dt, basis=bases[b])
        sc.svdcache_state_reset(st_r[b], N, D, ranks[b], dt)
        sc.svdcache_state_reset(st_s[b], N, D, ranks[b], dt)
    C = torch.zeros(nb, N * kmax, dtype=torch.float32, device=DEV)
    out_r = torch.empty(nb, N, D, dtype=torch.bfloat16, device=DEV)
    out_s = torch.empty_like(out_r)
    tracks = [None] * nb
    for t in (0, 2):
        F = torch.stack([s.features(t) for s in strs])
        sc.svdcache_full_step_ranked_batched(F, bases, st_r, ranks, 0.9, C_out=C)
        for b in range(nb):
            sc.svdcache_full_step(F[b], bases[b], st_s[b], ranks[b], 0.9)
            V = basis_as_consumed(bases[b], D, ranks[b], dt)
            tracks[b] = oracle.full_step(_np(F[b]), V, float(np.float32(0.9)), None if tracks[b] is None else tracks[b][2])
    sc.svdcache_cached_step_ranked_batched(st_r, bases, out_r, ranks)
    for b in range(nb):
        sc.svdcache_cached_step(st_s[b], bases[b], out_s[b], ranks[b])
    assert torch.equal(out_r, out_s)
    for b in range(nb):
        k = ranks[b]
        for x, y in zip(sc.state_views(st_r[b], N, D, k, dt), sc.state_views(st_s[b], N, D, k, dt)):
            assert torch.equal(x, y)
        Cr, R, chat = tracks[b]
        V = basis_as_consumed(bases[b], D, k, dt)
        rms = _rms(_np(strs[b].features(2)))
        check_close(f"C[{b}]", C[b][:N * k].view(N, k), Cr, dt, rms, coeff=D)
        check_close(f"Fhat[{b}]", out_r[b], oracle.cached_step(chat, V, R), dt, rms)
        assert sc.svdcache_state_query(st_r[b]) == (2, 0)


@pytest.mark.gpu
def test_singular_values_and_left_factors():
    spec = streams.StreamSpec("lf", blocks=1, rows=2000, D=256, dtype="f32", k=16, T=2, interval=1, rank=48,
                              amp=20.0, power=0.8, noise_std=0.02)
    F = streams.BlockStream(spec, 0, device=DEV).features(0)
    k, dt = 16, sc.F32
    Vk, lam, tr, _ = sc.svdcache_calibrate(F, k)
    sigma = sc.svdcache_singular_values(lam)
    np.testing.assert_allclose(_np(sigma), np.sqrt(_np(lam)), rtol=1e-15)
    s_ref = np.linalg.svd(_np(F), compute_uv=False)[:k]
    np.testing.assert_allclose(_np(sigma), s_ref, rtol=1e-8)                    # Eq. 7
    basis = sc.svdcache_basis_prepare(Vk, dt)
    state = sc.new_state(2000, 256, k, dt, DEV)
    C = torch.empty(2000, k, dtype=torch.float32, device=DEV)
    sc.svdcache_full_step(F, basis, state, k, 0.9, C_out=C)
    U = sc.svdcache_left_factors(C, sigma)
    Cr, R, _ = oracle.full_step(_np(F), _np(Vk), 0.9, None)
    Ur = oracle.left_factors(Cr, _np(sigma))
    assert np.linalg.norm(_np(U) - Ur) / np.linalg.norm(Ur) <= 1e-5
    np.testing.assert_allclose(_np(U).T @ _np(U), np.eye(k), atol=1e-4)         # F is the calibration stack itself
    sigma0 = sigma.clone()
    sigma0[-1] = 0.0
    assert bool((sc.svdcache_left_factors(C, sigma0)[:, -1] == 0).all())
