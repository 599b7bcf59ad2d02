"""Pins of the oracle routines beyond the method itself: the residual EMA of the ablation
(Sec. 4.5, Fig. 4(c)), the forecasts of other predictors on the principal coefficients
(Sec. 5.3, Fig. 4(b)) and the left factors of Eq. 8.  CPU only."""
import numpy as np
import pytest

from oracle import svdcache_oracle as oracle


def _basis(D, k, seed):
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((D, k)))
    return Q


# --------------------------------------------------------------- residual EMA ---

def test_residual_ema_with_beta_r_zero_is_the_method_itself():
    rng = np.random.default_rng(0)
    V = _basis(48, 8, 1)
    chat = rhat = chat0 = None
    for t in range(4):
        F = rng.standard_normal((20, 48))
        C0, R0, chat0 = oracle.full_step(F, V, 0.9, chat0)
        C1, rhat, chat = oracle.full_step_residual_ema(F, V, 0.9, 0.0, chat, rhat)
        assert np.array_equal(C0, C1) and np.array_equal(R0, rhat) and np.array_equal(chat0, chat)


def test_residual_ema_first_step_takes_the_residual_and_a_constant_stream_keeps_it():
    rng = np.random.default_rng(1)
    V = _basis(32, 4, 2)
    F = rng.standard_normal((10, 32))
    C, R, _ = oracle.full_step(F, V, 0.5, None)
    _, rhat, chat = oracle.full_step_residual_ema(F, V, 0.5, 0.7, None, None)
    assert np.array_equal(rhat, R)
    for _ in range(5):
        _, rhat, chat = oracle.full_step_residual_ema(F, V, 0.5, 0.7, chat, rhat)
    np.testing.assert_allclose(rhat, R, rtol=0, atol=1e-14)


def test_residual_ema_damps_a_sign_flipping_residual_to_its_closed_form():
    """r_t = (-1)^t e (the oscillation the paper reports for the residual subspace): the EMA started
    at r_0 = e obeys rhat_n = b rhat_{n-1} + (1-b)(-1)^n e, whose solution is
    rhat_n = e [ (1-b)/(1+b) (-1)^n + 2b/(1+b) b^n ] -- the smoothed residual shrinks to (1-b)/(1+b)."""
    rng = np.random.default_rng(2)
    D, k, b = 24, 4, 0.6
    V = _basis(D, k, 3)
    P = np.eye(D) - V @ V.T
    e = rng.standard_normal((6, D)) @ P          # lies in the residual subspace
    base = rng.standard_normal((6, k)) @ V.T     # principal part, constant
    chat = rhat = None
    for n in range(9):
        F = base + (-1) ** n * e
        _, rhat, chat = oracle.full_step_residual_ema(F, V, 0.9, b, chat, rhat)
        want = e * ((1 - b) / (1 + b) * (-1) ** n + 2 * b / (1 + b) * b ** n)
        np.testing.assert_allclose(rhat, want, rtol=0, atol=1e-13)


def test_residual_ema_general_weights():
    rng = np.random.default_rng(3)
    V = _basis(16, 3, 4)
    b = 0.8
    Fs = [rng.standard_normal((5, 16)) for _ in range(5)]
    Rs = [oracle.full_step(F, V, 0.0, None)[1] for F in Fs]
    chat = rhat = None
    for F in Fs:
        _, rhat, chat = oracle.full_step_residual_ema(F, V, 0.3, b, chat, rhat)
    n = len(Fs) - 1
    want = b ** n * Rs[0] + (1 - b) * sum(b ** (n - i) * Rs[i] for i in range(1, n + 1))
    np.testing.assert_allclose(rhat, want, rtol=0, atol=1e-13)


# ------------------------------------------------------------------- forecasts ---

@pytest.mark.parametrize("kind", ["taylor", "newton"])
def test_order_zero_is_plain_reuse(kind):
    c = np.arange(12.0).reshape(3, 4)
    for u in (0.0, 0.25, 1.0):
        assert np.array_equal(oracle.forecast([c], u, kind), c)


@pytest.mark.parametrize("kind", ["taylor", "newton"])
def test_hand_computed_values(kind):
    # newest 10, before 7, before that 5:  D1 = 3, D2 = 3 - 2 = 1;  u = 1/2
    h = [np.array([10.0]), np.array([7.0]), np.array([5.0])]
    want = {"taylor": 10 + 0.5 * 3 + 0.125 * 1, "newton": 10 + 0.5 * 3 + 0.5 * 1.5 / 2 * 1}[kind]
    assert oracle.forecast(h, 0.5, kind)[0] == pytest.approx(want, abs=1e-15)
    # first order: both are the straight line through the last two points
    assert oracle.forecast(h[:2], 0.5, kind)[0] == pytest.approx(11.5, abs=1e-15)
    # u = 0 returns the newest coefficients whatever the order
    assert oracle.forecast(h, 0.0, kind)[0] == 10.0


@pytest.mark.parametrize("order", [1, 2, 3, 4])
def test_newton_reproduces_polynomials_up_to_its_order_exactly(order):
    rng = np.random.default_rng(order)
    coef = rng.standard_normal((order + 1, 7))               # 7 independent polynomials of degree `order`
    poly = lambda x: sum(coef[d] * x ** d for d in range(order + 1))
    n = 6                                                     # index of the newest full step
    hist = [poly(float(n - j)) for j in range(order + 1)]
    for u in (1 / 6, 0.5, 5 / 6, 1.0, 2.0):
        np.testing.assert_allclose(oracle.forecast(hist, u, "newton"), poly(n + u), rtol=1e-12, atol=1e-12)
    # and it is the polynomial numpy fits through the same points
    xs = np.array([float(n - j) for j in range(order + 1)])
    fit = np.polyfit(xs, np.stack(hist), order)
    np.testing.assert_allclose(oracle.forecast(hist, 0.5, "newton"), np.polyval(fit, n + 0.5), rtol=1e-9, atol=1e-9)
    # one degree more is no longer reproduced
    hist_hi = [poly(float(n - j)) + (n - j) ** (order + 1) for j in range(order + 1)]
    assert np.abs(oracle.forecast(hist_hi, 0.5, "newton") - (poly(n + 0.5) + (n + 0.5) ** (order + 1))).min() > 1e-3


def test_taylor_is_exact_on_lines_and_lags_a_parabola_by_c_times_u():
    """c_j = a + b j + c j^2 at the full steps: D1 = b + c (2n - 1), D2 = 2c, so the second-order
    Taylor form gives c_n + u D1 + u^2 c = (true value at n + u) - c u."""
    a, b, c = 0.3, -1.2, 0.7
    seq = lambda x: a + b * x + c * x * x
    n = 5
    hist = [np.array([seq(float(n - j))]) for j in range(3)]
    for u in (0.2, 0.5, 1.0):
        got = oracle.forecast(hist, u, "taylor")[0]
        assert got == pytest.approx(seq(n + u) - c * u, abs=1e-12)
        line = [np.array([a + b * (n - j)]) for j in range(3)]
        assert oracle.forecast(line, u, "taylor")[0] == pytest.approx(a + b * (n + u), abs=1e-12)
    # the weights of the history sum to one: a constant sequence is kept
    k3 = [np.full(4, 2.5)] * 4
    assert np.allclose(oracle.forecast(k3, 0.7, "taylor"), 2.5) and np.allclose(oracle.forecast(k3, 0.7, "newton"), 2.5)


def test_forecast_is_linear_in_the_history():
    rng = np.random.default_rng(9)
    h1 = [rng.standard_normal(5) for _ in range(3)]
    h2 = [rng.standard_normal(5) for _ in range(3)]
    for kind in ("taylor", "newton"):
        lhs = oracle.forecast([2 * x - 3 * y for x, y in zip(h1, h2)], 0.4, kind)
        rhs = 2 * oracle.forecast(h1, 0.4, kind) - 3 * oracle.forecast(h2, 0.4, kind)
        np.testing.assert_allclose(lhs, rhs, atol=1e-13)


# ---------------------------------------------------------------- left factors ---

def test_left_factors_rebuild_the_principal_part_and_are_orthonormal_on_the_stack():
    rng = np.random.default_rng(4)
    F = rng.standard_normal((60, 20)) * np.linspace(3, 0.2, 20)
    k = 6
    V, lam, tr = oracle.calibrate(F, k)
    sigma = np.sqrt(lam)
    C, R, _ = oracle.full_step(F, V, 0.9, None)
    U = oracle.left_factors(C, sigma)
    np.testing.assert_allclose((U * sigma) @ V.T, F - R, atol=1e-12)          # Eq. 9
    np.testing.assert_allclose(U.T @ U, np.eye(k), atol=1e-10)                # left singular vectors of the stack
    s_np = np.linalg.svd(F, compute_uv=False)[:k]
    np.testing.assert_allclose(sigma, s_np, rtol=1e-10)                       # Eq. 7
    # a direction without energy gives a zero column, not a division by zero
    U0 = oracle.left_factors(C, np.r_[sigma[:-1], 0.0])
    assert np.all(U0[:, -1] == 0.0) and np.array_equal(U0[:, :-1], U[:, :-1])
