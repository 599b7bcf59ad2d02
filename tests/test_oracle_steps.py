"""Pins of the oracle's per-step path (project, residual, EMA, reconstruct) against the
paper's equations (Eq. 8 - Eq. 11 and the reconstruction rule of Sec. 3.5), closed forms
and special cases."""
import os

import numpy as np
import pytest

from oracle import svdcache_oracle as oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _orthonormal(rng, D, k):
    Q, _ = np.linalg.qr(rng.standard_normal((D, k)))
    return Q


def test_hand_computed_projection_and_ema_fixture():
    rows = np.loadtxt(os.path.join(GOLDEN, "projection_ema_fixture.txt"))
    V = np.array([[0.6], [0.8]])
    chat = None
    for step, f0, f1, c, r0, r1, ch, fh0, fh1 in rows:
        C, R, chat = oracle.full_step(np.array([[f0, f1]]), V, 0.9, chat)
        assert C[0, 0] == pytest.approx(c, abs=1e-14)
        np.testing.assert_allclose(R[0], [r0, r1], atol=1e-14)
        assert chat[0, 0] == pytest.approx(ch, abs=1e-14)
        Fh = oracle.cached_step(chat, V, R)
        np.testing.assert_allclose(Fh[0], [fh0, fh1], atol=1e-14)


def test_full_rank_basis_reconstructs_exactly():
    """k = D: the residual vanishes and C V^T = F; with no forecast applied (first step)
    the cached step returns F."""
    rng = np.random.default_rng(0)
    D = 24
    F = rng.standard_normal((9, D))
    V = _orthonormal(rng, D, D)
    C, R, Chat = oracle.full_step(F, V, 0.9)
    assert np.abs(R).max() <= 1e-14
    np.testing.assert_allclose(C @ V.T, F, atol=1e-14)
    np.testing.assert_allclose(oracle.cached_step(Chat, V, R), F, atol=1e-14)


@pytest.mark.parametrize("N,D,k", [(5, 16, 3), (33, 48, 16), (130, 96, 32)])
def test_residual_is_orthogonal_and_energy_splits(N, D, k):
    rng = np.random.default_rng(N)
    F = rng.standard_normal((N, D)) * 3.0
    V = _orthonormal(rng, D, k)
    C, R, _ = oracle.full_step(F, V, 0.9)
    assert np.abs(R @ V).max() <= 1e-13
    np.testing.assert_allclose(np.sum(F * F, 1), np.sum(C * C, 1) + np.sum(R * R, 1), rtol=1e-13)
    # F_k + R = F (Eq. 10)
    np.testing.assert_allclose(C @ V.T + R, F, atol=1e-13)


def test_inputs_inside_and_outside_the_subspace():
    rng = np.random.default_rng(5)
    D, k = 40, 8
    Q = _orthonormal(rng, D, 2 * k)
    V, W = Q[:, :k], Q[:, k:]
    inside = rng.standard_normal((6, k)) @ V.T
    C, R, Chat = oracle.full_step(inside, V, 0.9)
    assert np.abs(R).max() <= 1e-14
    outside = rng.standard_normal((6, k)) @ W.T
    C, R, Chat = oracle.full_step(outside, V, 0.9)
    assert np.abs(C).max() <= 1e-14
    np.testing.assert_allclose(R, outside, atol=1e-14)
    np.testing.assert_allclose(oracle.cached_step(Chat, V, R), outside, atol=1e-14)
    # projecting a residual again gives no principal part
    F = rng.standard_normal((6, D))
    _, R, _ = oracle.full_step(F, V, 0.9)
    C2, R2, _ = oracle.full_step(R, V, 0.9)
    assert np.abs(C2).max() <= 1e-14
    np.testing.assert_allclose(R2, R, atol=1e-14)


def test_transposed_basis_would_be_caught():
    """C[n, j] pairs column j of V_k with row n of F: check one entry by hand."""
    rng = np.random.default_rng(8)
    F = rng.standard_normal((3, 6))
    V = _orthonormal(rng, 6, 2)
    C, R, _ = oracle.full_step(F, V, 0.5)
    assert C[2, 1] == pytest.approx(sum(F[2, d] * V[d, 1] for d in range(6)), abs=1e-15)
    assert R[1, 4] == pytest.approx(F[1, 4] - sum(C[1, j] * V[4, j] for j in range(2)), abs=1e-15)


def _run_ema(Cs, beta):
    """Drive the oracle's EMA with prescribed coefficient sequences by feeding
    F_j = C_j V^T (so that the projection returns C_j)."""
    rng = np.random.default_rng(42)
    k = Cs[0].shape[1]
    V = _orthonormal(rng, 3 * k, k)
    chat = None
    out = []
    for Cj in Cs:
        _, _, chat = oracle.full_step(Cj @ V.T, V, beta, chat)
        out.append(chat.copy())
    return out


def test_ema_constant_sequence_is_a_fixed_point():
    C = np.random.default_rng(1).standard_normal((4, 5))
    for ch in _run_ema([C] * 6, 0.9):
        np.testing.assert_allclose(ch, C, atol=1e-13)


def test_ema_linear_sequence_closed_form():
    """C_j = a + b j with Chat_0 = C_0 gives Chat_j = C_j - b beta (1 - beta^j)/(1 - beta):
    the smoother lags a ramp by up to b beta/(1-beta) (9 b at beta = 0.9)."""
    rng = np.random.default_rng(2)
    a, b = rng.standard_normal((3, 4)), rng.standard_normal((3, 4))
    beta = 0.9
    outs = _run_ema([a + b * j for j in range(40)], beta)
    for j, ch in enumerate(outs):
        expect = a + b * j - b * beta * (1 - beta ** j) / (1 - beta)
        np.testing.assert_allclose(ch, expect, atol=1e-11)
    lag = (a + b * 39) - outs[-1]
    np.testing.assert_allclose(lag, 9 * b * (1 - beta ** 39), atol=1e-11)


def test_ema_general_weights():
    """Chat_j = beta^j C_0 + (1 - beta) sum_{i=1..j} beta^(j-i) C_i."""
    rng = np.random.default_rng(3)
    Cs = [rng.standard_normal((2, 3)) for _ in range(7)]
    beta = 0.7
    outs = _run_ema(Cs, beta)
    for j in range(7):
        expect = beta ** j * Cs[0] + (1 - beta) * sum(beta ** (j - i) * Cs[i] for i in range(1, j + 1))
        np.testing.assert_allclose(outs[j], expect, atol=1e-13)


def test_beta_zero_is_plain_feature_reuse():
    """beta = 0 turns the forecast into the latest coefficients, so the cached step
    returns the last fully computed feature: the reuse baseline of Eq. 3."""
    rng = np.random.default_rng(4)
    D, k = 32, 8
    V = _orthonormal(rng, D, k)
    chat = None
    for _ in range(3):
        F = rng.standard_normal((5, D))
        _, R, chat = oracle.full_step(F, V, 0.0, chat)
        np.testing.assert_allclose(oracle.cached_step(chat, V, R), F, atol=1e-14)


def test_beta_one_keeps_the_first_observation():
    rng = np.random.default_rng(6)
    D, k = 20, 4
    V = _orthonormal(rng, D, k)
    F0 = rng.standard_normal((3, D))
    C0, _, chat = oracle.full_step(F0, V, 1.0)
    for _ in range(3):
        _, _, chat = oracle.full_step(rng.standard_normal((3, D)), V, 1.0, chat)
    np.testing.assert_allclose(chat, C0, atol=1e-15)


def test_ema_on_coefficients_equals_ema_on_lowrank_features():
    """Eq. 11 is written on F_k (N x D).  With a fixed basis F_k = C V^T, so smoothing C
    and multiplying by V^T afterwards gives the same matrix."""
    rng = np.random.default_rng(9)
    D, k, beta = 30, 6, 0.9
    V = _orthonormal(rng, D, k)
    chat, Fk_hat = None, None
    for j in range(5):
        F = rng.standard_normal((4, D))
        C, R, chat = oracle.full_step(F, V, beta, chat)
        Fk = F - R                                           # Eq. 10 rearranged
        Fk_hat = Fk if Fk_hat is None else beta * Fk_hat + (1 - beta) * Fk   # Eq. 11 as printed
        np.testing.assert_allclose(chat @ V.T, Fk_hat, atol=1e-13)
        np.testing.assert_allclose(oracle.cached_step(chat, V, R), Fk_hat + R, atol=1e-13)


def test_sigma_cancels_between_eq8_and_eq9():
    """U = F V diag(sigma)^-1 (Eq. 8) followed by F_k = U_k diag(sigma_k) V_k^T (Eq. 9)
    is F V_k V_k^T whatever positive sigma is used."""
    rng = np.random.default_rng(10)
    D, k = 18, 5
    V = _orthonormal(rng, D, k)
    sigma = rng.uniform(0.5, 4.0, size=k)
    F = rng.standard_normal((7, D))
    U = (F @ V) / sigma
    Fk = (U * sigma) @ V.T
    _, R, _ = oracle.full_step(F, V, 0.9)
    np.testing.assert_allclose(F - R, Fk, atol=1e-13)


def test_steps_do_not_depend_on_thread_count():
    rng = np.random.default_rng(12)
    F = rng.standard_normal((64, 48))
    V = _orthonormal(rng, 48, 8)
    n0 = oracle.threads()
    try:
        oracle.set_threads(1)
        a = oracle.full_step(F, V, 0.9)
        oracle.set_threads(max(2, n0))
        b = oracle.full_step(F, V, 0.9)
    finally:
        oracle.set_threads(n0)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
