"""Pins of the oracle's calibration path (Gram matrix, eigen-solver, top-k basis, rank
selection) against what the paper's definitions and the mathematics fix: Eq. 4 - Eq. 7."""
import os

import numpy as np
import pytest

from oracle import svdcache_oracle as oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _fixture(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            rows[parts[0]] = np.array([float(x) for x in parts[1:]])
    return rows


def _lowrank(rng, M, D, rank, amp=10.0, power=1.0, noise=0.0):
    V, _ = np.linalg.qr(rng.standard_normal((D, rank)))
    s = amp * np.arange(1, rank + 1) ** (-power)
    U = rng.standard_normal((M, rank))
    F = (U * s) @ V.T
    if noise:
        F = F + noise * rng.standard_normal((M, D))
    return F, V, s


def _subspace_cosines(A, B):
    return np.linalg.svd(A.T @ B, compute_uv=False)


def test_hand_computed_svd_fixture():
    fx = _fixture("svd_fixture.txt")
    Fa = np.array([[3.0, 0.0], [0.0, 4.0], [0.0, 0.0]])
    V, lam, tr, lam_all = oracle.calibrate(Fa, 2, all_eigenvalues=True)
    np.testing.assert_allclose(np.sqrt(lam), fx["sigma_a"], atol=1e-14)
    np.testing.assert_allclose(V[:, 0], fx["v1_a"], atol=1e-14)
    np.testing.assert_allclose(V[:, 1], fx["v2_a"], atol=1e-14)
    assert tr == fx["trace_a"][0]
    assert oracle.rank_for_energy(lam_all, tr, 0.6) == 1
    assert oracle.rank_for_energy(lam_all, tr, 0.64) == 1
    assert oracle.rank_for_energy(lam_all, tr, 0.85) == 2
    Fb = np.ones((2, 2))
    V, lam, tr = oracle.calibrate(Fb, 1)
    np.testing.assert_allclose(np.sqrt(lam), fx["sigma_b"][:1], atol=1e-14)
    np.testing.assert_allclose(V[:, 0], fx["v1_b"], atol=1e-14)
    assert tr == fx["trace_b"][0]


def test_gram_is_the_definition_on_tiny_input():
    rng = np.random.default_rng(1)
    F = rng.standard_normal((7, 5))
    G = oracle.gram(F)
    for i in range(5):
        for j in range(5):
            assert G[i, j] == pytest.approx(sum(F[m, i] * F[m, j] for m in range(7)), abs=1e-14)
    assert np.array_equal(G, G.T)


@pytest.mark.parametrize("M,D,k", [(64, 24, 6), (300, 96, 16), (512, 160, 32)])
def test_basis_invariants(M, D, k):
    rng = np.random.default_rng(D)
    F, _, _ = _lowrank(rng, M, D, rank=min(D, 40), noise=0.05)
    V, lam, tr, lam_all = oracle.calibrate(F, k, all_eigenvalues=True)
    # orthonormal columns
    np.testing.assert_allclose(V.T @ V, np.eye(k), atol=1e-12)
    # descending, non-negative up to rounding
    assert np.all(np.diff(lam_all) <= 1e-9 * lam_all[0])
    # sum of all eigenvalues = trace(G) = |F|_F^2
    assert tr == pytest.approx(np.sum(F * F), rel=1e-13)
    assert np.sum(lam_all) == pytest.approx(tr, rel=1e-12)
    # Eckart-Young (Eq. 5): the rank-k truncation error is the discarded energy
    resid = F - (F @ V) @ V.T
    assert np.sum(resid * resid) == pytest.approx(tr - np.sum(lam), rel=1e-9)
    # eigen-equation G v = lambda v
    G = F.T @ F
    np.testing.assert_allclose(G @ V, V * lam, atol=1e-9 * lam[0])
    # sign convention: largest-magnitude entry of each column is positive
    assert np.all(V[np.argmax(np.abs(V), axis=0), np.arange(k)] > 0)


@pytest.mark.parametrize("m,n", [(40, 24), (96, 64), (10, 10)])
def test_jacobi_svd_brute_force_agrees_with_gram_route(m, n):
    rng = np.random.default_rng(m * 100 + n)
    # distinct, well separated singular values so individual vectors are comparable
    A, _, _ = _lowrank(rng, m, n, rank=min(m, n), amp=5.0, power=0.7)
    sig, Vj = oracle.jacobi_svd(A)
    V, lam, tr = oracle.calibrate(A, n)
    np.testing.assert_allclose(np.sqrt(np.maximum(lam, 0.0)), sig, rtol=1e-9, atol=1e-9)
    # columns agree up to sign
    dots = np.abs(np.sum(V * Vj, axis=0))
    np.testing.assert_allclose(dots[: min(m, n) - 1], 1.0, atol=1e-8)
    # the Jacobi factors reproduce A's Gram matrix: A^T A = V diag(sigma^2) V^T
    np.testing.assert_allclose((Vj * sig**2) @ Vj.T, A.T @ A, atol=1e-10 * sig[0] ** 2)


@pytest.mark.parametrize("n", [1, 2, 3, 17, 64, 130])
def test_eigh_against_lapack(n):
    rng = np.random.default_rng(n)
    B = rng.standard_normal((n, n))
    A = B + B.T
    w, Z = oracle.eigh_desc(A)
    wl = np.linalg.eigvalsh(A)[::-1]
    np.testing.assert_allclose(w, wl, atol=1e-12 * max(1.0, np.abs(wl).max()))
    np.testing.assert_allclose(Z.T @ Z, np.eye(n), atol=1e-12)
    np.testing.assert_allclose(Z @ np.diag(w) @ Z.T, A, atol=1e-11 * max(1.0, np.abs(wl).max()))


def test_eigh_handles_diagonal_and_repeated_eigenvalues():
    w, Z = oracle.eigh_desc(np.diag([1.0, 5.0, 3.0, 5.0]))
    np.testing.assert_allclose(w, [5.0, 5.0, 3.0, 1.0])
    np.testing.assert_allclose(Z.T @ Z, np.eye(4), atol=1e-14)
    A = np.full((6, 6), 2.0)  # rank one: eigenvalues 12, 0 x5
    w, Z = oracle.eigh_desc(A)
    np.testing.assert_allclose(w, [12, 0, 0, 0, 0, 0], atol=1e-13)
    np.testing.assert_allclose(np.abs(Z[:, 0]), np.full(6, 6 ** -0.5), atol=1e-14)


def test_topk_subspace_against_lapack_svd():
    rng = np.random.default_rng(7)
    F, _, _ = _lowrank(rng, 400, 128, rank=64, amp=20.0, power=1.1, noise=0.01)
    k = 16
    V, lam, _ = oracle.calibrate(F, k)
    _, s, Vt = np.linalg.svd(F, full_matrices=False)
    np.testing.assert_allclose(np.sqrt(lam), s[:k], rtol=1e-10)
    cos = _subspace_cosines(V, Vt[:k].T)
    assert cos.min() >= 1 - 1e-12


def test_generator_ground_truth_noise_free():
    """With no noise and k = generator rank, span(V_k) is the generator's basis and the
    residual of the stack vanishes."""
    rng = np.random.default_rng(11)
    F, Vgen, _ = _lowrank(rng, 200, 48, rank=12, amp=3.0, power=0.5)
    V, lam, tr = oracle.calibrate(F, 12)
    assert _subspace_cosines(V, Vgen).min() >= 1 - 1e-12
    assert np.sum(lam) == pytest.approx(tr, rel=1e-12)
    assert np.abs(F - (F @ V) @ V.T).max() <= 1e-11


def test_large_stack_asymptote_of_the_stream_generator():
    """For the synthetic streams the left factors are sines of independent uniform
    phases (variance 1/2), so G/M -> 1/2 V diag(s^2) V^T + std^2 I."""
    import torch
    from paper_2601_07396_b200 import streams
    spec = streams.StreamSpec("probe", blocks=1, rows=4096, D=64, dtype="f32", k=4, T=4,
                              interval=2, rank=8, amp=10.0, power=1.0, noise_std=0.05)
    st = streams.BlockStream(spec, block=0)
    F = st.features(0).double().numpy()
    V, lam, tr = oracle.calibrate(F, 4)
    s = st.s.numpy()
    expect = 0.5 * s[:4] ** 2 + spec.noise_std ** 2
    np.testing.assert_allclose(lam / spec.rows, expect, rtol=0.15)
    cos = _subspace_cosines(V, st.V_gen.numpy()[:, :8])
    assert cos.min() >= 0.999  # V_k lies inside the generator's rank-8 span


def test_rank_for_energy_definition():
    lam = np.array([8.0, 4.0, 2.0, 1.0, 1.0])
    tr = 16.0
    assert oracle.rank_for_energy(lam, tr, 0.5) == 1
    assert oracle.rank_for_energy(lam, tr, 0.51) == 2
    assert oracle.rank_for_energy(lam, tr, 0.75) == 2
    assert oracle.rank_for_energy(lam, tr, 0.85) == 3
    assert oracle.rank_for_energy(lam, tr, 1.0) == 5
    assert oracle.rank_for_energy(lam[:2], tr, 0.99) == 2  # short list: capped


def test_result_does_not_depend_on_thread_count():
    rng = np.random.default_rng(3)
    F = rng.standard_normal((200, 40))
    n0 = oracle.threads()
    try:
        oracle.set_threads(1)
        a = oracle.calibrate(F, 8)
        oracle.set_threads(max(2, n0))
        b = oracle.calibrate(F, 8)
    finally:
        oracle.set_threads(n0)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and a[2] == b[2]
