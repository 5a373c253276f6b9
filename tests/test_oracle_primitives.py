"""Pins for the oracle's dense primitives: each one against numpy/LAPACK or a defining property."""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20260921)


@pytest.mark.parametrize("ta,tb", [(False, False), (False, True), (True, False), (True, True)])
def test_matmul_matches_numpy(ta, tb):
    M, N, K = 13, 7, 19
    A = RNG.standard_normal((K, M) if ta else (M, K))
    B = RNG.standard_normal((N, K) if tb else (K, N))
    ref = (A.T if ta else A) @ (B.T if tb else B)
    got = oracle.matmul(A, B, ta, tb)
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("rows,cols", [(5, 5), (40, 7), (33, 1), (64, 24)])
def test_householder_orth(rows, cols):
    Y = RNG.standard_normal((rows, cols))
    Q = oracle.householder_orth(Y)
    assert np.allclose(Q.T @ Q, np.eye(cols), atol=1e-13)
    # same span, and R = Q^T Y upper triangular with a non-negative diagonal (unique QR factor)
    R = Q.T @ Y
    assert np.allclose(Q @ R, Y, atol=1e-12)
    assert np.allclose(np.tril(R, -1), 0, atol=1e-12)
    assert np.all(np.diag(R) > 0)
    q_np, r_np = np.linalg.qr(Y)
    q_np = q_np * np.sign(np.diag(r_np))[None, :]
    assert np.allclose(Q, q_np, atol=1e-12)


@pytest.mark.parametrize("rows,cols", [(6, 6), (50, 9), (20, 1), (96, 24)])
def test_jacobi_svd_matches_lapack(rows, cols):
    M = RNG.standard_normal((rows, cols)) @ np.diag(10.0 ** RNG.uniform(-3, 1, cols))
    U, s, V = oracle.jacobi_svd(M)
    s_np = np.linalg.svd(M, compute_uv=False)
    assert np.all(np.diff(s) <= 0)
    assert np.allclose(s, s_np, rtol=1e-11)
    assert np.allclose(U.T @ U, np.eye(cols), atol=1e-12)
    assert np.allclose(V.T @ V, np.eye(cols), atol=1e-12)
    assert np.allclose((U * s) @ V.T, M, atol=1e-12 * s[0])


@pytest.mark.parametrize("n", [1, 2, 9, 40])
def test_jacobi_eig_matches_lapack(n):
    H = RNG.standard_normal((n, n))
    H = H + H.T
    lam, E = oracle.jacobi_eig(H)
    assert np.allclose(np.sort(lam), np.linalg.eigvalsh(H), atol=1e-12 * max(1.0, np.abs(lam).max()))
    assert np.allclose(E.T @ E, np.eye(n), atol=1e-12)
    assert np.allclose((E * lam) @ E.T, H, atol=1e-11)


def test_lanczos_upper_is_an_upper_bound_and_tight():
    n = 60
    Q, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    lam = np.concatenate([[3.0, -2.5], RNG.uniform(-1, 1, n - 2)])
    Z = (Q * lam) @ Q.T
    Z = 0.5 * (Z + Z.T)
    theta = oracle.lanczos_upper(Z, RNG.standard_normal(n), steps=20)
    nrm2 = np.abs(np.linalg.eigvalsh(Z)).max()
    assert theta >= nrm2 * (1 - 1e-12)
    assert theta <= nrm2 * 1.05


def test_lanczos_exact_when_krylov_space_is_full():
    # with steps = n the largest Ritz value of Z^2 is lambda_max(Z^2) and the residual vanishes
    n = 8
    Z = RNG.standard_normal((n, n))
    Z = Z + Z.T
    theta = oracle.lanczos_upper(Z, RNG.standard_normal(n), steps=n)
    assert np.isclose(theta, np.abs(np.linalg.eigvalsh(Z)).max(), rtol=1e-6)


def test_fill_gaussian_moments_and_determinism():
    x = oracle.fill_gaussian(200000, 12345)
    y = oracle.fill_gaussian(200000, 12345)
    z = oracle.fill_gaussian(1000, 12346)
    assert np.array_equal(x, y)
    assert not np.array_equal(x[:1000], z)
    assert abs(x.mean()) < 0.01
    assert abs(x.var() - 1.0) < 0.01
    assert abs((x ** 4).mean() - 3.0) < 0.1
    # a prefix of a longer stream is the shorter stream (counter based)
    assert np.array_equal(oracle.fill_gaussian(777, 12345), x[:777])
