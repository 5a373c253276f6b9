"""Pins of the inverse-root oracle (oracle/inv_root.py) against what the mathematics fixes: closed forms of the scalar
iteration, LAPACK's eigendecomposition as the plain definition of A^(-1/p), the exact-deflation identity in the
eigenbasis, independence of the padding value. No GPU."""
import numpy as np
import pytest

import oracle
from oracle import inv_root

RNG = np.random.default_rng(20260921)


def _haar(n):
    q, r = np.linalg.qr(RNG.standard_normal((n, n)))
    return q * np.sign(np.diag(r))[None, :]


def _spd(n, lam):
    q = _haar(n)
    return (q * lam) @ q.T, q


def _inv_root(A, p):
    w, v = np.linalg.eigh(A)
    return (v * w ** (-1.0 / p)) @ v.T


@pytest.mark.parametrize("m0", [1.0, 0.6, 0.05, 1e-3])
def test_scalar_iteration_closed_forms(m0):
    # p = 1 is Newton's iteration for the reciprocal: 1 - m_T = (1 - m0)^(2^T), z_T = m_T / m0
    for T in (1, 3, 6):
        z, m = inv_root.inv_root_scalar(m0, 1, T)
        assert np.isclose(1.0 - m, (1.0 - m0) ** (2 ** T), rtol=1e-10, atol=1e-15)
        assert np.isclose(z, m / m0, rtol=1e-12)
    # any p: m_T = m0 z_T^p (both are multiplied by the same factors), one is the fixed point, and the first
    # step multiplies a small m by ((p+1)/p)^p
    for p in (2, 3, 4):
        z, m = inv_root.inv_root_scalar(m0, p, 5)
        assert np.isclose(m, m0 * z ** p, rtol=1e-12)
        assert inv_root.inv_root_scalar(1.0, p, 7) == (1.0, 1.0)
        z1, m1 = inv_root.inv_root_scalar(1e-9, p, 1)
        assert np.isclose(m1 / 1e-9, ((p + 1) / p) ** p, rtol=1e-8)
    # convergence to the inverse root from anywhere in (0, 1]
    for p in (1, 2, 4):
        z, m = inv_root.inv_root_scalar(m0, p, 60)
        assert np.isclose(z, m0 ** (-1.0 / p), rtol=1e-12) and np.isclose(m, 1.0, rtol=1e-12)


@pytest.mark.parametrize("p", [1, 2, 4])
def test_matrix_iteration_is_the_scalar_iteration_on_the_spectrum(p):
    n = 12
    lam = np.linspace(1.0, 0.02, n)
    X0, q = _spd(n, lam)
    for T in (1, 4, 9):
        Z, M = inv_root.coupled_newton(X0, p, T)
        zs, ms = zip(*[inv_root.inv_root_scalar(l, p, T) for l in lam])
        assert np.allclose(q.T @ Z @ q, np.diag(zs), atol=1e-10 * max(zs))
        assert np.allclose(q.T @ M @ q, np.diag(ms), atol=1e-10)
        assert np.allclose(M, X0 @ np.linalg.matrix_power(Z, p), atol=1e-9 * max(zs) ** p)      # the coupling invariant
    Z, _ = inv_root.coupled_newton(X0, p, 40)
    assert np.allclose(Z, _inv_root(X0, p), rtol=0, atol=1e-10 * lam.min() ** (-1.0 / p))


@pytest.mark.parametrize("p", [2, 4])
def test_exact_deflation_restores_the_head_exactly_and_filters_the_rest(p):
    n, k, T, gamma = 40, 3, 6, 1.25
    lam = np.concatenate([[900.0, 400.0, 150.0], np.linspace(1.0, 0.08, n - k)])
    A, q = _spd(n, lam)
    v0 = RNG.standard_normal(n)
    out, Vn, lam_o, ndef, theta = inv_root.deflated_inv_root(A, q[:, :k].copy(), k, p, T, gamma=gamma, lanczos_v0=v0)
    assert ndef == k and np.allclose(lam_o, lam[:k], rtol=1e-12)
    assert 1.0 <= theta <= 1.05                                # the residual's largest eigenvalue is 1
    D = q.T @ out @ q
    want = np.concatenate([lam[:k] ** (-1.0 / p),
                           [theta ** (-1.0 / p) * inv_root.inv_root_scalar(l / theta, p, T)[0] for l in lam[k:]]])
    assert np.allclose(D, np.diag(want), atol=1e-9 * want.max())
    # the padding value drops out
    out2, *_ = inv_root.deflated_inv_root(A, q[:, :k].copy(), k, p, T, gamma=2.0, lanczos_v0=v0)
    assert np.allclose(out, out2, atol=1e-10 * want.max())
    # the basis moves on by one block step: span of A V
    assert np.allclose(Vn @ (Vn.T @ (A @ q[:, :k])), A @ q[:, :k], atol=1e-9 * lam[0])


def test_deflation_lowers_the_error_of_a_fixed_depth(  ):
    n, k, K, T, p = 48, 4, 6, 6, 2
    lam = np.concatenate([[2e3, 1.5e3, 800.0, 500.0], np.linspace(1.0, 0.05, n - 4)])
    A, q = _spd(n, lam)
    exact = _inv_root(A, p)
    v0 = RNG.standard_normal(n)
    Vb = oracle.householder_orth(q[:, :K] + 1e-3 * RNG.standard_normal((n, K)))
    plain, *_ = inv_root.deflated_inv_root(A, None, 0, p, T, lanczos_v0=v0)
    for _ in range(2):                                          # two block steps sharpen the perturbed basis
        defl, Vb, _, ndef, _ = inv_root.deflated_inv_root(A, Vb, k, p, T, lanczos_v0=v0)
    assert ndef == k
    e_plain = np.linalg.norm(plain - exact) / np.linalg.norm(exact)
    e_defl = np.linalg.norm(defl - exact) / np.linalg.norm(exact)
    assert e_plain > 0.5                 # the floor 0.05 / 2000 is out of reach of six steps
    assert e_defl < 1e-2 * e_plain
    # warm-up calls do not deflate but still advance the basis
    w, Vw, _, nd, _ = inv_root.deflated_inv_root(A, Vb, k, p, T, warmup=True, lanczos_v0=v0)
    assert nd == 0 and np.allclose(w, plain, atol=1e-12 * np.abs(plain).max()) and Vw.shape == (n, K)


def test_undeflated_call_is_the_scaled_iteration():
    n, p, T = 16, 2, 5
    A, q = _spd(n, np.linspace(7.0, 0.9, n))
    v0 = RNG.standard_normal(n)
    out, Vn, lam, ndef, theta = inv_root.deflated_inv_root(A, None, 0, p, T, lanczos_v0=v0)
    assert Vn is None and ndef == 0 and lam.size == 0
    assert theta == oracle.lanczos_upper(A, v0)
    Z, _ = inv_root.coupled_newton(A / theta, p, T)
    assert np.allclose(out, 0.5 * (Z + Z.T) / np.sqrt(theta), atol=1e-13)
