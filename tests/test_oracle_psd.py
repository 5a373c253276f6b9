"""Pins for the PSD-projection side of the oracle (Algorithm 2, Eq. 6-7, Proposition 2)."""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(21102)


def _sym_with_spectrum(lam):
    n = len(lam)
    q, r = np.linalg.qr(RNG.standard_normal((n, n)))
    q = q * np.sign(np.diag(r))[None, :]
    Z = (q * lam) @ q.T
    return 0.5 * (Z + Z.T), q


def _psd_brute(Z):
    w, v = np.linalg.eigh(Z)
    return (v * np.maximum(w, 0)) @ v.T


def _p(x, coeffs):
    for a, b, c in coeffs:
        x = a * x + b * x ** 3 + c * x ** 5
    return x


def _head_spectrum(n, k):
    heads = np.array([30.0, -25.0, 22.0, -18.0, 15.0, 12.0])[:k]
    bulk = RNG.uniform(-1, 1, n - k)
    bulk[np.abs(bulk) < 0.05] = 0.3
    return np.concatenate([heads, bulk])


def test_eq6_matrix_relu_through_sign():
    lam = _head_spectrum(20, 3)
    Z, q = _sym_with_spectrum(lam)
    sgn = (q * np.sign(lam)) @ q.T
    assert np.allclose(0.5 * Z @ (np.eye(20) + sgn), _psd_brute(Z), atol=1e-11)


def test_undeflated_baseline_is_eq7():
    n = 24
    lam = _head_spectrum(n, 2)
    Z, q = _sym_with_spectrum(lam)
    T = 6
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, T)
    theta = 31.0
    P, _, _, ndef, scale = oracle.psd_project(Z, None, 0, coeffs, norm_mode=oracle.NORM_GIVEN, theta=theta)
    assert ndef == 0 and scale == theta
    ref = (q * (0.5 * lam * (1 + _p(lam / theta, coeffs)))) @ q.T
    assert np.allclose(P, ref, atol=1e-11)
    assert np.array_equal(P, P.T)
    # warm-up flag gives the same baseline even when a basis and k are passed
    P2, Vn, lam_r, ndef2, _ = oracle.psd_project(Z, q[:, :4], 2, coeffs, warmup=True,
                                                 norm_mode=oracle.NORM_GIVEN, theta=theta)
    assert ndef2 == 0
    assert np.allclose(P2, P, atol=1e-12)
    # ... and still advances the basis: Vnext spans Z V
    ZV = Z @ q[:, :4]
    assert np.allclose(Vn @ (Vn.T @ ZV), ZV, atol=1e-10)
    assert np.allclose(Vn.T @ Vn, np.eye(4), atol=1e-12)


@pytest.mark.parametrize("gamma", [1.0, 1.1, 2.0])
def test_prop2_closed_form_error_and_gamma_independence(gamma):
    n, k, T = 28, 3, 4
    lam = _head_spectrum(n, k)
    Z, q = _sym_with_spectrum(lam)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, T)
    theta_hat = 1.02                    # any upper bound on ||R_k||_2 = max|bulk| <= 1
    # exact eigenvectors of the k dominant eigenvalues as the basis: Rayleigh-Ritz is then exact
    P, Vn, lam_r, ndef, scale = oracle.psd_project(Z, q[:, :k], k, coeffs, gamma=gamma,
                                                   norm_mode=oracle.NORM_GIVEN, theta=theta_hat)
    assert ndef == k and scale == theta_hat
    assert np.allclose(np.sort(lam_r), np.sort(lam[:k]), atol=1e-11)
    # closed-form error matrix of the proof of Proposition 2
    err_coef = np.zeros(n)
    err_coef[k:] = -0.5 * np.abs(lam[k:]) * (1 - _p(np.abs(lam[k:]) / theta_hat, coeffs))
    ref = _psd_brute(Z) + (q * err_coef) @ q.T
    assert np.allclose(P, ref, atol=1e-10)
    assert np.array_equal(P, P.T)
    # gamma independence: compare with gamma = 1.3
    P3, *_ = oracle.psd_project(Z, q[:, :k], k, coeffs, gamma=1.3, norm_mode=oracle.NORM_GIVEN, theta=theta_hat)
    assert np.allclose(P, P3, atol=1e-10)


def test_prop2_ratio_bound_with_exact_scales():
    n, k, L, d = 26, 2, 3, 2
    lam = _head_spectrum(n, k)
    Z, q = _sym_with_spectrum(lam)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, L)
    mags = np.sort(np.abs(lam))[::-1]
    theta, theta_k = mags[0], mags[k]
    base, *_ = oracle.psd_project(Z, None, 0, coeffs, norm_mode=oracle.NORM_GIVEN, theta=theta)
    defl, *_ = oracle.psd_project(Z, q[:, :k], k, coeffs, gamma=1.1, norm_mode=oracle.NORM_GIVEN, theta=theta_k)
    ex = _psd_brute(Z)
    e_b, e_d = np.linalg.norm(base - ex, 2), np.linalg.norm(defl - ex, 2)
    ell = mags[-1] / theta
    alpha = theta / theta_k
    assert e_d / e_b <= ((1 - alpha ** 2 * ell ** 2) / (1 - ell ** 2)) ** ((d + 1) ** L) + 1e-12
    assert e_d <= theta_k / 2 * (1 - alpha ** 2 * ell ** 2) ** ((d + 1) ** L) + 1e-12
    # scalarised equality for the deflated error
    x = np.abs(lam[k:]) / theta_k
    assert np.isclose(e_d, theta_k / 2 * np.max(x * (1 - _p(x, coeffs))), atol=1e-11)


def test_only_positive_heads_are_restored_and_selection_is_by_magnitude():
    n, k = 22, 4
    lam = _head_spectrum(n, k)           # heads 30, -25, 22, -18
    Z, q = _sym_with_spectrum(lam)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 14)
    # basis = 6 exact eigenvectors (4 heads + 2 bulk directions), deflate the 4 of largest |lambda|
    idx = [0, 1, 2, 3, 7, 9]
    P, Vn, lam_r, ndef, _ = oracle.psd_project(Z, q[:, idx], k, coeffs, gamma=1.1,
                                               norm_mode=oracle.NORM_GIVEN, theta=1.0)
    assert ndef == 4
    assert np.allclose(np.abs(lam_r), np.sort(np.abs(lam[idx]))[::-1], atol=1e-11)
    assert np.allclose(P, _psd_brute(Z), atol=1e-7)


def test_rayleigh_ritz_and_basis_update_with_inexact_basis():
    n, K, k = 40, 6, 3
    lam = _head_spectrum(n, k)
    Z, q = _sym_with_spectrum(lam)
    V0, _ = np.linalg.qr(RNG.standard_normal((n, K)))
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 12)
    V = V0
    for it in range(9):                  # a static Z: the block steps converge the head (Ritz pairs lag one step)
        P, V, lam_r, ndef, scale = oracle.psd_project(Z, V, k, coeffs, gamma=1.1, lanczos_v0=RNG.standard_normal(n))
        assert np.allclose(V.T @ V, np.eye(K), atol=1e-12)
    assert ndef == k
    assert np.allclose(lam_r[:k], lam[:k], rtol=1e-6)
    # Lanczos scale is an upper bound on the residual's norm here and close to it
    nr = np.abs(lam[k:]).max()
    assert nr * (1 - 1e-6) <= scale <= nr * 1.2
    assert np.allclose(P, _psd_brute(Z), atol=1e-5)


def test_gate_on_magnitudes():
    n, K = 24, 6
    lam = _head_spectrum(n, 3)           # 30, -25, 22 then |bulk| <= 1
    Z, q = _sym_with_spectrum(lam)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 6)
    # window r = 5 Ritz magnitudes (30,25,22,<=1,<=1): s_r < tau s_1 -> fire, deflate the three above 3.0
    P, _, lam_r, ndef, _ = oracle.psd_project(Z, q[:, :K], 5, coeffs, tau=0.1, norm_mode=oracle.NORM_GIVEN, theta=1.0)
    assert ndef == 3
    # window r = 2: s_2 = 25 >= 3: gate stays off, baseline with the given scale
    P2, _, _, ndef2, _ = oracle.psd_project(Z, q[:, :K], 2, coeffs, tau=0.1, norm_mode=oracle.NORM_GIVEN, theta=30.0)
    assert ndef2 == 0
    base, *_ = oracle.psd_project(Z, None, 0, coeffs, norm_mode=oracle.NORM_GIVEN, theta=30.0)
    assert np.allclose(P2, base, atol=1e-12)


def test_frobenius_scale_option():
    n = 16
    lam = _head_spectrum(n, 2)
    Z, q = _sym_with_spectrum(lam)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 2)
    _, _, _, _, scale = oracle.psd_project(Z, q[:, :2], 2, coeffs, norm_mode=oracle.NORM_FROBENIUS)
    assert np.isclose(scale, np.sqrt((lam[2:] ** 2).sum()), rtol=1e-10)
