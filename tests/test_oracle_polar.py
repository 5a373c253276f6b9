"""Pins for the polar side of the oracle: what the paper prints and what the mathematics fixes.

None of the expected values below comes from the oracle itself: they are the paper's printed
numbers (tests/golden), closed forms, or numpy/LAPACK factorizations used as brute force.
"""
import os

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(2609)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            out[parts[0]] = [float(x) for x in parts[1:]]
    return out


def _haar(rows, cols):
    q, r = np.linalg.qr(RNG.standard_normal((rows, cols)))
    return q * np.sign(np.diag(r))[None, :]


def _polar(M):
    u, s, vt = np.linalg.svd(M, full_matrices=False)
    keep = s > 1e-12 * s[0]
    return u[:, keep] @ vt[keep]


def _p_quintic(x, coeffs, L):
    a, b, c = coeffs
    for _ in range(L):
        x = a * x + b * x ** 3 + c * x ** 5
    return x


# ---------------------------------------------------------------------------------------------
# Coefficients: Eq. 2's printed triple and the closed form of Appendix B (proof of Theorem 1)
# ---------------------------------------------------------------------------------------------
def test_bjorck_bowie_reproduces_printed_quintic():
    g = _golden("classical_quintic.txt")
    a = oracle.bjorck_bowie(2)
    assert np.allclose(a, [g["a"][0], g["b"][0], g["c"][0]], atol=1e-15)


@pytest.mark.parametrize("d", [1, 2, 3, 4])
def test_bjorck_bowie_is_x_times_h_of_one_minus_x2(d):
    # Lemma 1: p_d(x) = x h_d(1 - x^2), h_d(z) = sum_j 4^-j C(2j,j) z^j (truncated series of z -> (1-z)^-1/2)
    from math import comb
    a = oracle.bjorck_bowie(d)
    x = np.linspace(0, 1, 41)
    p = sum(a[i] * x ** (2 * i + 1) for i in range(d + 1))
    h = sum(comb(2 * j, j) / 4.0 ** j * (1 - x ** 2) ** j for j in range(d + 1))
    assert np.allclose(p, x * h, atol=1e-14)
    # Lemma 1's residual identity 1 - p^2 = (1-x^2)^{d+1} omega_d(1-x^2)
    cj = [comb(2 * j, j) / 4.0 ** j for j in range(d + 1)]
    z = 1 - x ** 2
    omega = (2 * d + 1) * cj[d] * sum(cj[j] / (d + j + 1) * z ** j for j in range(d + 1))
    assert np.allclose(1 - p ** 2, z ** (d + 1) * omega, atol=1e-14)
    # and p_d(1) = 1 (one is a fixed point), slope at 0 is a_0
    assert np.isclose(a.sum(), 1.0)


# ---------------------------------------------------------------------------------------------
# Example 1: the printed numbers
# ---------------------------------------------------------------------------------------------
def test_example1_printed_values():
    g = _golden("example1.txt")
    sig = np.array(g["sigma"])
    U, V = _haar(8, 5), _haar(5, 5)
    M = (U * sig) @ V.T
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 5)

    def close(val, key):
        ref, half = g[key]
        assert abs(val - ref) <= half * 1.0000001, (key, val, ref)

    # undeflated: X0 = M/||M||_F, five classical steps
    out0, k0, rho0 = oracle.alg1(M, None, None, None, coeffs)
    assert k0 == 0
    close(rho0, "frob_M")
    close(sig[4] / rho0, "floor_base")
    s_out0 = np.linalg.svd(out0, compute_uv=False)
    close(s_out0.min(), "sigma5_base_after_5")
    # deflate sigma_1 exactly, no padding (gamma = 1), restore by addition (Eq. 3)
    out1, k1, rho1 = oracle.alg1(M, U[:, :1], sig[:1], V[:, :1], coeffs, gamma=1.0, mode=oracle.ADD)
    assert k1 == 1
    close(rho1, "frob_R1")
    close(rho0 / rho1, "alpha_1")
    close(sig[4] / rho1, "floor_deflated")
    s_out1 = np.linalg.svd(out1, compute_uv=False)
    close(s_out1.min(), "sigma5_deflated_after_5")
    # the padded form of Algorithm 1 with gamma = 1 gives the same matrix when the head is exact
    out2, _, _ = oracle.alg1(M, U[:, :1], sig[:1], V[:, :1], coeffs, gamma=1.0, mode=oracle.PADDED)
    assert np.allclose(out1, out2, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# The filter acts on singular values only (proof of Theorem 1, scalarisation)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,n", [(12, 30), (30, 12), (16, 16)])
@pytest.mark.parametrize("coeffs", [oracle.CLASSICAL_QUINTIC, oracle.MUON_QUINTIC])
def test_filter_maps_singular_values(m, n, coeffs):
    r = min(m, n)
    U, V = _haar(m, r), _haar(n, r)
    x = np.sort(RNG.uniform(0.01, 1.0, r))[::-1]
    X0 = (U * x) @ V.T
    L = 4
    XL = oracle.filter_quintic(X0, oracle.schedule(coeffs, L))
    D = U.T @ XL @ V
    assert np.allclose(D, np.diag(_p_quintic(x, coeffs, L)), atol=1e-11)


def test_filter_per_step_schedule_is_applied_in_order():
    sched = np.array([[3.0, -3.2, 1.2], [2.0, -1.5, 0.5], [1.875, -1.25, 0.375]])
    U, V = _haar(9, 6), _haar(6, 6)
    x = np.linspace(0.9, 0.05, 6)
    XL = oracle.filter_quintic((U * x) @ V.T, sched)
    y = x.copy()
    for a, b, c in sched:
        y = a * y + b * y ** 3 + c * y ** 5
    assert np.allclose(U.T @ XL @ V, np.diag(y), atol=1e-12)
    # reversed order gives a different answer, so the order matters and is tested
    y2 = x.copy()
    for a, b, c in sched[::-1]:
        y2 = a * y2 + b * y2 ** 3 + c * y2 ** 5
    assert not np.allclose(y, y2, atol=1e-6)


@pytest.mark.parametrize("d", [1, 2, 3])
def test_filter_classical_general_degree(d):
    U, V = _haar(10, 7), _haar(7, 7)
    x = np.linspace(0.95, 0.1, 7)
    XL = oracle.filter_classical((U * x) @ V.T, d, 3)
    a = oracle.bjorck_bowie(d)
    y = x.copy()
    for _ in range(3):
        y = sum(a[i] * y ** (2 * i + 1) for i in range(d + 1))
    assert np.allclose(U.T @ XL @ V, np.diag(y), atol=1e-12)


# ---------------------------------------------------------------------------------------------
# Eq. 3 and Theorem 1 against a brute-force polar factor
# ---------------------------------------------------------------------------------------------
def _head_dominated(m, n, k):
    r = min(m, n)
    sig = np.concatenate([np.linspace(80, 40, k), np.sort(10.0 ** RNG.uniform(-1.5, 0, r - k))[::-1]])
    U, V = _haar(m, r), _haar(n, r)
    return (U * sig) @ V.T, U, sig, V


@pytest.mark.parametrize("m,n", [(24, 40), (40, 24)])
@pytest.mark.parametrize("mode", [oracle.PADDED, oracle.ADD])
def test_exact_deflation_converges_to_polar(m, n, mode):
    k = 3
    M, U, sig, V = _head_dominated(m, n, k)
    # 16 steps: enough for the floor (about 0.015) to reach one, few enough that rounding noise
    # along the removed directions (amplified by 1.875 per step in ADD mode) stays negligible
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 16)
    out, kk, rho = oracle.alg1(M, U[:, :k], sig[:k], V[:, :k], coeffs, gamma=1.01, mode=mode)
    assert kk == k
    assert np.isclose(rho, np.sqrt((sig[k:] ** 2).sum()), rtol=1e-12)
    assert np.allclose(out, _polar(M), atol=1e-9)
    # Eq. 3: polar(M) = U_k V_k^T + polar(R_k), checked with LAPACK only
    R = M - (U[:, :k] * sig[:k]) @ V[:, :k].T
    assert np.allclose(_polar(M), U[:, :k] @ V[:, :k].T + _polar(R), atol=1e-10)


@pytest.mark.parametrize("L", [0, 1, 3, 5])
@pytest.mark.parametrize("gamma", [1.0, 1.01, 1.1])
def test_theorem1_scalarised_error_and_ratio_bound(L, gamma):
    m, n, k, d = 20, 32, 2, 2
    M, U, sig, V = _head_dominated(m, n, k)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, L) if L else np.zeros((0, 3))
    P = _polar(M)
    base, _, nf = oracle.alg1(M, None, None, None, coeffs)
    defl, _, rho = oracle.alg1(M, U[:, :k], sig[:k], V[:, :k], coeffs, gamma=gamma, mode=oracle.PADDED)
    ell = sig[-1] / nf
    alpha = nf / rho
    phi = min(alpha * ell, 1.0 / gamma)
    err_base = np.linalg.norm(P - base, 2)
    err_defl = np.linalg.norm(P - defl, 2)
    # equality: error = 1 - p^L(floor)
    assert np.isclose(err_base, 1 - _p_quintic(ell, oracle.CLASSICAL_QUINTIC, L), atol=1e-10)
    assert np.isclose(err_defl, 1 - _p_quintic(phi, oracle.CLASSICAL_QUINTIC, L), atol=1e-10)
    # bounds
    assert err_defl <= (1 - phi ** 2) ** ((d + 1) ** L) + 1e-12
    assert err_defl / err_base <= ((1 - phi ** 2) / (1 - ell ** 2)) ** ((d + 1) ** L) + 1e-12
    assert err_defl < err_base


def test_gate_semantics():
    m, n = 18, 30
    M, U, sig, V = _head_dominated(m, n, 3)
    coeffs = oracle.schedule(oracle.MUON_QUINTIC, 5)
    r = 6
    # gate fires (s_r/s_1 < tau): k = #{s_i > tau s_1}
    tau = 0.1
    out, k, _ = oracle.alg1(M, U[:, :r], sig[:r], V[:, :r], coeffs, tau=tau)
    assert k == int((sig[:r] > tau * sig[0]).sum()) == 3
    ref, _, _ = oracle.alg1(M, U[:, :3], sig[:3], V[:, :3], coeffs)
    assert np.array_equal(out, ref)
    # gate does not fire: reduces exactly to the plain filter
    out2, k2, nf = oracle.alg1(M, U[:, :2], sig[:2], V[:, :2], coeffs, tau=tau)
    assert k2 == 0
    plain = oracle.filter_quintic(M / np.linalg.norm(M), coeffs)   # numpy's norm sums in another order
    assert np.allclose(out2, plain, rtol=0, atol=1e-13)
    assert np.isclose(nf, np.linalg.norm(M))
    # and it is bit-identical to passing no triplets at all
    out3, _, _ = oracle.alg1(M, None, None, None, coeffs)
    assert np.array_equal(out2, out3)


# ---------------------------------------------------------------------------------------------
# Algorithm 3
# ---------------------------------------------------------------------------------------------
def test_brsvd_invariants_and_sandwich_bound():
    rows, cols, k, p, J = 60, 40, 4, 4, 1
    sig = np.concatenate([[50, 30, 20, 12], np.sort(RNG.uniform(0.05, 1.0, cols - 4))[::-1]])
    Uex, Vex = _haar(rows, cols), _haar(cols, cols)
    A = (Uex * sig) @ Vex.T
    l = k + p
    Om = RNG.standard_normal((cols, l))
    U, s, V = oracle.brsvd(A, Om, J)
    assert np.allclose(U.T @ U, np.eye(l), atol=1e-12)
    assert np.allclose(V.T @ V, np.eye(l), atol=1e-12)
    assert np.all(np.diff(s) <= 1e-14) and np.all(s >= 0)
    # U diag(s) V^T = Q Q^T A with Q = span(U): residual norm identity
    res = A - (U * s) @ V.T
    assert np.isclose(np.linalg.norm(res) ** 2, np.linalg.norm(A) ** 2 - (s ** 2).sum(), rtol=1e-10)
    assert np.allclose(U.T @ A, (V * s).T, atol=1e-11)
    # sandwich bound on the singular values with the actual sketch (Appendix D, "Bounds for randomized subspace iteration")
    Om1 = Vex[:, :k].T @ Om
    Om2 = Vex[:, k:].T @ Om
    c = np.linalg.norm(Om2 @ np.linalg.pinv(Om1), 2)
    for i in range(k):
        lo = sig[i] / np.sqrt(1 + (sig[k] / sig[i]) ** (2 * (2 * J + 1)) * c ** 2)
        assert sig[i] * (1 + 1e-12) >= s[i] >= lo * (1 - 1e-12)


def test_brsvd_many_iterations_recover_exact_head():
    rows, cols, k = 48, 30, 3
    sig = np.concatenate([[20, 10, 5], np.linspace(1.0, 0.1, cols - 3)])
    Uex, Vex = _haar(rows, cols), _haar(cols, cols)
    A = (Uex * sig) @ Vex.T
    U, s, V = oracle.brsvd(A, RNG.standard_normal((cols, k + 3)), 12)
    assert np.allclose(s[:k], sig[:k], rtol=1e-10)
    H = (U[:, :k] * s[:k]) @ V[:, :k].T
    assert np.allclose(H, (Uex[:, :k] * sig[:k]) @ Vex[:, :k].T, atol=1e-8)


def test_brsvd_full_width_is_exact_svd():
    # l = cols: the sketch spans everything, Q Q^T A = A and the triplets are the SVD
    rows, cols = 20, 6
    A = RNG.standard_normal((rows, cols))
    U, s, V = oracle.brsvd(A, RNG.standard_normal((cols, cols)), 0)
    assert np.allclose(s, np.linalg.svd(A, compute_uv=False), rtol=1e-11)
    assert np.allclose((U * s) @ V.T, A, atol=1e-12)


@pytest.mark.parametrize("m,n", [(36, 20), (20, 36)])
def test_deflated_polar_orientation_and_accuracy(m, n):
    k, p, J = 3, 3, 2
    M, U, sig, V = _head_dominated(m, n, k)
    ms = min(m, n)
    Om = RNG.standard_normal((ms, k + p))
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 30)
    out, s, kk, rho = oracle.deflated_polar(M, k, k + p, Om, J, coeffs, gamma=1.01)
    assert kk == k
    assert np.allclose(s[:k], sig[:k], rtol=1e-3)
    assert np.allclose(out, _polar(M), atol=1e-6)
    # transposing the input transposes the output (the sketch lives on the short side either way)
    outT, *_ = oracle.deflated_polar(M.T.copy(), k, k + p, Om, J, coeffs, gamma=1.01)
    assert np.allclose(outT, out.T, atol=1e-12)
    # k = 0 is the plain filter
    plain, _, k0, nf = oracle.deflated_polar(M, 0, 0, None, 0, coeffs)
    assert k0 == 0 and np.isclose(nf, np.linalg.norm(M))
    assert np.array_equal(plain, oracle.filter_quintic(M / np.linalg.norm(M), coeffs)) or \
        np.allclose(plain, oracle.filter_quintic(M / np.linalg.norm(M), coeffs), atol=1e-13)


def test_deflation_lowers_error_on_head_dominated_input_with_estimated_head():
    # Theorem 1's statement with the randomized-SVD estimate in place of exact triplets, classical map, L = 5
    m, n, k = 32, 48, 3
    M, *_ = _head_dominated(m, n, k)
    coeffs = oracle.schedule(oracle.CLASSICAL_QUINTIC, 5)
    P = _polar(M)
    base, *_ = oracle.deflated_polar(M, 0, 0, None, 0, coeffs)
    defl, *_ = oracle.deflated_polar(M, k, k + 4, RNG.standard_normal((m, k + 4)), 1, coeffs, gamma=1.01)
    assert np.linalg.norm(P - defl, 2) < np.linalg.norm(P - base, 2)
    assert np.linalg.norm(P - defl) < np.linalg.norm(P - base)
