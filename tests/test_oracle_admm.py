"""Pins for the oracle's ADMM loop (Appendix E.1 "ADMM for Standard-Form SDP" iteration, Appendix E.4, "Experimental Details" residual terms): an analytically built KKT
point must be a fixed point, a 2 x 2 instance has a closed-form optimum, and on small max-cut instances the loop with
LAPACK's exact projection must drive the optimality conditions of the SDP pair to zero. Nothing expected here comes
from the oracle."""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(260923)


def _exact_projection(Z, warmup=False):
    w, v = np.linalg.eigh(0.5 * (Z + Z.T))
    return (v * np.maximum(w, 0.0)) @ v.T


def _kkt_point(n, r):
    """(C, b, X*, S*, y*) with X*, S* PSD, X* S* = 0, diag(X*) = b, C = S* + Diag(y*): optimal by construction."""
    q, _ = np.linalg.qr(RNG.standard_normal((n, n)))
    X = (q[:, :r] * RNG.uniform(0.5, 2.0, r)) @ q[:, :r].T
    S = (q[:, r:] * RNG.uniform(0.5, 2.0, n - r)) @ q[:, r:].T
    y = RNG.standard_normal(n)
    return S + np.diag(y), np.diag(X).copy(), X, S, y


@pytest.mark.parametrize("sigma", [0.5, 1.0, 3.0])
def test_kkt_point_is_a_fixed_point(sigma):
    C, b, X, S, y = _kkt_point(12, 4)
    X1, S1, y1, res = oracle.admm_diag_sdp(C, b, sigma, 3, X, S, _exact_projection)
    assert np.allclose(X1, X, atol=1e-10) and np.allclose(S1, S, atol=1e-10) and np.allclose(y1, y, atol=1e-10)
    assert np.all(res < 1e-10)


def test_two_by_two_closed_form():
    # min 2 c x  s.t.  [[1, x], [x, 1]] PSD  <=>  |x| <= 1: x* = -sign(c), value -2 |c|
    for c in (0.7, -1.3):
        C = np.array([[0.0, c], [c, 0.0]])
        X, S, y, res = oracle.admm_diag_sdp(C, np.ones(2), 1.0, 400, np.zeros((2, 2)), np.zeros((2, 2)), _exact_projection)
        assert np.allclose(X, [[1.0, -np.sign(c)], [-np.sign(c), 1.0]], atol=1e-6)
        assert abs(np.sum(C * X) + 2 * abs(c)) < 1e-6
        assert np.all(res[-1] < 1e-6)


def test_small_maxcut_reaches_the_optimality_conditions():
    n = 16
    A = np.triu((RNG.uniform(size=(n, n)) < 0.4).astype(float), 1)
    A = A + A.T
    C = -0.25 * (np.diag(A.sum(1)) - A)              # max-cut: min <-L/4, X>
    b = np.ones(n)
    X, S, y, res = oracle.admm_diag_sdp(C, b, 1.0, 3000, np.zeros((n, n)), np.zeros((n, n)), _exact_projection)
    # primal and dual feasibility, zero gap, complementarity, cone membership: the SDP pair's optimality conditions
    assert np.linalg.norm(np.diag(X) - b) < 1e-6
    assert np.linalg.norm(np.diag(y) + S - C) < 1e-6
    assert abs(np.sum(C * X) - b @ y) < 1e-5
    assert np.linalg.eigvalsh(X).min() > -1e-8 and np.linalg.eigvalsh(S).min() > -1e-8
    assert abs(np.sum(X * S)) < 1e-5
    # the residual terms reported are those quantities, normalised as in Appendix E.4, "Experimental Details"
    assert np.isclose(res[-1, 0], np.linalg.norm(np.diag(X) - b) / (1 + np.linalg.norm(b)), atol=1e-12)
    assert res[-1].max() < 1e-6 and res[0].max() > 1e-2
    # the value is bounded by the trivial cut bounds: every edge cut gives -|E|, and the SDP relaxes max-cut
    assert -A.sum() / 2 - 1e-6 <= np.sum(C * X) <= 0.0


def test_filter_projection_inside_the_loop_matches_the_exact_loop():
    """With the filter-based projection of Eq. 7 as the S-update (k = 0, classical quintic, many steps: the filter
    is the sign function to rounding on every eigenvalue that matters) the loop must follow the loop with LAPACK's
    projection. (With deflation the projection is exact only for exact eigenpairs, Proposition 2, so that case is
    left to the projection's own pins.)"""
    n = 24
    A = np.triu((RNG.uniform(size=(n, n)) < 0.5).astype(float), 1)
    A = A + A.T
    C = -0.25 * (np.diag(A.sum(1)) - A)
    b = np.ones(n)
    v0 = RNG.standard_normal(n)

    def proj(Z, warm):
        return oracle.psd_project(Z, None, 0, [oracle.CLASSICAL_QUINTIC] * 60, lanczos_v0=v0)[0]
    Xd, Sd, yd, rd = oracle.admm_diag_sdp(C, b, 1.0, 12, np.zeros((n, n)), np.zeros((n, n)), proj)
    Xe, Se, ye, re = oracle.admm_diag_sdp(C, b, 1.0, 12, np.zeros((n, n)), np.zeros((n, n)), _exact_projection)
    assert np.linalg.norm(Xd - Xe) <= 1e-6 * np.linalg.norm(Xe)
    assert np.linalg.norm(Sd - Se) <= 1e-6 * np.linalg.norm(Se)
    assert np.allclose(rd, re, atol=1e-7)
