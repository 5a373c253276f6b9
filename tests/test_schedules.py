"""Pins for the schedule tools (Eq. 2 / closed form in Appendix B, the proof of Theorem 1; Appendix E.2, "Composite Minimax Filter" stage one): the printed classical
coefficients, the equioscillation that characterises a best uniform approximation, an independent linear-programming
solution of the same minimax problem, and the limits the construction must reach."""
import os

import numpy as np
import pytest
from scipy.optimize import linprog

from paper_2609_21102_b200 import schedules as S

GOLD = os.path.join(os.path.dirname(__file__), "golden", "classical_quintic.txt")


def test_bjorck_bowie_matches_the_printed_quintic_and_cubic():
    vals = [float(x) for line in open(GOLD) if line.strip() and not line.startswith("#") for x in line.split()[1:]]
    assert np.allclose(S.bjorck_bowie(2), vals[:3], rtol=0, atol=1e-15)
    assert S.bjorck_bowie(1) == (1.5, -0.5)                       # the cubic Newton-Schulz map
    for d in (1, 2, 3, 4):                                        # 1 is a fixed point with zero slope
        c = np.array(S.bjorck_bowie(d))
        powers = 2 * np.arange(d + 1) + 1
        assert abs(c.sum() - 1.0) < 1e-14                          # N_d(1) = 1
        assert abs((c * powers).sum()) < 1e-13                     # N_d'(1) = 0


@pytest.mark.parametrize("interval", [(1e-3, 1.0), (0.05, 1.4), (0.5, 1.1)])
def test_minimax_quintic_equioscillates_and_beats_linear_programming_grid(interval):
    lo, hi = interval
    coef, E = S.minimax_odd_quintic(lo, hi)
    x = np.linspace(lo, hi, 200001)
    err = S._quintic(coef, x) - 1.0
    assert abs(np.max(np.abs(err)) - E) < 1e-9
    # four alternating extrema of equal size (Chebyshev's criterion for 3 free coefficients)
    idx = [0] + [i for i in range(1, len(x) - 1) if (err[i] - err[i - 1]) * (err[i + 1] - err[i]) < 0] + [len(x) - 1]
    ext = err[idx]
    assert len(ext) == 4
    assert np.all(np.sign(ext[:-1]) == -np.sign(ext[1:]))
    assert np.allclose(np.abs(ext), E, rtol=1e-6)
    # the same problem as a linear programme on a grid: min E s.t. |a x + b x^3 + c x^5 - 1| <= E
    g = np.linspace(lo, hi, 2001)
    A = np.stack([g, g ** 3, g ** 5], axis=1)
    A_ub = np.block([[A, -np.ones((len(g), 1))], [-A, -np.ones((len(g), 1))]])
    b_ub = np.concatenate([np.ones(len(g)), -np.ones(len(g))])
    sol = linprog([0, 0, 0, 1], A_ub=A_ub, b_ub=b_ub, bounds=[(None, None)] * 4, method="highs")
    assert sol.success
    assert sol.x[3] <= E + 1e-9                     # a grid relaxes the problem
    assert E - sol.x[3] < 1e-4 * max(E, 1e-3)       # ... by next to nothing


def test_stage_one_schedule_reaches_the_sign_function():
    sched, errs = S.remez_sign_schedule(1e-3, 7)
    assert len(sched) == 7 and all(len(c) == 3 for c in sched)
    assert all(e2 < e1 for e1, e2 in zip(errs, errs[1:]))          # every stage tightens the interval around 1
    x = np.linspace(1e-3, 1.0, 100001)
    y = S.compose(sched, x)
    assert np.max(np.abs(y - 1.0)) < 1e-8
    assert np.allclose(S.compose(sched, -x), -y)                     # odd: -1 on the reflected interval
    # once the interval has collapsed on 1 the best approximation is the polynomial with the highest contact at 1
    assert np.allclose(sched[-1], S.bjorck_bowie(2), atol=1e-5)
    # seven classical steps from 1e-3 are nowhere near: 1e-3 * 1.875^7 = 0.08
    assert abs(S.compose([S.bjorck_bowie(2)] * 7, np.array([1e-3]))[0] - 1.0) > 0.9


def test_margin_rescales_the_first_stage_only():
    s0, _ = S.remez_sign_schedule(1e-3, 7)
    s1, _ = S.remez_sign_schedule(1e-3, 7, margin=0.02)
    assert s0[1:] == s1[1:]
    x = np.linspace(1.02e-3, 1.02, 50001)
    assert np.allclose(S.compose(s1, x), S.compose(s0, x / 1.02), rtol=0, atol=1e-12)
    assert np.max(np.abs(S.compose(s1, x) - 1.0)) < 1e-8           # valid up to 1.02 now
    with np.errstate(over="ignore", invalid="ignore"):          # without the margin 1.05 is outside the valid range
        far = S.compose(s0, np.array([1.05]))[0]
    assert not np.isfinite(far) or abs(far) > 10


def test_stage_two_lowers_the_relu_error_and_never_raises_it():
    """Stage two: the refined composite has a smaller matrix-ReLU error than stage one (whose error sits in the zone
    |x| < eps that the sign approximation leaves out, while it is 1e-9 accurate on [eps, 1], far more than the ReLU
    needs), a refinement step never raises the error, and the result is still an odd composite of T quintics."""
    eps, T = 1e-3, 7
    x = np.sort(np.concatenate([np.linspace(-1.0, 1.0, 40001), np.linspace(-2 * eps, 2 * eps, 20001)]))
    s1, errs = S.remez_sign_schedule(eps, T)
    e1 = S.relu_error(s1, x)
    assert errs[-1] < 1e-8
    # |x| (1 - g(|x|)) / 2 on [0, eps]: below eps / 2, and not tiny
    assert 1e-6 < e1 <= 0.5 * eps
    s2, before, after = S.stage_two_schedule(eps, T, iters=6)
    assert before == pytest.approx(e1)
    assert after == pytest.approx(S.relu_error(s2, x))
    assert after < 0.8 * before
    assert len(s2) == T and all(len(c) == 3 for c in s2)
    xs = np.linspace(-1.0, 1.0, 2001)
    assert np.allclose(S.compose(s2, -xs), -S.compose(s2, xs))
    # the polish alone: never worse than what it was given
    s3, b3, a3 = S.refine_relu_schedule(s1, iters=3, grid=x)
    assert b3 == pytest.approx(e1) and a3 <= b3


def test_gradient_through_the_composition_matches_finite_differences():
    sched, _ = S.remez_sign_schedule(1e-2, 3)
    x = np.array([-0.7, -0.01, 0.003, 0.2, 0.9])
    g, grad = S._compose_with_gradient(sched, x)
    assert np.allclose(g, S.compose(sched, x))
    for t in range(3):
        for i in range(3):
            h = 1e-6 * max(1.0, abs(sched[t][i]))
            up = [list(c) for c in sched]
            dn = [list(c) for c in sched]
            up[t][i] += h
            dn[t][i] -= h
            fd = (S.compose([tuple(c) for c in up], x) - S.compose([tuple(c) for c in dn], x)) / (2 * h)
            assert np.allclose(grad[t, i], fd, rtol=1e-5, atol=1e-7)


@pytest.mark.parametrize("a_k,T", [(0.05, 3), (0.2, 2), (0.01, 5)])
def test_filter_regenerated_on_the_deflated_interval_meets_theorem_3(a_k, T):
    """Theorem 3: started on [a_k, 1], the sequential minimax composite satisfies max |1 - g| <= (1 - a_k^2)^(3^T) on
    that interval (the classical composition meets the bound, the minimax one is at least as good), and raising the
    floor from eps to a_k, which is what deflation does, buys orders of magnitude at the same depth."""
    sched, errs, ak, bound = S.deflated_interval_schedule(a_k * 3.0, 3.0, T)
    assert ak == pytest.approx(a_k)
    x = np.linspace(a_k, 1.0, 100001)
    err = float(np.max(np.abs(S.compose(sched, x) - 1.0)))
    classical = float(np.max(np.abs(S.compose([S.bjorck_bowie(2)] * T, x) - 1.0)))
    assert classical <= bound * (1 + 1e-12) + 1e-15
    assert err <= classical + 1e-12
    assert err == pytest.approx(errs[-1], rel=1e-3, abs=1e-12)
    wide, _ = S.remez_sign_schedule(a_k / 50.0, T)
    xw = np.linspace(a_k / 50.0, 1.0, 100001)
    assert err < 0.5 * float(np.max(np.abs(S.compose(wide, xw) - 1.0)))
    with pytest.raises(ValueError):
        S.deflated_interval_schedule(2.0, 1.0, 3)
