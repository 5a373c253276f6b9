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
