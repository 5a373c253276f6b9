"""Coefficient schedules for the fixed polynomial filter (host side, fp64, numpy only; no GPU, no oracle).

* `bjorck_bowie(d)`: the classical Newton-Schulz map N_d of Eq. 2 (closed form in Appendix B, the proof of Theorem 1), as odd-power
  coefficients; d = 2 gives (15/8, -5/4, 3/8).
* `remez_sign_schedule(eps, T)`: stage one of the composite minimax sign filter (Appendix E.2, "Composite Minimax Filter"): T odd quintics
  g_t(x) = a x + b x^3 + c x^5, g_t the best uniform approximation of 1 on [a_t, b_t], [a_1, b_1] = [eps, 1],
  [a_{t+1}, b_{t+1}] = g_t([a_t, b_t]). The composition g_T o ... o g_1 approximates sign(x) on
  [-1, -eps] u [eps, 1]. (Stage two, the joint gradient refinement for the ReLU error, is not implemented.)

A schedule is a list of (a, b, c) triples, the form every entry point of the library takes.
"""
import math

import numpy as np


def bjorck_bowie(d):
    """Coefficients (c_1, c_3, ..., c_{2d+1}) of N_d(x) = x sum_{j<=d} binom(2j, j) / 4^j (1 - x^2)^j."""
    poly = np.zeros(d + 1)                      # in powers of u = x^2
    one_minus_u = np.array([1.0])
    for j in range(d + 1):
        w = math.comb(2 * j, j) / 4.0 ** j
        poly[: len(one_minus_u)] += w * one_minus_u
        one_minus_u = np.convolve(one_minus_u, [1.0, -1.0])
    return tuple(float(x) for x in poly)


def _quintic(coef, x):
    a, b, c = coef
    x2 = x * x
    return x * (a + x2 * (b + x2 * c))


def _interior_extrema(coef, lo, hi):
    """Points of (lo, hi) where g'(x) = a + 3 b x^2 + 5 c x^4 vanishes (a quadratic in x^2)."""
    a, b, c = coef
    roots = np.roots([5.0 * c, 3.0 * b, a]) if c != 0.0 else (np.array([-a / (3.0 * b)]) if b != 0.0 else np.array([]))
    out = []
    for u in roots:
        if abs(u.imag) < 1e-14 * max(1.0, abs(u)) and u.real > 0.0:
            x = math.sqrt(u.real)
            if lo < x < hi:
                out.append(x)
    return sorted(out)


def minimax_odd_quintic(lo, hi, iters=100):
    """Best uniform approximation of the constant 1 on [lo, hi] (0 < lo < hi) by an odd quintic, by Remez
    exchange: the error g - 1 equioscillates at four points. Returns ((a, b, c), E) with E = max |g - 1|."""
    if not (0.0 < lo < hi):
        raise ValueError("need 0 < lo < hi")
    # start from Chebyshev points of the interval
    ref = np.array([0.5 * (lo + hi) - 0.5 * (hi - lo) * math.cos(math.pi * i / 3.0) for i in range(4)])
    coef, err = (1.0, 0.0, 0.0), 0.0
    for _ in range(iters):
        # g(x_i) - 1 = (-1)^i E  for the four reference points: linear in (a, b, c, E)
        M = np.stack([ref, ref ** 3, ref ** 5, -np.array([(-1.0) ** i for i in range(4)])], axis=1)
        a, b, c, err = np.linalg.solve(M, np.ones(4))
        coef = (float(a), float(b), float(c))
        # the error's extrema on [lo, hi]: the end points and the interior stationary points
        cand = [lo] + _interior_extrema(coef, lo, hi) + [hi]
        if len(cand) != 4:
            break                                   # degenerate (tiny interval): the reference is as good as it gets
        new = np.array(cand)
        vals = _quintic(coef, new) - 1.0
        if np.max(np.abs(np.abs(vals) - abs(err))) <= 1e-15 * max(1.0, abs(err)) + 1e-16 or np.allclose(new, ref, rtol=0, atol=1e-16):
            ref = new
            break
        ref = new
    grid = np.linspace(lo, hi, 20001)
    return coef, float(np.max(np.abs(_quintic(coef, grid) - 1.0)))


def remez_sign_schedule(eps=1e-3, T=7, margin=0.0):
    """Stage one of Appendix E.2, "Composite Minimax Filter": [(a_t, b_t, c_t)] for t = 1..T and the per-stage errors max |g_t - 1| on [a_t, b_t].

    Unlike the classical map, these polynomials are only meant for |x| <= 1: an input eigenvalue slightly above 1
    (the Lanczos scale of Appendix E.1, "Normalization scale" is a heuristic upper estimate) leaves the next stage's interval and the
    composition diverges. `margin` > 0 composes the first stage with x / (1 + margin), i.e. the schedule then
    covers [-(1 + margin), 1 + margin] and approximates the sign function from eps (1 + margin) on."""
    lo, hi = float(eps), 1.0
    sched, errs = [], []
    for _ in range(T):
        if hi - lo < 1e-9:                       # the interval has collapsed on 1: the limit is the classical quintic
            coef, e = bjorck_bowie(2), 0.0
        else:
            coef, e = minimax_odd_quintic(lo, hi)
        sched.append(coef)
        errs.append(e)
        # g_t is not monotone on the interval: its image is [1 - E, 1 + E] by equioscillation
        grid = np.linspace(lo, hi, 20001)
        vals = _quintic(coef, grid)
        lo, hi = float(vals.min()), float(vals.max())
    if margin > 0.0:
        a, b, c = sched[0]
        m = 1.0 + float(margin)
        sched[0] = (a / m, b / m ** 3, c / m ** 5)
    return sched, errs


def compose(schedule, x):
    """(g_T o ... o g_1)(x) for an array x."""
    y = np.array(x, dtype=np.float64)
    for coef in schedule:
        y = _quintic(coef, y)
    return y
