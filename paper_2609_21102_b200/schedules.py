"""Coefficient schedules for the fixed polynomial filter (host side, fp64, numpy and scipy; no GPU, no oracle).

* `bjorck_bowie(d)`: the classical Newton-Schulz map N_d of Eq. 2 (closed form in Appendix B, the proof of Theorem 1), as odd-power
  coefficients; d = 2 gives (15/8, -5/4, 3/8).
* `remez_sign_schedule(eps, T)`: stage one of the composite minimax sign filter (Appendix E.2, "Composite Minimax Filter"): T odd quintics
  g_t(x) = a x + b x^3 + c x^5, g_t the best uniform approximation of 1 on [a_t, b_t], [a_1, b_1] = [eps, 1],
  [a_{t+1}, b_{t+1}] = g_t([a_t, b_t]). The composition g_T o ... o g_1 approximates sign(x) on
  [-1, -eps] u [eps, 1].
* `stage_two_schedule(eps, T)` / `refine_relu_schedule(schedule)`: stage two of the same appendix: the coefficients of all T quintics are refined
  jointly, by descent steps linearised through the composition, to lower max over [-1, 1] of
  |x/2 (1 + (p_T o ... o p_1)(x)) - max(x, 0)| evaluated on a dense grid; the composite form is kept.
* `deflated_interval_schedule(lam_min, theta_k, T)`: the filter of Theorem 3, the same sequential construction started
  on the deflated interval [a_k, 1], a_k = |lambda_q| / theta_k, with the theorem's bound (1 - a_k^2)^(3^T).

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


def relu_error(schedule, grid=None):
    """max over the grid of |x/2 (1 + g(x)) - max(x, 0)| for g = p_T o ... o p_1 (the matrix-ReLU error of the
    projection P = Z (I + g(Z / theta)) / 2 per unit of theta); the default grid is 40001 points of [-1, 1]."""
    x = np.linspace(-1.0, 1.0, 40001) if grid is None else np.asarray(grid, dtype=np.float64)
    return float(np.max(np.abs(0.5 * x * (1.0 + compose(schedule, x)) - np.maximum(x, 0.0))))


def _compose_with_gradient(coefs, x):
    """g(x) and d g(x) / d coefs[t][i] for every stage t and coefficient i, by the chain rule through the
    composition: returns (g, grad) with grad of shape [T, 3, len(x)]."""
    T = len(coefs)
    ys = [np.array(x, dtype=np.float64)]
    for a, b, c in coefs:
        ys.append(_quintic((a, b, c), ys[-1]))
    grad = np.zeros((T, 3, len(ys[0])))
    back = np.ones_like(ys[0])                       # d g / d y_{t+1}, walking from the last stage to the first
    for t in range(T - 1, -1, -1):
        y = ys[t]
        y2 = y * y
        grad[t, 0], grad[t, 1], grad[t, 2] = back * y, back * y * y2, back * y * y2 * y2
        a, b, c = coefs[t]
        back = back * (a + y2 * (3.0 * b + y2 * 5.0 * c))
    return ys[-1], grad


def stage_two_schedule(eps=1e-3, T=7, iters=20, grid=None):
    """The two-stage construction in one call: stage one on [eps, 1], then stage two. Stage two has two parts here.
    (a) The sign-optimal composite is far more accurate on [eps, 1] than the matrix ReLU needs (1e-9 for eps = 1e-3,
    T = 7) while the ReLU error comes from the zone |x| < eps that it leaves out: re-running stage one from a smaller
    left end trades the one for the other, and a golden-section search over that left end (between eps / 10 and eps)
    picks the composite with the smallest ReLU error. (b) refine_relu_schedule polishes all coefficients jointly.
    Returns (schedule, relu_error_stage_one, relu_error_stage_two)."""
    x = (np.sort(np.concatenate([np.linspace(-1.0, 1.0, 40001), np.linspace(-2.0 * eps, 2.0 * eps, 20001)]))
         if grid is None else np.asarray(grid, dtype=np.float64))
    s1, _ = remez_sign_schedule(eps, T)
    e1 = relu_error(s1, x)
    f = lambda le: relu_error(remez_sign_schedule(math.exp(le), T)[0], x)
    lo, hi = math.log(eps / 10.0), math.log(eps)
    ratio = 0.5 * (math.sqrt(5.0) - 1.0)
    c, d = hi - ratio * (hi - lo), lo + ratio * (hi - lo)
    fc, fd = f(c), f(d)
    for _ in range(18):
        if fc < fd:
            hi, d, fd = d, c, fc
            c = hi - ratio * (hi - lo)
            fc = f(c)
        else:
            lo, c, fc = c, d, fd
            d = lo + ratio * (hi - lo)
            fd = f(d)
    le = c if fc < fd else d
    best, eb = (remez_sign_schedule(math.exp(le), T)[0], min(fc, fd)) if min(fc, fd) < e1 else (s1, e1)
    s2, _, e2 = refine_relu_schedule(best, iters=iters, grid=x)
    return s2, e1, e2


def refine_relu_schedule(schedule, iters=40, grid=None, radius=1e-3):
    """Stage two of the composite filter: jointly refine all coefficients to lower the matrix-ReLU error
    max |x/2 (1 + g(x)) - max(x, 0)| on a dense grid of [-1, 1], keeping g = p_T o ... o p_1.

    Descent on the maximum itself by sequential linear programming: the error is linearised in the 3T coefficients
    (gradient through the composition), the linear minimax problem is solved inside a trust region of relative size
    `radius` per coefficient (the composition is stiff: a change of a percent in an early coefficient sends the later
    stages outside the interval on which they contract), and the step is kept only if the true maximum falls, so the
    result is never worse than the input schedule. Returns (schedule, error_before, error_after)."""
    from scipy.optimize import linprog
    x = np.linspace(-1.0, 1.0, 40001) if grid is None else np.asarray(grid, dtype=np.float64)
    target = np.maximum(x, 0.0)
    coefs = np.array([list(c) for c in schedule], dtype=np.float64)
    nvar = coefs.size

    def errors(cf):
        with np.errstate(over="ignore", invalid="ignore"):
            return 0.5 * x * (1.0 + compose([tuple(r) for r in cf], x)) - target

    best = float(np.max(np.abs(errors(coefs))))
    first = best
    for _ in range(iters):
        g, grad = _compose_with_gradient([tuple(r) for r in coefs], x)
        e = 0.5 * x * (1.0 + g) - target
        J = (grad.reshape(nvar, -1) * (0.5 * x)).T                      # [points, 3T]
        keep = np.abs(e) >= 0.2 * best
        keep[::25] = True                                               # a coarse net over the rest of the interval
        Jk, ek = J[keep], e[keep]
        ones = np.ones((len(ek), 1))
        A_ub = np.block([[Jk, -ones], [-Jk, -ones]])
        b_ub = np.concatenate([-ek, ek])
        lim = radius * np.maximum(np.abs(coefs.reshape(-1)), 1e-6)
        bounds = [(-l, l) for l in lim] + [(0.0, None)]
        sol = linprog(np.concatenate([np.zeros(nvar), [1.0]]), A_ub=A_ub, b_ub=b_ub, bounds=bounds, method="highs")
        if not sol.success:
            break
        trial = coefs + sol.x[:nvar].reshape(coefs.shape)
        et = errors(trial)
        mt = float(np.max(np.abs(et))) if np.all(np.isfinite(et)) else np.inf
        if mt < best * (1.0 - 1e-9):
            coefs, best = trial, mt
            radius = min(radius * 2.0, 0.05)
        else:
            radius *= 0.25
            if radius < 1e-9:
                break
    return [tuple(float(v) for v in r) for r in coefs], first, best


def deflated_interval_schedule(lam_min, theta_k, T):
    """The filter of the idealised analysis (Theorem 3): the sequential minimax construction started on the deflated
    interval [a_k, 1], a_k = |lambda_q| / theta_k (smallest nonzero eigenvalue magnitude over the norm of the deflated
    residual), instead of [eps, 1]. Returns (schedule, per-stage errors, a_k, bound) with the theorem's bound
    (1 - a_k^2)^(3^T) on max |1 - g| over [a_k, 1] for quintic stages (d = 2)."""
    a_k = abs(float(lam_min)) / float(theta_k)
    if not (0.0 < a_k <= 1.0):
        raise ValueError("need 0 < |lambda_q| <= theta_k")
    sched, errs = remez_sign_schedule(a_k, T)
    return sched, errs, a_k, float((1.0 - a_k * a_k) ** (3.0 ** T))
