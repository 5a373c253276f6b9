"""Sensitivity of the filter to the storage format of its iterate, evaluated with the oracle (test infrastructure).

The library keeps the filter's iterate X_t in a narrow format between steps (IEEE half scaled by 32, bf16, or fp32
rounded to tf32); the oracle keeps it in fp64. How far that rounding alone moves the result depends on the input
(its singular values below the filter's knee are multiplied by the first slope at every step) and on the restore
mode, not on any kernel. The functions here measure it on the oracle's side: the oracle's own filter step is applied
step by step and the iterate is rounded between steps the way the storage format demands. The distance between that
result and the oracle's unrounded result is the error the storage format explains; a parity test whose tolerance is
tied to it asserts that the kernels add nothing of that size on top.

Only numpy roundings and calls of the oracle; nothing here touches the CUDA library.
"""
import numpy as np

import oracle


def round_half_scaled(x, scale=32.0):
    """Values as an IEEE half buffer holding scale * x keeps them (round to nearest even, gradual underflow)."""
    with np.errstate(over="ignore"):
        return (np.asarray(x, dtype=np.float64) * scale).astype(np.float16).astype(np.float64) / scale


def round_bf16(x):
    return oracle.round_to_storage(x, "bf16")


def round_tf32(x):
    """fp32 values rounded to nearest (ties away from zero, as cvt.rna does) on 10 explicit mantissa bits."""
    x32 = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    bits = x32.view(np.uint32).astype(np.uint64)
    bits = ((bits + 0x1000) >> 13) << 13
    return bits.astype(np.uint32).view(np.float32).reshape(x32.shape).astype(np.float64)


ROUNDERS = {"half": round_half_scaled, "half1": lambda x: round_half_scaled(x, 1.0), "bf16": round_bf16, "tf32": round_tf32,
            "none": lambda x: np.asarray(x, dtype=np.float64)}


def filter_with_storage(X0, sched, formats):
    """p_L o ... o p_1 applied to X0 by the oracle's filter, one step per call, with the iterate rounded to
    formats[t] before step t+1 reads it (formats[0] is the storage of X0 itself); the last result is not rounded."""
    X = np.asarray(X0, dtype=np.float64)
    for t, c in enumerate(sched):
        X = ROUNDERS[formats[t]](X)
        X = oracle.filter_quintic(X, [list(c)])
    return X


def polar_filter_with_storage(X0, sched, formats, passes=None):
    """The filter of the bf16 polar path the way the path stores it: per step the iterate X, the short-side Gram matrix
    A = X X^T (or X^T X) and B = a I + b A + c A^2 are each rounded when written, to the step's format ("half": X is
    kept as 32 X and A as 1024 A in IEEE half, B unscaled; "bf16": plain bf16); products by the oracle's matmul, exact
    in between. `passes` (a list of 1s and 2s, see polar_passes) marks the steps that share one pass over X: there
    B_t^2, A_{t+1} = B_t^2 A_t, B_{t+1} and B_{t+1} B_t are formed on the short side, each rounded when written and with
    its upper triangle mirrored as the kernels mirror it, and X is multiplied once. The last result is not rounded."""
    X = np.asarray(X0, dtype=np.float64)
    m, n = X.shape
    wide = m <= n
    ms = min(m, n)
    mirror = lambda M: np.triu(M) + np.triu(M, 1).T
    t = 0
    for npass in (passes if passes is not None else [1] * len(sched)):
        a, b, c = sched[t]
        fmt = formats[t]
        rx = ROUNDERS[fmt]
        ra = (lambda v: round_half_scaled(v, 1024.0)) if fmt == "half" else rx
        rb = ROUNDERS["half1"] if fmt == "half" else rx
        X = rx(X)
        A = ra(oracle.matmul(X, X, tb=True) if wide else oracle.matmul(X, X, ta=True))
        B = rb(a * np.eye(ms) + b * A + c * oracle.matmul(A, A))
        if npass == 2:
            a1, b1, c1 = sched[t + 1]
            S = rb(mirror(oracle.matmul(B, B)))
            A1 = ra(mirror(oracle.matmul(S, A)))
            B1 = rb(a1 * np.eye(ms) + b1 * A1 + c1 * oracle.matmul(A1, A1))
            B = rb(mirror(oracle.matmul(B1, B)))
        X = oracle.matmul(B, X) if wide else oracle.matmul(X, B)
        t += npass
    return X


def polar_passes(m, n, sched, paired=None, option=0):
    """How the path walks the filter steps (1 = a step of its own, 2 = two steps in one pass over X): greedily from
    the first step, a pair starts at step t when there is a next step, |a_t| <= 4.5 and |b_{t+1} + 2 c_{t+1}| <= 1, provided the long side is at
    least twice the short one and the iterates are not bf16 throughout (option 1). `paired` False switches the pairing
    off (the fp32 engine, the knob)."""
    ms, ml = min(m, n), max(m, n)
    L = len(sched)
    if paired is False or option == 1 or ml < 2 * ms:
        return [1] * L
    out, t = [], 0
    while t < L:
        two = t + 1 < L and abs(sched[t][0]) <= 4.5 and abs(sched[t + 1][1] + 2.0 * sched[t + 1][2]) <= 1.0
        out.append(2 if two else 1)
        t += 2 if two else 1
    return out


def polar_formats(L, add_mode, option=0, passes=None):
    """Iterate storage of the bf16 polar path per step: option 0 = scaled half in the first two steps (every step in
    ADD mode; every step up to the last paired one where steps are paired), bf16 after; 1 = bf16 throughout; 2 = half
    throughout."""
    if option == 1:
        return ["bf16"] * L
    n_half = L if (option == 2 or add_mode) else min(L, 2)
    t = 0
    for q in (passes or []):
        t += q
        if q == 2:
            n_half = max(n_half, t)                 # both steps of a pair are kept in scaled half
    return ["half"] * n_half + ["bf16"] * (L - n_half)


def polar_entry(G, k, l, Omega, J, gamma, add_mode):
    """The oracle's filter input X0 for one matrix (Algorithm 3 then lines 3-4 of Algorithm 1), the head U_k V_k^T
    that ADD mode adds back, in the caller's orientation."""
    G = np.asarray(G, dtype=np.float64)
    m, n = G.shape
    tall = m >= n
    A = G if tall else G.T
    none = np.zeros((0, 3))
    if k == 0:
        out0, _, _ = oracle.alg1(A, None, None, None, none)
        return (out0 if tall else out0.T), np.zeros_like(G)
    U, s, V = oracle.brsvd(A, Omega, J)
    U, s, V = U[:, :k], s[:k], V[:, :k]
    head = U @ V.T
    out0, _, _ = oracle.alg1(A, U, s, V, none, gamma=gamma, mode=oracle.ADD if add_mode else oracle.PADDED)
    X0 = out0 - head if add_mode else out0        # with no filter steps ADD mode returns X0 + head
    return (X0 if tall else X0.T), (head if tall else head.T)


def polar_storage_error(G, k, l, Omega, J, sched, gamma, add_mode, option=0, round_output=False, paired=None):
    """Relative Frobenius distance between the oracle's result with the iterate rounded to the path's storage
    formats (and, with round_output, the result rounded to bf16 as the path returns it) and its result in fp64
    throughout: what the storage format alone explains for this input."""
    X0, head = polar_entry(G, k, l, Omega, J, gamma, add_mode)
    exact = oracle.filter_quintic(X0, sched) + (head if add_mode else 0.0)
    passes = polar_passes(np.shape(G)[0], np.shape(G)[1], sched, paired, option)
    stored = polar_filter_with_storage(X0, sched, polar_formats(len(sched), add_mode, option, passes), passes) + (head if add_mode else 0.0)
    if round_output:
        stored = round_bf16(stored)
    return float(np.linalg.norm(stored - exact) / np.linalg.norm(exact))


def psd_pieces(Z, Vb, k, gamma, warmup, lanczos_v0):
    """The quantities Algorithm 2 builds before and after its filter, from oracle primitives in the algorithm's order:
    Ritz pairs of the incoming basis, the deflated residual R, the Lanczos scale theta, the filter input X0 and the
    restored positive head. Returns (R, X0, head_plus)."""
    Z = np.asarray(Z, dtype=np.float64)
    n = Z.shape[0]
    idx = []
    if not warmup and k > 0 and Vb is not None and Vb.shape[1] > 0:
        Zt = oracle.matmul(Z, Vb)
        H = oracle.matmul(Vb, Zt, ta=True)
        H = 0.5 * (H + H.T)
        lam, E = oracle.jacobi_eig(H)
        U = oracle.matmul(Vb, E)
        order = sorted(range(len(lam)), key=lambda i: (-abs(lam[i]), i))
        idx = order[:k]
    R = Z.copy()
    for i in idx:
        R -= lam[i] * np.outer(U[:, i], U[:, i])
    theta = oracle.lanczos_upper(R, lanczos_v0)
    X0 = R / theta
    head_plus = np.zeros((n, n))
    for i in idx:
        X0 += np.sign(lam[i]) / gamma * np.outer(U[:, i], U[:, i])
        if lam[i] > 0:
            head_plus += lam[i] * np.outer(U[:, i], U[:, i])
    return R, X0, head_plus


def symmetric_filter_with_storage(X0, sched, fmt):
    """The symmetric filter the way the path stores it: per step W = X^2, T = a I + b W + c W^2, X <- X T, with X, W and
    T each rounded to `fmt` when written (products by the oracle's matmul, exact in between); the result is rounded to
    tf32, the type in which it enters the reconstruction product."""
    rnd = ROUNDERS[fmt]
    X = rnd(np.asarray(X0, dtype=np.float64))
    n = X.shape[0]
    for a, b, c in sched:
        W = rnd(oracle.matmul(X, X))
        T = rnd(a * np.eye(n) + b * W + c * oracle.matmul(W, W))
        X = oracle.matmul(X, T)
        X = rnd(np.triu(X) + np.triu(X, 1).T)          # the path computes the upper triangle and mirrors it
    return round_tf32(X)


def psd_storage_error(Z, Vb, k, sched, gamma, warmup, lanczos_v0, fmt):
    """Relative Frobenius distance between the projection with the filter's stored quantities rounded to `fmt` ("tf32",
    or "half1" for unscaled IEEE half) and the projection in fp64 throughout, both from the oracle's steps; also returns
    the unrounded projection (it must equal oracle.psd_project's)."""
    R, X0, head_plus = psd_pieces(Z, Vb, k, gamma, warmup, lanczos_v0)

    def project(gX):
        P = 0.5 * (R + oracle.matmul(R, gX)) + head_plus
        return 0.5 * (P + P.T)
    exact = project(oracle.filter_quintic(X0, sched))
    stored = project(symmetric_filter_with_storage(X0, sched, fmt))
    return float(np.linalg.norm(stored - exact) / np.linalg.norm(exact)), exact




def inv_root_pieces(A, Vb, k, gamma, warmup, lanczos_v0):
    """What the deflated inverse root builds before its iteration, from oracle primitives in its order: Ritz pairs of
    the incoming basis, the residual, the Lanczos scale and the padded, normalised X0. Returns (X0, theta, U_I, lam_I)
    with the removed Ritz vectors in the columns of U_I."""
    A = np.asarray(A, dtype=np.float64)
    n = A.shape[0]
    UI, lamI = np.zeros((n, 0)), np.zeros(0)
    if not warmup and k > 0 and Vb is not None and Vb.shape[1] > 0:
        H = oracle.matmul(Vb, oracle.matmul(A, Vb), ta=True)
        lam, E = oracle.jacobi_eig(0.5 * (H + H.T))
        U = oracle.matmul(Vb, E)
        idx = sorted(range(len(lam)), key=lambda i: (-abs(lam[i]), i))[:k]
        UI, lamI = U[:, idx], np.array([lam[i] for i in idx])
    R = A - (UI * lamI) @ UI.T
    theta = oracle.lanczos_upper(R, lanczos_v0)
    return R / theta + UI @ UI.T / gamma, theta, UI, lamI


def inv_root_iteration_with_storage(X0, p, steps, fmt):
    """Z_T of the coupled Newton iteration the way the path stores it: X0, every step matrix T_t, every Z_t and every
    power and M_t are rounded to `fmt` when written; products by the oracle's matmul (exact in between), each taken
    with its upper triangle mirrored into the lower one, as the path does (the rounded factors no longer commute
    exactly, so the product has a small antisymmetric part, which the mirror turns into a symmetric error)."""
    rnd = ROUNDERS[fmt]
    n = X0.shape[0]
    sym = lambda X: np.triu(X) + np.triu(X, 1).T
    M = rnd(np.asarray(X0, dtype=np.float64))
    Z = np.eye(n)
    for t in range(steps):
        T = rnd(((p + 1) * np.eye(n) - M) / p)
        Z = T if t == 0 else rnd(sym(oracle.matmul(Z, T)))
        if t + 1 == steps:
            break
        P = T
        for _ in range({1: 0, 2: 1, 4: 2}[p]):
            P = rnd(sym(oracle.matmul(P, P)))
        M = rnd(sym(oracle.matmul(P, M)))
    return Z


def inv_root_storage_error(A, Vb, k, p, steps, gamma, warmup, lanczos_v0, fmt="tf32"):
    """Relative Frobenius distance between the deflated inverse root with the iteration's stored matrices rounded to
    `fmt` and the same in fp64 throughout, both from the oracle's steps; also returns the unrounded result (it must
    equal inv_root.deflated_inv_root's)."""
    from oracle import inv_root
    X0, theta, UI, lamI = inv_root_pieces(A, Vb, k, gamma, warmup, lanczos_v0)
    z_pad, _ = inv_root.inv_root_scalar(1.0 / gamma, p, steps)
    scale = theta ** (-1.0 / p)

    def restore(Z):
        out = scale * Z + (UI * (lamI ** (-1.0 / p) - scale * z_pad)) @ UI.T if lamI.size else scale * Z
        return 0.5 * (out + out.T)
    exact = restore(inv_root.coupled_newton(X0, p, steps)[0])
    stored = restore(inv_root_iteration_with_storage(X0, p, steps, fmt))
    return float(np.linalg.norm(stored - exact) / np.linalg.norm(exact)), exact
