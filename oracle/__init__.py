"""ctypes front end of the fp64 CPU oracle (test infrastructure, never used by the product path).

Only the tests, ``__graft_entry__.smoke()`` and the benchmark's CPU-baseline leg import this
package. It compiles ``defl_oracle.cpp`` with g++ on first use and exposes each ``orc_*`` routine
on numpy float64 arrays (row-major, contiguous). The CUDA library and this package share no code.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "defl_oracle.cpp")
_LIB = os.path.join(_HERE, "libdefl_oracle.so")
_lib = None

PADDED, ADD = 0, 1
NORM_LANCZOS, NORM_FROBENIUS, NORM_GIVEN = 0, 1, 2

MUON_QUINTIC = (3.4445, -4.7750, 2.0315)      # Section 4, "General setup"
CLASSICAL_QUINTIC = (15.0 / 8.0, -5.0 / 4.0, 3.0 / 8.0)   # Eq. 2


def build(force=False):
    """Compile the oracle into a shared library next to its source."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O3", "-mavx2", "-mfma", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_lanczos_upper.restype = ctypes.c_double
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


_L = ctypes.c_long
_D = ctypes.c_double
_I = ctypes.c_int


def schedule(coeffs, L=None):
    """[L][3] float64 array from one (a,b,c) triple repeated L times or from a list of triples."""
    c = np.asarray(coeffs, dtype=np.float64)
    if c.ndim == 1:
        c = np.tile(c[None, :], (L, 1))
    return np.ascontiguousarray(c)


def matmul(A, B, ta=False, tb=False):
    A, B = _f64(A), _f64(B)
    M = A.shape[1] if ta else A.shape[0]
    K = A.shape[0] if ta else A.shape[1]
    N = B.shape[0] if tb else B.shape[1]
    C = np.empty((M, N))
    lib().orc_matmul(_I(int(ta)), _I(int(tb)), _L(M), _L(N), _L(K), _p(A), _p(B), _p(C))
    return C


def householder_orth(Y):
    Y = _f64(Y)
    Q = np.empty_like(Y)
    lib().orc_householder_orth(_L(Y.shape[0]), _L(Y.shape[1]), _p(Y), _p(Q))
    return Q


def jacobi_svd(M):
    M = _f64(M)
    r, c = M.shape
    U, s, V = np.empty((r, c)), np.empty(c), np.empty((c, c))
    lib().orc_jacobi_svd(_L(r), _L(c), _p(M), _p(U), _p(s), _p(V))
    return U, s, V


def jacobi_eig(H):
    H = _f64(H)
    n = H.shape[0]
    lam, E = np.empty(n), np.empty((n, n))
    lib().orc_jacobi_eig(_L(n), _p(H), _p(lam), _p(E))
    return lam, E


def bjorck_bowie(d):
    a = np.empty(d + 1)
    lib().orc_bjorck_bowie(_I(d), _p(a))
    return a


def filter_quintic(X, coeffs):
    """Eq. 1 with quintic steps; coeffs is [L][3]."""
    X = _f64(X).copy()
    c = schedule(coeffs)
    lib().orc_filter(_L(X.shape[0]), _L(X.shape[1]), _p(X), _I(c.shape[0]), _p(c))
    return X


def filter_classical(X, d, L):
    X = _f64(X).copy()
    lib().orc_filter_classical(_L(X.shape[0]), _L(X.shape[1]), _p(X), _I(d), _I(L))
    return X


def brsvd(A, Omega, J):
    """Algorithm 3 on one tall matrix; returns all l triplets."""
    A, Omega = _f64(A), _f64(Omega)
    rows, cols = A.shape
    l = Omega.shape[1]
    assert rows >= cols and Omega.shape[0] == cols
    U, s, V = np.empty((rows, l)), np.empty(l), np.empty((cols, l))
    lib().orc_brsvd(_L(rows), _L(cols), _p(A), _L(l), _p(Omega), _I(J), _p(U), _p(s), _p(V))
    return U, s, V


def alg1(M, U, s, V, coeffs, tau=0.0, gamma=1.01, mode=PADDED):
    """Algorithm 1 with given triplets (U[rows,r], s[r], V[cols,r]); returns (out, k, rho)."""
    M = _f64(M)
    rows, cols = M.shape
    c = schedule(coeffs)
    r = 0 if s is None else len(s)
    U_ = _f64(U) if r else None
    s_ = _f64(s) if r else None
    V_ = _f64(V) if r else None
    out, info = np.empty((rows, cols)), np.empty(2)
    lib().orc_alg1(_L(rows), _L(cols), _p(M), _L(r), _p(U_), _p(s_), _p(V_), _D(tau), _D(gamma), _I(mode),
                   _I(c.shape[0]), _p(c), _p(out), _p(info))
    return out, int(info[0]), float(info[1])


def deflated_polar(G, k, l, Omega, J, coeffs, tau=0.0, gamma=1.01, mode=PADDED):
    """Algorithm 3 then Algorithm 1 on one matrix G[m,n]; returns (out, s[l], k_used, rho)."""
    G = _f64(G)
    m, n = G.shape
    c = schedule(coeffs)
    Om = _f64(Omega) if (k > 0 and l > 0) else None
    out, s, info = np.empty((m, n)), np.zeros(max(l, 1)), np.empty(2)
    lib().orc_deflated_polar(_L(m), _L(n), _p(G), _L(k), _L(l), _p(Om), _I(J), _D(tau), _D(gamma), _I(mode),
                             _I(c.shape[0]), _p(c), _p(out), _p(s), _p(info))
    return out, s[:l], int(info[0]), float(info[1])


def round_to_storage(x, storage):
    """Values as a `storage` buffer holds them: None or 'f64' = unchanged, 'f32', or 'bf16' (round to nearest, ties to
    even, on the float32 bit pattern: keep the upper 16 bits after adding 0x7FFF plus the lowest kept bit)."""
    if storage in (None, "f64"):
        return np.array(x, dtype=np.float64)
    x32 = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    if storage == "f32":
        return x32.astype(np.float64)
    if storage != "bf16":
        raise ValueError(storage)
    bits = x32.view(np.uint32).astype(np.uint64)
    bits = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return bits.astype(np.uint32).view(np.float32).reshape(x32.shape).astype(np.float64)


def muon_step(W, Mom, Grad, lr, mu, k, l, Omega, J, coeffs, nesterov=False, weight_decay=0.0, scale=1.0,
              storage=None, tau=0.0, gamma=1.01, mode=PADDED):
    """One Deflated Muon step on one matrix (Section 1, "Two applications": W <- W - lambda polar(M), M the momentum
    matrix; Section 3, "Muon with deflation": polar is Algorithm 3 + Algorithm 1). The momentum rule, Nesterov form,
    decoupled weight decay and `scale` follow the usual Muon conventions (the paper takes them from its Muon
    references): Mom' = mu Mom + Grad, kept in `storage`; D = Mom' or Grad + mu Mom'; W' = (1 - lr wd) W - lr scale F(D).
    Returns (W', Mom')."""
    W, Mom = _f64(W), _f64(Mom)
    if Grad is None:
        Mom1 = Mom.copy()
    else:
        Grad = _f64(Grad)
        Mom1 = round_to_storage(mu * Mom + Grad, storage)
    D = (Grad + mu * Mom1) if nesterov else Mom1
    F = deflated_polar(D, k, l, Omega, J, coeffs, tau=tau, gamma=gamma, mode=mode)[0]
    return (1.0 - lr * weight_decay) * W - lr * scale * F, Mom1


def lanczos_upper(Z, v0, steps=20):
    Z, v0 = _f64(Z), _f64(v0)
    return float(lib().orc_lanczos_upper(_L(Z.shape[0]), _p(Z), _I(steps), _p(v0)))


def psd_project(Z, Vb, k, coeffs, tau=0.0, gamma=1.1, warmup=False, norm_mode=NORM_LANCZOS,
                theta=0.0, lanczos_v0=None):
    """Algorithm 2; returns (P, Vnext, lam sorted by decreasing magnitude, n_deflated, scale)."""
    Z = _f64(Z)
    n = Z.shape[0]
    Vb = _f64(Vb) if Vb is not None else np.zeros((n, 0))
    K = Vb.shape[1]
    c = schedule(coeffs)
    v0 = _f64(lanczos_v0) if lanczos_v0 is not None else None
    P, Vn, lam, info = np.empty((n, n)), np.empty((n, max(K, 1))), np.zeros(max(K, 1)), np.empty(2)
    lib().orc_psd_project(_L(n), _p(Z), _L(K), _p(Vb), _L(k), _D(tau), _D(gamma), _I(int(warmup)),
                          _I(norm_mode), _D(theta), _p(v0), _I(c.shape[0]), _p(c),
                          _p(P), _p(Vn), _p(lam), _p(info))
    return P, Vn[:, :K], lam[:K], int(info[0]), float(info[1])


def admm_diag_sdp(C, b, sigma, iters, X, S, project, warmup_iters=0):
    """Three-block ADMM of Appendix E.1, "ADMM for Standard-Form SDP" for  min <C,X>  s.t.  diag(X) = b, X PSD  (A = diag, A* = Diag, A A* = I),
    `iters` iterations from the iterates (X, S). `project(Z, warmup)` returns the S-update, e.g. a closure over
    psd_project that carries the basis along, or an exact eigenvalue projection. Returns (X, S, y, res[iters,3])
    with the three eigenvalue-free KKT terms of Appendix E.4, "Experimental Details" after every iteration."""
    C, X, S, b = _f64(C), _f64(X).copy(), _f64(S).copy(), _f64(b)
    n = C.shape[0]
    y = np.zeros(n)
    res = np.zeros((iters, 3))
    nb, nc = np.linalg.norm(b), np.linalg.norm(C)
    for it in range(iters):
        y = b / sigma - np.diag(X / sigma + S - C)
        Z = C - np.diag(y) - X / sigma
        S = project(Z, it < warmup_iters)
        X = X + sigma * (S + np.diag(y) - C)
        obj, dual = float(np.sum(C * X)), float(b @ y)
        res[it, 0] = np.linalg.norm(np.diag(X) - b) / (1.0 + nb)
        res[it, 1] = np.linalg.norm(np.diag(y) + S - C) / (1.0 + nc)
        res[it, 2] = abs(obj - dual) / (1.0 + abs(obj) + abs(dual))
    return X, S, y, res


def fill_gaussian(count, seed):
    out = np.empty(count)
    lib().orc_fill_gaussian(_p(out), _L(count), ctypes.c_uint64(seed))
    return out
