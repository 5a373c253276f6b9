"""fp64 CPU oracle of the deflated inverse matrix root (test infrastructure, never used by the product path).

The paper's Conclusion names inverse matrix roots (the preconditioners of Shampoo-type optimizers) as the next
instance of spectral deflation and gives no algorithm for it. The construction here applies the framework's three
moves to f(A) = A^(-1/p), A symmetric positive definite, and every step is one the paper defines for its own two
instances:

  * the leading eigenpairs come from a tracked basis by one block step and Rayleigh-Ritz, and are removed from A
    (Algorithm 2, lines 1-5);
  * the residual is normalised by the Lanczos upper estimate of its spectral norm (Appendix E.1, "Normalization
    scale") and the removed directions are padded back at 1/gamma, inside the interval (Algorithm 1, line 4;
    Algorithm 2, line 7);
  * a fixed number of matrix-product-only steps runs on the normalised matrix: here the coupled Newton iteration
    for the inverse p-th root,  T_t = ((p+1) I - M_t)/p,  Z_{t+1} = Z_t T_t,  M_{t+1} = T_t^p M_t,  M_0 = X0, Z_0 = I,
    whose iterates are polynomials in X0 (so they commute with it, and a direction padded at 1/gamma comes out at
    the scalar iteration's value z_T(1/gamma));
  * the target is restored exactly on the removed directions (Algorithm 1, line 6 in its padded form; Eq. 3):
    out = theta^(-1/p) (Z_T - z_T(1/gamma) U U^T) + U diag(lambda_i^(-1/p)) U^T,  symmetrised.

The removed pairs must be accurate: a Ritz pair (lambda, u) with residual r leaves R = A - lambda u u^T indefinite (an
eigenvalue near -|r|^2 / a, a = r^T A r / |r|^2); the padding keeps X0 positive definite while |r|^2 < a theta / gamma, and
the iteration diverges on an eigenvalue that is not positive. Hence warm-up calls (basis advanced, nothing removed)
until the basis has settled, the protocol the paper uses for its projection.

Plain numpy on top of the oracle's own primitives (its matrix product, Jacobi eigensolver, Householder
orthonormalisation and Lanczos estimate); no blocking, no fusion.
"""
import numpy as np

from . import householder_orth, jacobi_eig, lanczos_upper, matmul


def inv_root_scalar(m0, p, steps):
    """The scalar iteration t = ((p+1) - m)/p, z <- z t, m <- m t^p from (m0, 1): returns (z, m)."""
    m, z = float(m0), 1.0
    for _ in range(steps):
        t = ((p + 1) - m) / p
        z *= t
        m *= t ** p
    return z, m


def coupled_newton(X0, p, steps):
    """Z_T of the coupled Newton iteration for X0^(-1/p) (eigenvalues of X0 in (0, 1]); also returns M_T."""
    X0 = np.asarray(X0, dtype=np.float64)
    n = X0.shape[0]
    M, Z = X0.copy(), np.eye(n)
    for _ in range(steps):
        T = ((p + 1) * np.eye(n) - M) / p
        Z = matmul(Z, T)
        for _ in range(p):
            M = matmul(T, M)
    return Z, M


def deflated_inv_root(A, Vb, k, p, steps, gamma=1.1, warmup=False, lanczos_v0=None):
    """Deflated inverse p-th root of the symmetric positive definite A with the tracked basis Vb[n, K] (orthonormal
    columns; None or K = 0: no deflation). Returns (out, Vnext, lam sorted by decreasing magnitude, n_deflated, theta)."""
    A = np.asarray(A, dtype=np.float64)
    n = A.shape[0]
    K = 0 if Vb is None else Vb.shape[1]
    idx, lam, U, Vnext = [], np.zeros(0), None, None
    if K > 0:
        At = matmul(A, Vb)                              # block step
        H = matmul(Vb, At, ta=True)
        H = 0.5 * (H + H.T)
        lam_raw, E = jacobi_eig(H)
        U = matmul(Vb, E)
        order = sorted(range(K), key=lambda i: (-abs(lam_raw[i]), i))
        lam = np.array([lam_raw[i] for i in order])
        if not warmup and k > 0:
            idx = order[:min(k, K)]
        Vnext = householder_orth(At)
    R = A.copy()
    for i in idx:
        R -= lam_raw[i] * np.outer(U[:, i], U[:, i])
    theta = lanczos_upper(R, lanczos_v0)
    X0 = R / theta
    for i in idx:
        X0 += np.outer(U[:, i], U[:, i]) / gamma
    Z, _ = coupled_newton(X0, p, steps)
    z_pad, _ = inv_root_scalar(1.0 / gamma, p, steps)
    scale = theta ** (-1.0 / p)
    out = scale * Z
    for i in idx:
        out += (lam_raw[i] ** (-1.0 / p) - scale * z_pad) * np.outer(U[:, i], U[:, i])
    out = 0.5 * (out + out.T)
    return out, Vnext, lam, len(idx), theta
