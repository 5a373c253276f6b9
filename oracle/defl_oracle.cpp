// fp64 CPU oracle for the spectrally deflated matrix filter.
//
// THIS IS TEST INFRASTRUCTURE. It is the slow, plain statement of what the CUDA library must
// compute, written from the paper's algorithms in the paper's order and notation. Only the
// tests, the smoke check and the benchmark's CPU-baseline leg may call it; the product library
// never does, and the two share no code. Everything is fp64, row-major, with plain loops
// (OpenMP over independent rows only). There is no blocking, fusion or reordering beyond what
// the cited passage states.
//
// Passages followed (paper's numbering):
//   Eq. 1          fixed-depth filter  X0 = A/theta, X_t = p_t(X_{t-1})
//   Eq. 2          quintic Newton-Schulz map  N(X) = aX + b(XX^T)X + c(XX^T)^2 X
//   Eq. 3          decomposition identities used by "restore"
//   Eq. 5 + Appendix B (proof of Theorem 1): Bjorck-Bowie coefficients of the degree-(2d+1) family
//   Algorithm 1    deflated polar factor (gate, subtract, normalise, padded init, filter)
//   Algorithm 2    deflated PSD projection (Rayleigh-Ritz, gate on |lambda|, padded init,
//                  reconstruction, symmetrisation, basis update)
//   Algorithm 3    batched randomized SVD (sketch, orthonormalise, J subspace iterations,
//                  thin SVD of Q^T A, truncate)
//   Appendix E.1, "Normalization scale"       20-step Lanczos upper estimate theta = sqrt(rho + ||Z^2 v - rho v||)
//   Eq. 6, Eq. 7   PSD projection through the sign function, and the undeflated baseline
//
// Pinned (tests/test_oracle_*.py): Example 1's printed values, the Bjorck-Bowie closed form,
// Lemma 1's residual identity, Eq. 3 against a brute-force LAPACK SVD/eig, the scalarised error
// of Theorem 1 and Proposition 2, the randomized-SVD sandwich bound, and every linear-algebra
// primitive against numpy. Parity unpinned: none of the functions below.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>
#include <numeric>

typedef std::vector<double> vec;

// ------------------------------------------------------------------------------------------
// Plain dense primitives
// ------------------------------------------------------------------------------------------

// C[M,N] = op(A) op(B), op = transpose when the flag is set. A is [M,K] (or [K,M] if ta),
// B is [K,N] (or [N,K] if tb); all row-major with no padding.
static void mm(bool ta, bool tb, long M, long N, long K, const double* A, const double* B, double* C) {
#pragma omp parallel for schedule(static)
  for (long i = 0; i < M; ++i) {
    double* c = C + i * N;
    if (tb && !ta) {                       // rows of A against rows of B
      const double* a = A + i * K;
      for (long j = 0; j < N; ++j) {
        const double* b = B + j * K;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (long k = 0; k < K; ++k) acc += a[k] * b[k];
        c[j] = acc;
      }
      continue;
    }
    for (long j = 0; j < N; ++j) c[j] = 0.0;
    for (long k = 0; k < K; ++k) {
      const double a = ta ? A[k * M + i] : A[i * K + k];
      if (!tb) {
        const double* b = B + k * N;
#pragma omp simd
        for (long j = 0; j < N; ++j) c[j] += a * b[j];
      } else {
        for (long j = 0; j < N; ++j) c[j] += a * B[j * K + k];
      }
    }
  }
}

static double frob(const double* A, long n) {
  double s = 0.0;
  for (long i = 0; i < n; ++i) s += A[i] * A[i];
  return std::sqrt(s);
}

// Thin orthonormal factor of Y[rows,cols] (rows >= cols) by Householder reflections.
// Columns are signed so that the triangular factor has a non-negative diagonal, which makes Q
// the unique QR factor (the same Q a Cholesky-based QR returns in exact arithmetic).
static void householder_orth(long rows, long cols, const double* Y, double* Q) {
  vec W(Y, Y + rows * cols);
  vec Vs(rows * cols, 0.0);   // reflector j in column j (entries j..rows-1)
  vec beta(cols, 0.0), rdiag(cols, 0.0);
  for (long j = 0; j < cols; ++j) {
    double nrm = 0.0;
    for (long i = j; i < rows; ++i) nrm += W[i * cols + j] * W[i * cols + j];
    nrm = std::sqrt(nrm);
    if (nrm == 0.0) { beta[j] = 0.0; rdiag[j] = 0.0; continue; }
    const double x0 = W[j * cols + j];
    const double alpha = (x0 >= 0.0) ? -nrm : nrm;      // R_jj
    for (long i = j; i < rows; ++i) Vs[i * cols + j] = W[i * cols + j];
    Vs[j * cols + j] = x0 - alpha;
    double vn = 0.0;
    for (long i = j; i < rows; ++i) vn += Vs[i * cols + j] * Vs[i * cols + j];
    beta[j] = (vn > 0.0) ? 2.0 / vn : 0.0;
    rdiag[j] = alpha;
    for (long c = j; c < cols; ++c) {
      double d = 0.0;
      for (long i = j; i < rows; ++i) d += Vs[i * cols + j] * W[i * cols + c];
      d *= beta[j];
      for (long i = j; i < rows; ++i) W[i * cols + c] -= d * Vs[i * cols + j];
    }
  }
  // Q = H_0 H_1 ... H_{cols-1} [I; 0]
  for (long i = 0; i < rows; ++i)
    for (long c = 0; c < cols; ++c) Q[i * cols + c] = (i == c) ? 1.0 : 0.0;
  for (long j = cols - 1; j >= 0; --j) {
    if (beta[j] == 0.0) continue;
    for (long c = 0; c < cols; ++c) {
      double d = 0.0;
      for (long i = j; i < rows; ++i) d += Vs[i * cols + j] * Q[i * cols + c];
      d *= beta[j];
      for (long i = j; i < rows; ++i) Q[i * cols + c] -= d * Vs[i * cols + j];
    }
  }
  for (long c = 0; c < cols; ++c)
    if (rdiag[c] < 0.0)
      for (long i = 0; i < rows; ++i) Q[i * cols + c] = -Q[i * cols + c];
}

// One-sided (Hestenes) Jacobi SVD of M[rows,cols], rows >= cols:
// M = U diag(s) V^T, s descending, U[rows,cols], V[cols,cols].
static void jacobi_svd(long rows, long cols, const double* M, double* U, double* s, double* V) {
  vec W(M, M + rows * cols);
  vec R(cols * cols, 0.0);
  for (long i = 0; i < cols; ++i) R[i * cols + i] = 1.0;
  const double eps = 1e-15;
  for (int sweep = 0; sweep < 60; ++sweep) {
    long rotations = 0;
    for (long p = 0; p < cols - 1; ++p)
      for (long q = p + 1; q < cols; ++q) {
        double alpha = 0, beta = 0, gamma = 0;
        for (long i = 0; i < rows; ++i) {
          const double a = W[i * cols + p], b = W[i * cols + q];
          alpha += a * a; beta += b * b; gamma += a * b;
        }
        if (gamma == 0.0 || std::fabs(gamma) <= eps * std::sqrt(alpha * beta)) continue;
        ++rotations;
        const double zeta = (beta - alpha) / (2.0 * gamma);
        const double t = ((zeta >= 0) ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
        const double c = 1.0 / std::sqrt(1.0 + t * t), sn = c * t;
        for (long i = 0; i < rows; ++i) {
          const double a = W[i * cols + p], b = W[i * cols + q];
          W[i * cols + p] = c * a - sn * b;
          W[i * cols + q] = sn * a + c * b;
        }
        for (long i = 0; i < cols; ++i) {
          const double a = R[i * cols + p], b = R[i * cols + q];
          R[i * cols + p] = c * a - sn * b;
          R[i * cols + q] = sn * a + c * b;
        }
      }
    if (rotations == 0) break;
  }
  vec nrm(cols);
  for (long j = 0; j < cols; ++j) {
    double a = 0;
    for (long i = 0; i < rows; ++i) a += W[i * cols + j] * W[i * cols + j];
    nrm[j] = std::sqrt(a);
  }
  std::vector<long> ord(cols);
  std::iota(ord.begin(), ord.end(), 0L);
  std::stable_sort(ord.begin(), ord.end(), [&](long a, long b) { return nrm[a] > nrm[b]; });
  for (long jj = 0; jj < cols; ++jj) {
    const long j = ord[jj];
    s[jj] = nrm[j];
    for (long i = 0; i < rows; ++i) U[i * cols + jj] = (nrm[j] > 0) ? W[i * cols + j] / nrm[j] : 0.0;
    for (long i = 0; i < cols; ++i) V[i * cols + jj] = R[i * cols + j];
  }
}

// Cyclic two-sided Jacobi for a symmetric H[n,n]: H = E diag(lam) E^T (unsorted).
static void jacobi_eig(long n, const double* H, double* lam, double* E) {
  vec A(H, H + n * n);
  for (long i = 0; i < n; ++i)
    for (long j = 0; j < n; ++j) E[i * n + j] = (i == j) ? 1.0 : 0.0;
  for (int sweep = 0; sweep < 100; ++sweep) {
    double off = 0, diag = 0;
    for (long i = 0; i < n; ++i)
      for (long j = 0; j < n; ++j) (i == j ? diag : off) += A[i * n + j] * A[i * n + j];
    if (off <= 1e-32 * (diag + off)) break;
    for (long p = 0; p < n - 1; ++p)
      for (long q = p + 1; q < n; ++q) {
        const double apq = A[p * n + q];
        if (apq == 0.0) continue;
        const double zeta = (A[q * n + q] - A[p * n + p]) / (2.0 * apq);
        const double t = ((zeta >= 0) ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
        const double c = 1.0 / std::sqrt(1.0 + t * t), s = c * t;
        for (long i = 0; i < n; ++i) {   // columns p,q
          const double a = A[i * n + p], b = A[i * n + q];
          A[i * n + p] = c * a - s * b;
          A[i * n + q] = s * a + c * b;
        }
        for (long i = 0; i < n; ++i) {   // rows p,q
          const double a = A[p * n + i], b = A[q * n + i];
          A[p * n + i] = c * a - s * b;
          A[q * n + i] = s * a + c * b;
        }
        for (long i = 0; i < n; ++i) {
          const double a = E[i * n + p], b = E[i * n + q];
          E[i * n + p] = c * a - s * b;
          E[i * n + q] = s * a + c * b;
        }
      }
  }
  for (long i = 0; i < n; ++i) lam[i] = A[i * n + i];
}

// ------------------------------------------------------------------------------------------
// Eq. 5 / Appendix B (proof of Theorem 1): Bjorck-Bowie coefficients a_i = (-1)^i sum_{j=i..d} 4^-j C(2j,j) C(j,i)
// ------------------------------------------------------------------------------------------
static double binom(int n, int k) {
  double r = 1.0;
  for (int i = 1; i <= k; ++i) r = r * (n - k + i) / i;
  return r;
}

extern "C" void orc_bjorck_bowie(int d, double* a /* [d+1] */) {
  for (int i = 0; i <= d; ++i) {
    double s = 0.0;
    for (int j = i; j <= d; ++j) s += std::pow(4.0, -j) * binom(2 * j, j) * binom(j, i);
    a[i] = ((i % 2) ? -1.0 : 1.0) * s;
  }
}

// ------------------------------------------------------------------------------------------
// Eq. 2 (and Eq. 5 for general degree): one map  X <- sum_i a_i (X X^T)^i X  on X[m,n].
// The Gram matrix is taken on the short side, using (X X^T) X = X (X^T X).
// Each power is applied to the running product, in the order the equation lists its terms.
// ------------------------------------------------------------------------------------------
static void ns_map(long m, long n, double* X, int d, const double* a) {
  const bool left = (m <= n);
  const long g = left ? m : n;
  vec A(g * g), T(X, X + m * n), Tn(m * n), Xn(m * n);
  if (left) mm(false, true, m, m, n, X, X, A.data());   // X X^T
  else      mm(true, false, n, n, m, X, X, A.data());   // X^T X
  for (long i = 0; i < m * n; ++i) Xn[i] = a[0] * X[i];
  for (int p = 1; p <= d; ++p) {
    if (left) mm(false, false, m, n, m, A.data(), T.data(), Tn.data());
    else      mm(false, false, m, n, n, T.data(), A.data(), Tn.data());
    T.swap(Tn);
    for (long i = 0; i < m * n; ++i) Xn[i] += a[p] * T[i];
  }
  std::memcpy(X, Xn.data(), sizeof(double) * m * n);
}

// Eq. 1: X_t = p_t(X_{t-1}) for t = 1..L with quintic steps (a_t, b_t, c_t); in place.
extern "C" void orc_filter(long m, long n, double* X, int L, const double* coeffs /* [L][3] */) {
  for (int t = 0; t < L; ++t) ns_map(m, n, X, 2, coeffs + 3 * t);
}

// Eq. 5: L steps of the degree-(2d+1) classical map; in place.
extern "C" void orc_filter_classical(long m, long n, double* X, int d, int L) {
  vec a(d + 1);
  orc_bjorck_bowie(d, a.data());
  for (int t = 0; t < L; ++t) ns_map(m, n, X, d, a.data());
}

// ------------------------------------------------------------------------------------------
// Algorithm 3 for one matrix A[rows,cols], rows >= cols, with the sketch Omega[cols,l] given.
// Returns all l triplets (the caller truncates to the window): U[rows,l], s[l], V[cols,l].
// ------------------------------------------------------------------------------------------
extern "C" void orc_brsvd(long rows, long cols, const double* A, long l, const double* Omega, int J,
                          double* U, double* s, double* V) {
  vec Y(rows * l), Q(rows * l), Yp(cols * l), Qp(cols * l);
  mm(false, false, rows, l, cols, A, Omega, Y.data());            // A Omega
  householder_orth(rows, l, Y.data(), Q.data());
  for (int j = 0; j < J; ++j) {
    mm(true, false, cols, l, rows, A, Q.data(), Yp.data());       // A^T Q
    householder_orth(cols, l, Yp.data(), Qp.data());
    mm(false, false, rows, l, cols, A, Qp.data(), Y.data());      // A Y
    householder_orth(rows, l, Y.data(), Q.data());
  }
  vec Gt(cols * l);                                               // (Q^T A)^T = A^T Q, [cols,l]
  mm(true, false, cols, l, rows, A, Q.data(), Gt.data());
  // thin SVD of G = Q^T A through its transpose: G^T = V diag(s) U_G^T
  vec UG(l * l);
  jacobi_svd(cols, l, Gt.data(), V, s, UG.data());
  mm(false, false, rows, l, l, Q.data(), UG.data(), U);           // U = Q U_G
}

// ------------------------------------------------------------------------------------------
// Algorithm 1 for one matrix M[rows,cols] (any orientation; the algorithm is symmetric under
// transposition because polar(M^T) = polar(M)^T), with triplets U[rows,r], s[r], V[cols,r].
//   tau > 0 : the paper's gate; k = max{i : s_i > tau s_1} if s_r/s_1 < tau, else no deflation.
//   tau <= 0: deflate exactly the r given triplets (fixed-k reading).
//   mode 0 (PADDED): X0 = R/||R||_F + U_k V_k^T / gamma, return N^L(X0)        (Algorithm 1)
//   mode 1 (ADD)   : X0 = R/||R||_F,                    return N^L(X0) + U_k V_k^T (Eq. 3)
// Outputs: out[rows,cols]; info[0] = k used, info[1] = ||R||_F (or ||M||_F when k = 0).
// ------------------------------------------------------------------------------------------
extern "C" void orc_alg1(long rows, long cols, const double* M, long r, const double* U, const double* s,
                         const double* V, double tau, double gamma, int mode, int L, const double* coeffs,
                         double* out, double* info) {
  long k = r;
  if (tau > 0.0 && r > 0) {
    if (s[r - 1] / s[0] < tau) {
      k = 0;
      for (long i = 0; i < r; ++i) if (s[i] > tau * s[0]) k = i + 1;
    } else {
      k = 0;
    }
  }
  vec R(M, M + rows * cols), H(rows * cols, 0.0);
  for (long i = 0; i < rows; ++i)
    for (long j = 0; j < cols; ++j) {
      double hs = 0.0, h = 0.0;
      for (long t = 0; t < k; ++t) {
        hs += U[i * r + t] * s[t] * V[j * r + t];
        h += U[i * r + t] * V[j * r + t];
      }
      R[i * cols + j] -= hs;
      H[i * cols + j] = h;
    }
  const double rho = frob(R.data(), rows * cols);
  for (long i = 0; i < rows * cols; ++i) {
    double x0 = (rho > 0.0) ? R[i] / rho : 0.0;
    if (mode == 0 && k > 0) x0 += H[i] / gamma;
    out[i] = x0;
  }
  orc_filter(rows, cols, out, L, coeffs);
  if (mode == 1 && k > 0)
    for (long i = 0; i < rows * cols; ++i) out[i] += H[i];
  if (info) { info[0] = (double)k; info[1] = rho; }
}

// Algorithm 3 followed by Algorithm 1 for one matrix G[m,n] in the caller's orientation.
// A = G if m >= n, else G^T (the paper transposes wide matrices); the sketch is Omega[min(m,n), l];
// the window is the leading k of the l computed triplets. s_out[l] receives all estimates.
extern "C" void orc_deflated_polar(long m, long n, const double* G, long k, long l, const double* Omega, int J,
                                   double tau, double gamma, int mode, int L, const double* coeffs,
                                   double* out, double* s_out, double* info) {
  const bool tall = (m >= n);
  const long rows = tall ? m : n, cols = tall ? n : m;
  vec A(rows * cols);
  if (tall) std::memcpy(A.data(), G, sizeof(double) * m * n);
  else
    for (long i = 0; i < m; ++i)
      for (long j = 0; j < n; ++j) A[j * m + i] = G[i * n + j];
  vec res(rows * cols);
  if (k <= 0 || l <= 0) {
    orc_alg1(rows, cols, A.data(), 0, nullptr, nullptr, nullptr, tau, gamma, mode, L, coeffs, res.data(), info);
  } else {
    vec U(rows * l), s(l), V(cols * l);
    orc_brsvd(rows, cols, A.data(), l, Omega, J, U.data(), s.data(), V.data());
    if (s_out) std::memcpy(s_out, s.data(), sizeof(double) * l);
    vec Uk(rows * k), Vk(cols * k);
    for (long i = 0; i < rows; ++i) for (long t = 0; t < k; ++t) Uk[i * k + t] = U[i * l + t];
    for (long i = 0; i < cols; ++i) for (long t = 0; t < k; ++t) Vk[i * k + t] = V[i * l + t];
    orc_alg1(rows, cols, A.data(), k, Uk.data(), s.data(), Vk.data(), tau, gamma, mode, L, coeffs, res.data(), info);
  }
  if (tall) std::memcpy(out, res.data(), sizeof(double) * m * n);
  else
    for (long i = 0; i < m; ++i)
      for (long j = 0; j < n; ++j) out[i * n + j] = res[j * m + i];
}

// ------------------------------------------------------------------------------------------
// Appendix E.1, "Normalization scale": Lanczos on Z^2 (applied as Z(Zv), never formed), `steps` steps with full
// reorthogonalisation from the start vector v0; (rho, v) = largest Ritz pair;
// theta = sqrt(rho + ||Z^2 v - rho v||_2).
// ------------------------------------------------------------------------------------------
static void symv(long n, const double* Z, const double* x, double* y) {
#pragma omp parallel for schedule(static)
  for (long i = 0; i < n; ++i) {
    double a = 0;
    for (long j = 0; j < n; ++j) a += Z[i * n + j] * x[j];
    y[i] = a;
  }
}

extern "C" double orc_lanczos_upper(long n, const double* Z, int steps, const double* v0) {
  if (steps > n) steps = (int)n;
  vec Q((long)steps * n, 0.0), alpha(steps, 0.0), beta(steps, 0.0), t(n), w(n);
  double nv = frob(v0, n);
  if (nv == 0.0) return 0.0;
  for (long i = 0; i < n; ++i) Q[i] = v0[i] / nv;
  int m = 0;
  for (int j = 0; j < steps; ++j) {
    const double* q = &Q[(long)j * n];
    symv(n, Z, q, t.data());
    symv(n, Z, t.data(), w.data());
    double a = 0;
    for (long i = 0; i < n; ++i) a += q[i] * w[i];
    alpha[j] = a;
    m = j + 1;
    for (int pass = 0; pass < 2; ++pass)       // full reorthogonalisation, twice
      for (int p = 0; p <= j; ++p) {
        const double* qp = &Q[(long)p * n];
        double d = 0;
        for (long i = 0; i < n; ++i) d += qp[i] * w[i];
        for (long i = 0; i < n; ++i) w[i] -= d * qp[i];
      }
    const double b = frob(w.data(), n);
    if (j + 1 == steps) break;
    if (b <= 1e-12 * std::fabs(alpha[0])) break;
    beta[j] = b;
    for (long i = 0; i < n; ++i) Q[(long)(j + 1) * n + i] = w[i] / b;
  }
  vec T((long)m * m, 0.0), lam(m), E((long)m * m);
  for (int i = 0; i < m; ++i) {
    T[i * m + i] = alpha[i];
    if (i + 1 < m) { T[i * m + i + 1] = beta[i]; T[(i + 1) * m + i] = beta[i]; }
  }
  jacobi_eig(m, T.data(), lam.data(), E.data());
  int best = 0;
  for (int i = 1; i < m; ++i) if (lam[i] > lam[best]) best = i;
  const double rho = lam[best];
  vec v(n, 0.0);
  for (int p = 0; p < m; ++p)
    for (long i = 0; i < n; ++i) v[i] += E[p * m + best] * Q[(long)p * n + i];
  symv(n, Z, v.data(), t.data());
  symv(n, Z, t.data(), w.data());
  double res = 0;
  for (long i = 0; i < n; ++i) { const double d = w[i] - rho * v[i]; res += d * d; }
  return std::sqrt(std::max(0.0, rho) + std::sqrt(res));
}

// ------------------------------------------------------------------------------------------
// Algorithm 2: one deflated PSD projection of the symmetric Z[n,n] with the orthonormal basis
// Vb[n,K] from the previous call.
//   k      : deflate the k Ritz pairs of largest |lambda| (fixed-k reading, tau <= 0), or with
//            tau > 0 the paper's gate on the leading k magnitudes: if s_k < tau s_1 deflate
//            {i : |lambda_i| > tau s_1}, else nothing.
//   k = 0 or warmup != 0 : the undeflated baseline P = Z (I + g(Z/theta)) / 2  (Eq. 7).
//   norm_mode 0 : Lanczos upper estimate (Appendix E.1, "Normalization scale") with start vector lanczos_v0[n];
//             1 : Frobenius norm;  2 : the value theta_given.
//   g = p_T o ... o p_1 with quintics coeffs[T][3].
// Outputs: P[n,n] (exactly symmetric), Vnext[n,K] = orth(Z Vb), lam[K] Ritz values in the order
// of decreasing magnitude, info[0] = number deflated, info[1] = scale used.
// ------------------------------------------------------------------------------------------
extern "C" void orc_psd_project(long n, const double* Z, long K, const double* Vb, long k, double tau,
                                double gamma, int warmup, int norm_mode, double theta_given,
                                const double* lanczos_v0, int T, const double* coeffs,
                                double* P, double* Vnext, double* lam_out, double* info) {
  vec Zt(n * K), H(K * K), lam(K), E(K * K), U(n * K);
  std::vector<long> ord(K);
  if (K > 0) {
    mm(false, false, n, K, n, Z, Vb, Zt.data());                   // Z~ = Z V
    mm(true, false, K, K, n, Vb, Zt.data(), H.data());             // V^T Z~
    for (long i = 0; i < K; ++i)
      for (long j = i + 1; j < K; ++j) {
        const double a = 0.5 * (H[i * K + j] + H[j * K + i]);
        H[i * K + j] = a; H[j * K + i] = a;
      }
    jacobi_eig(K, H.data(), lam.data(), E.data());
    mm(false, false, n, K, K, Vb, E.data(), U.data());             // U = V E
    std::iota(ord.begin(), ord.end(), 0L);
    std::stable_sort(ord.begin(), ord.end(),
                     [&](long a, long b) { return std::fabs(lam[a]) > std::fabs(lam[b]); });
    if (lam_out) for (long i = 0; i < K; ++i) lam_out[i] = lam[ord[i]];
  }
  std::vector<long> I;
  if (!warmup && k > 0 && K > 0) {
    if (k > K) k = K;
    if (tau > 0.0) {
      const double s1 = std::fabs(lam[ord[0]]), sr = std::fabs(lam[ord[k - 1]]);
      if (sr < tau * s1)
        for (long i = 0; i < K; ++i) if (std::fabs(lam[ord[i]]) > tau * s1) I.push_back(ord[i]);
    } else {
      for (long i = 0; i < k; ++i) I.push_back(ord[i]);
    }
  }
  vec R(Z, Z + n * n);
  for (long idx : I)
    for (long i = 0; i < n; ++i)
      for (long j = 0; j < n; ++j) R[i * n + j] -= lam[idx] * U[i * K + idx] * U[j * K + idx];
  double theta;
  if (norm_mode == 0) theta = orc_lanczos_upper(n, R.data(), 20, lanczos_v0);
  else if (norm_mode == 1) theta = frob(R.data(), n * n);
  else theta = theta_given;
  vec X(n * n);
  for (long i = 0; i < n * n; ++i) X[i] = (theta > 0.0) ? R[i] / theta : 0.0;
  for (long idx : I) {
    const double sg = (lam[idx] > 0) ? 1.0 : ((lam[idx] < 0) ? -1.0 : 0.0);
    for (long i = 0; i < n; ++i)
      for (long j = 0; j < n; ++j) X[i * n + j] += sg / gamma * U[i * K + idx] * U[j * K + idx];
  }
  orc_filter(n, n, X.data(), T, coeffs);                           // g(X0)
  vec RG(n * n);
  mm(false, false, n, n, n, R.data(), X.data(), RG.data());        // R g(X0)
  for (long i = 0; i < n * n; ++i) P[i] = 0.5 * (R[i] + RG[i]);
  for (long idx : I)
    if (lam[idx] > 0)
      for (long i = 0; i < n; ++i)
        for (long j = 0; j < n; ++j) P[i * n + j] += lam[idx] * U[i * K + idx] * U[j * K + idx];
  for (long i = 0; i < n; ++i)
    for (long j = i + 1; j < n; ++j) {
      const double a = 0.5 * (P[i * n + j] + P[j * n + i]);
      P[i * n + j] = a; P[j * n + i] = a;
    }
  if (K > 0 && Vnext) householder_orth(n, K, Zt.data(), Vnext);
  if (info) { info[0] = (double)I.size(); info[1] = theta; }
}

// ------------------------------------------------------------------------------------------
// Primitives exported so that the tests can pin each one against an independent library.
// ------------------------------------------------------------------------------------------
extern "C" void orc_matmul(int ta, int tb, long M, long N, long K, const double* A, const double* B, double* C) {
  mm(ta != 0, tb != 0, M, N, K, A, B, C);
}
extern "C" void orc_householder_orth(long rows, long cols, const double* Y, double* Q) {
  householder_orth(rows, cols, Y, Q);
}
extern "C" void orc_jacobi_svd(long rows, long cols, const double* M, double* U, double* s, double* V) {
  jacobi_svd(rows, cols, M, U, s, V);
}
extern "C" void orc_jacobi_eig(long n, const double* H, double* lam, double* E) {
  jacobi_eig(n, H, lam, E);
}

// ------------------------------------------------------------------------------------------
// Counter-based Gaussian generator for a sketch drawn inside the library (the paper only says
// "Gaussian", Algorithm 3 line 2). Element idx of a stream with a given seed:
//   h(x): x += 0x9E3779B97F4A7C15; x = (x ^ x>>30) * 0xBF58476D1CE4E5B9;
//         x = (x ^ x>>27) * 0x94D049BB133111EB; return x ^ x>>31
//   j = idx/2; r1 = h(h(seed) ^ 2j); r2 = h(h(seed) ^ (2j+1));
//   u1 = ((r1>>11)+1) 2^-53, u2 = (r2>>11) 2^-53; radius = sqrt(-2 ln u1)
//   value = radius cos(2 pi u2) for even idx, radius sin(2 pi u2) for odd idx.
// ------------------------------------------------------------------------------------------
static inline uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

extern "C" void orc_fill_gaussian(double* dst, long count, uint64_t seed) {
  const uint64_t hs = mix64(seed);
  const double two_pi = 6.283185307179586476925286766559;
  for (long idx = 0; idx < count; ++idx) {
    const uint64_t j = (uint64_t)idx / 2;
    const uint64_t r1 = mix64(hs ^ (2 * j)), r2 = mix64(hs ^ (2 * j + 1));
    const double u1 = ((double)(r1 >> 11) + 1.0) * (1.0 / 9007199254740992.0);
    const double u2 = (double)(r2 >> 11) * (1.0 / 9007199254740992.0);
    const double rad = std::sqrt(-2.0 * std::log(u1));
    dst[idx] = (idx % 2 == 0) ? rad * std::cos(two_pi * u2) : rad * std::sin(two_pi * u2);
  }
}
