// Small-panel kernels of the randomized SVD front end (Algorithm 3) and helpers:
//   * Gram matrices of tall skinny panels (CholeskyQR and the Gram core of the thin SVD)
//   * l x l Cholesky factorisation + triangular inverse in shared memory (fp64)
//   * one-sided Jacobi eigensolver of the l x l core in shared memory, one warp per column
//     pair, rotations through warp shuffles (fp64)
//   * panel x small-matrix products, column scaling, Frobenius partial sums, scaling,
//     the counter-based Gaussian fill.
// All reductions run in a fixed order so that repeated runs are bit-identical.
#include "common.cuh"
#include "panel.cuh"

namespace defl {

// ---------------------------------------------------------------------------------------------
// Gram partials: for panel Y[b, rows, l] (fp32, leading dimension ld), CTA (chunk, batch) writes
// partial[b, chunk, l, l] = sum over its rows of y_r y_r^T  (fp32 products over 32-row groups,
// groups added in fp64).
// ---------------------------------------------------------------------------------------------
constexpr int GRAM_ROWS = 256;   // rows per CTA
constexpr int GRAM_SUB = 32;     // rows per fp32 sub-accumulation

__global__ void __launch_bounds__(256) gram_partial_kernel(const float* __restrict__ Y, const float* __restrict__ Y2,
                                                           long long batch_stride, int rows, int l, int ld, int nchunk,
                                                           double* __restrict__ partial) {
  __shared__ float tile[GRAM_SUB][MAX_L + 1];
  __shared__ float tile2[GRAM_SUB][MAX_L + 1];
  const int chunk = blockIdx.x, bz = blockIdx.y, tid = threadIdx.x;
  const float* Yb = Y + (long long)bz * batch_stride;
  const float* Y2b = Y2 ? Y2 + (long long)bz * batch_stride : nullptr;
  const int tx = tid % 16, ty = tid / 16;   // 16 x 16 threads, each a 4 x 4 block of the l x l Gram
  double acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
  const int r_begin = chunk * GRAM_ROWS, r_end = min(rows, r_begin + GRAM_ROWS);
  for (int r0 = r_begin; r0 < r_end; r0 += GRAM_SUB) {
    for (int e = tid; e < GRAM_SUB * l; e += 256) {
      const int rr = e / l, c = e % l;
      const int gr = r0 + rr;
      tile[rr][c] = (gr < r_end) ? Yb[(long long)gr * ld + c] : 0.f;
      tile2[rr][c] = Y2b ? ((gr < r_end) ? Y2b[(long long)gr * ld + c] : 0.f) : tile[rr][c];
    }
    __syncthreads();
    float f[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) f[i][j] = 0.f;
    for (int rr = 0; rr < GRAM_SUB; ++rr) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = (ty * 4 + i < l) ? tile[rr][ty * 4 + i] : 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = (tx * 4 + j < l) ? tile2[rr][tx * 4 + j] : 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) f[i][j] = fmaf(a[i], b[j], f[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] += (double)f[i][j];
    __syncthreads();
  }
  double* out = partial + ((long long)bz * nchunk + chunk) * l * l;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gi = ty * 4 + i, gj = tx * 4 + j;
      if (gi < l && gj < l) out[gi * l + gj] = acc[i][j];
    }
}

int gram_num_chunks(int rows) { return (rows + GRAM_ROWS - 1) / GRAM_ROWS; }

cudaError_t gram_partial_launch(const float* Y, long long batch_stride, int batch, int rows, int l, int ld,
                                double* partial, cudaStream_t st, long long* launches, const float* Y2) {
  const int nchunk = gram_num_chunks(rows);
  gram_partial_kernel<<<dim3(nchunk, batch), 256, 0, st>>>(Y, Y2, batch_stride, rows, l, ld, nchunk, partial);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Cholesky of W = sum of partials (l x l, fp64, shared memory), W = R^T R, output Rinv = R^-1
// (upper triangular, fp32, row-major [l,l]). A non-positive pivot restarts with W + shift I and
// sets DEFL_ST_CHOL_SHIFT (bit 1) in status[b].
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) chol_inv_kernel(const double* __restrict__ partial, int nchunk, int l,
                                                       float* __restrict__ Rinv, int* __restrict__ status) {
  extern __shared__ double sm[];
  // rows are padded to an odd number of doubles: a column walk (row stride apart) then touches every bank once
  // instead of one bank 32 times (l = 48 doubles = 96 words = 0 mod 32)
  const int ls = l | 1;
  double* W = sm;                              // [l][ls] original Gram
  double* Lm = sm + MAX_L * (MAX_L + 1);       // [l][ls] lower factor, then its inverse
  __shared__ int bad;
  __shared__ double rdiag[MAX_L];
  const int bz = blockIdx.x, tid = threadIdx.x;
  const double* pb = partial + (long long)bz * nchunk * l * l;
  for (int e = tid; e < l * l; e += blockDim.x) {
    double t = 0.0;
#pragma unroll 8
    for (int c = 0; c < nchunk; ++c) t += pb[(long long)c * l * l + e];
    W[(e / l) * ls + e % l] = t;
  }
  __syncthreads();
  // symmetrise exactly
  for (int e = tid; e < l * l; e += blockDim.x) {
    const int i = e / l, j = e % l;
    if (i < j) { const double a = 0.5 * (W[i * ls + j] + W[j * ls + i]); Lm[i * ls + j] = a; Lm[j * ls + i] = a; }
    else if (i == j) Lm[i * ls + j] = W[i * ls + j];
  }
  __syncthreads();
  for (int e = tid; e < l * l; e += blockDim.x) { const int o = (e / l) * ls + e % l; W[o] = Lm[o]; }
  __syncthreads();
  double trace = 0.0;
  for (int i = 0; i < l; ++i) trace += W[i * ls + i];
  double shift = 0.0;
  for (int attempt = 0; attempt < 6; ++attempt) {
    for (int e = tid; e < l * l; e += blockDim.x) {
      const int i = e / l, j = e % l;
      Lm[i * ls + j] = W[i * ls + j] + ((i == j) ? shift : 0.0);
    }
    __syncthreads();
    // Right-looking Cholesky on the lower triangle, one barrier per column: in phase j every thread reads the
    // pivot d_j itself (so a bad pivot is seen by all alike), the trailing block is updated from the UNSCALED
    // column j times 1/d_j, and column j-1 (which nobody reads any more) is scaled in passing.
    // (one reciprocal square root per column and thread: 1/d = rsqrt(d)^2, sqrt(d) = d rsqrt(d); a division and a
    // square root in fp64 cost several hundred cycles of latency each, more than the rest of the column)
    bool failed = false;
    double sd_prev = 1.0, isd_prev = 1.0;
    const int ti = tid >> 6, tc = tid & 63;        // 8 rows x 64 columns of the trailing block per pass
    for (int j = 0; j < l; ++j) {
      const double d = Lm[j * ls + j];
      if (!(d > 0.0) || !isfinite(d)) { failed = true; break; }
      const double isd = rsqrt(d), inv_d = isd * isd;
      if (j > 0) {
        for (int i = j - 1 + tid; i < l; i += blockDim.x) Lm[i * ls + j - 1] = (i == j - 1) ? sd_prev : Lm[i * ls + j - 1] * isd_prev;
      }
      const int c = j + 1 + tc;
      if (c < l) {
        const double lc = Lm[c * ls + j] * inv_d;
        // all loads of the thread's (up to MAX_L / 8) rows first, then the updates: written as one loop, every
        // iteration's loads wait for the previous iteration's store (the compiler cannot tell they do not alias)
        double a[MAX_L / 8], bj[MAX_L / 8];
#pragma unroll
        for (int u = 0; u < MAX_L / 8; ++u) {
          const int i = j + 1 + ti + 8 * u;
          const bool on = i < l && c <= i;
          a[u] = on ? Lm[i * ls + c] : 0.0;
          bj[u] = on ? Lm[i * ls + j] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < MAX_L / 8; ++u) {
          const int i = j + 1 + ti + 8 * u;
          if (i < l && c <= i) Lm[i * ls + c] = a[u] - bj[u] * lc;
        }
      }
      sd_prev = d * isd; isd_prev = isd;
      __syncthreads();
    }
    if (!failed && tid == 0) Lm[(l - 1) * ls + l - 1] = sd_prev;
    if (tid == 0) bad = failed ? 1 : 0;
    __syncthreads();
    if (!bad) break;
    // shift as in shifted CholeskyQR: proportional to the trace, growing per attempt
    shift = (shift == 0.0) ? 1e-10 * (trace > 0.0 ? trace : 1.0) : shift * 100.0;
    if (tid == 0 && status) atomicOr(&status[bz], 1);
    __syncthreads();
  }
  // Linv by forward substitution, one column per thread: L X = I
  // X[:,c] for c: x_c = 1/L_cc; x_i = -(sum_{t=c}^{i-1} L_it x_t)/L_ii
  __syncthreads();
  double* X = W;   // reuse
  for (int e = tid; e < l * ls; e += blockDim.x) X[e] = 0.0;
  if (tid < l) rdiag[tid] = bad ? 0.0 : 1.0 / Lm[tid * ls + tid];
  __syncthreads();
  if (!bad) {
    // Eight lanes per column c of X = L^-1 (blockDim / 8 = 64 columns at once), column-oriented: lane `sub` keeps,
    // in registers, the running sums s_r = sum_{k<i} L_rk x_k of the rows r = sub (mod 8). Step i: the owner of row i
    // hands s_i to the group (one shuffle), everybody forms x_i = (delta_ic - s_i) / L_ii, and adds L_ri x_i to its
    // sums of the rows below. Per step that is one shuffle and one multiply on the critical path and at most
    // MAX_L / 8 independent multiply-adds per lane; the row-oriented form (a dot product split over the lanes,
    // three shuffle levels and a warp barrier per row) spent 2.5x the fp64 instructions, which is what bounds it.
    const int c = tid >> 3, sub = tid & 7;
    const int c_warp0 = (tid >> 5) * 4;          // first column of this warp
    double srow[MAX_L / 8];
#pragma unroll
    for (int u = 0; u < MAX_L / 8; ++u) srow[u] = 0.0;
    if (c_warp0 < l) {                           // (a warp whose four columns all lie beyond l has nothing to do)
#pragma unroll
      for (int u = 0; u < MAX_L / 8; ++u) {
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          const int i = 8 * u + w;
          if (i < l && i >= c_warp0) {           // uniform in the warp: rows above its first column give x_i = 0
            const double si = __shfl_sync(0xffffffffu, srow[u], w, 8);
            double xi = 0.0;
            if (c < l && i >= c) xi = ((i == c) ? 1.0 - si : -si) * rdiag[i];
            if (sub == w && c < l) X[i * ls + c] = xi;
#pragma unroll
            for (int u2 = u; u2 < MAX_L / 8; ++u2) {
              const int r = 8 * u2 + sub;
              if (r > i && r < l) srow[u2] = fma(Lm[r * ls + i], xi, srow[u2]);
            }
          }
        }
      }
    }
  }
  __syncthreads();
  // Rinv = Linv^T (upper triangular)
  float* out = Rinv + (long long)bz * l * l;
  for (int e = tid; e < l * l; e += blockDim.x) {
    const int i = e / l, j = e % l;
    out[e] = (float)X[j * ls + i];
  }
}

cudaError_t chol_inv_launch(const double* partial, int nchunk, int batch, int l, float* Rinv, int* status,
                            cudaStream_t st, long long* launches) {
  const size_t smem = 2 * (size_t)MAX_L * (MAX_L + 1) * sizeof(double);
  // (the attribute belongs to the current device's copy of the kernel: set at every launch, a host-side call)
  cudaFuncSetAttribute(chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  chol_inv_kernel<<<batch, 512, smem, st>>>(partial, nchunk, l, Rinv, status);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Out[b, rows, kout] = In[b, rows, l] * Mtx[b, l(, ldm)] (first kout columns of Mtx). In-place safe.
// ---------------------------------------------------------------------------------------------
constexpr int PA_ROWS = 64;
__global__ void __launch_bounds__(256) panel_apply_kernel(const float* In, long long in_bs, int ld_in,
                                                          const float* __restrict__ Mtx, int ldm, int rows, int l,
                                                          int kout, float* Out, long long out_bs, int ld_out) {
  __shared__ float tile[PA_ROWS][MAX_L + 1];
  __shared__ float mt[MAX_L][MAX_L + 1];
  const int bz = blockIdx.y, tid = threadIdx.x;
  const int r0 = blockIdx.x * PA_ROWS;
  const float* Ib = In + (long long)bz * in_bs;
  const float* Mb = Mtx + (long long)bz * l * ldm;
  for (int e = tid; e < l * kout; e += 256) mt[e / kout][e % kout] = Mb[(e / kout) * ldm + (e % kout)];
  for (int e = tid; e < PA_ROWS * l; e += 256) {
    const int rr = e / l, c = e % l;
    tile[rr][c] = (r0 + rr < rows) ? Ib[(long long)(r0 + rr) * ld_in + c] : 0.f;
  }
  __syncthreads();
  float* Ob = Out + (long long)bz * out_bs;
  for (int e = tid; e < PA_ROWS * kout; e += 256) {
    const int rr = e / kout, c = e % kout;
    if (r0 + rr >= rows) continue;
    float t = 0.f;
    for (int q = 0; q < l; ++q) t = fmaf(tile[rr][q], mt[q][c], t);
    Ob[(long long)(r0 + rr) * ld_out + c] = t;
  }
}

cudaError_t panel_apply_launch(const float* In, long long in_bs, int ld_in, const float* Mtx, int ldm, int batch,
                               int rows, int l, int kout, float* Out, long long out_bs, int ld_out, cudaStream_t st,
                               long long* launches) {
  if (kout <= 0) return cudaSuccess;
  panel_apply_kernel<<<dim3((rows + PA_ROWS - 1) / PA_ROWS, batch), 256, 0, st>>>(In, in_bs, ld_in, Mtx, ldm, rows, l,
                                                                                 kout, Out, out_bs, ld_out);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// One-sided Jacobi eigensolver of the symmetric positive semidefinite core C = sum of partials
// (l x l). Columns of A = C V are rotated pairwise until mutually orthogonal; then ||a_j|| are the
// eigenvalues and V the eigenvectors. One warp per column pair (round-robin pairing), lanes over
// rows, dot products by warp shuffles; fp64 throughout. Outputs (sorted by decreasing eigenvalue):
//   s[b, l]     = sqrt(eigenvalue)             (singular values of the panel whose Gram this is)
//   E[b, l, l]  = eigenvectors in columns      (fp32)
//   Es[b, l, l] = E diag(1/s)                  (fp32; zero column where s is numerically zero)
// With `signed_input` the matrix is a general symmetric one (Rayleigh quotient of Algorithm 2):
// eigenvalues keep their sign (lambda_j = v_j^T a_j), sorted by decreasing magnitude, s = lambda.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// eight lanes of a warp add up their values (the lanes sub = 0..7 of one column pair)
__device__ __forceinline__ double group8_sum(double v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  return v;
}

constexpr int JAC_THREADS = 256;        // 32 column pairs x 8 lanes
constexpr int JAC_NR = MAX_L / 8;       // rows per lane

__global__ void __launch_bounds__(JAC_THREADS) jacobi_eig_kernel(const double* __restrict__ partial, int nchunk, int l,
                                                                 int signed_input, float* __restrict__ s_out,
                                                                 float* __restrict__ E, float* __restrict__ Es,
                                                                 int* __restrict__ status, int max_sweeps) {
  extern __shared__ double sm[];
  const int ls = l | 1;       // column stride (odd: the four pairs of a warp start in different banks)
  double* A = sm;             // column-major: A[c * ls + r]
  double* V = sm + MAX_L * (MAX_L + 1);     // column-major
  __shared__ double lam[MAX_L];
  __shared__ double nrm2[MAX_L];      // squared column norms of A, carried along by the rotations
  __shared__ int order[MAX_L];
  __shared__ int rotated;
  const int bz = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const double* pb = partial + (long long)bz * nchunk * l * l;
  for (int e = tid; e < l * l; e += blockDim.x) {
    const int r = e / l, c = e % l;
    double t = 0.0, u = 0.0;
    for (int ch = 0; ch < nchunk; ++ch) {
      t += pb[(long long)ch * l * l + r * l + c];
      u += pb[(long long)ch * l * l + c * l + r];
    }
    A[c * ls + r] = 0.5 * (t + u);
    V[c * ls + r] = (r == c) ? 1.0 : 0.0;
  }
  __syncthreads();
  const int np = (l + 1) & ~1;        // players, padded to even
  const int npairs = np / 2;
  // Eight lanes per column pair, four pairs per warp: the three dot products of a pair take three shuffle steps
  // each instead of five, and a round issues a sixth of the shuffles of the one-warp-per-pair form (whose
  // shuffle traffic, not its arithmetic, filled the round).
  const int grp = tid >> 3, sub = tid & 7;
  const int nr = (l + 7) >> 3;        // rows per lane actually present
  // The eigenvector accumulation V is needed only for a signed spectrum (to tell the sign of an eigenvalue). For
  // a Gram matrix the columns of A converge to lambda_j v_j with lambda_j >= 0, so the eigenvectors are the
  // normalised columns: the rotations skip V, a third of the fp64 work (fp64 issue is what bounds this kernel).
  const bool track_v = signed_input != 0;
  int sweep = 0;
  for (; sweep < max_sweeps; ++sweep) {
    if (tid == 0) rotated = 0;
    // Squared column norms, exact at the start of every sweep. Within the sweep a rotation by tan t moves
    // t gamma from one column's squared norm to the other's (alpha' = alpha - t gamma, beta' = beta + t gamma), so
    // a round computes one dot product per pair instead of three; the sweep that finds nothing to rotate, which
    // ends the iteration, has tested every pair against exact norms.
    for (int j0 = 0; j0 < l; j0 += JAC_THREADS / 8) {      // (the same trip count for every lane: shuffles inside)
      const int j = j0 + grp;
      double acc = 0.0;
#pragma unroll
      for (int i = 0; i < JAC_NR; ++i) {
        const int r = sub + 8 * i;
        if (i < nr && r < l && j < l) { const double v = A[j * ls + r]; acc = fma(v, v, acc); }
      }
      acc = group8_sum(acc);
      if (sub == 0 && j < l) nrm2[j] = acc;
    }
    __syncthreads();
    for (int round = 0; round < np - 1; ++round) {
      int p = 0, q = l;
      if (grp < npairs) {
        if (grp == 0) { p = np - 1; q = round; }
        else {
          // (round + grp) and (round - grp) modulo np - 1: both lie within one period of the range
          p = round + grp; if (p >= np - 1) p -= np - 1;
          q = round - grp; if (q < 0) q += np - 1;
        }
        if (p > q) { const int t = p; p = q; q = t; }
      }
      const bool live = q < l;            // (a pair with the padding player, or a group beyond the pairs, idles)
      double* ap = A + p * ls; double* aq = A + (live ? q : p) * ls;
      double x[JAC_NR], y[JAC_NR];
      double pg = 0.0;
#pragma unroll
      for (int i = 0; i < JAC_NR; ++i) {
        if (i < nr) {
          const int r = sub + 8 * i;
          const bool in = live && r < l;
          x[i] = in ? ap[r] : 0.0;
          y[i] = in ? aq[r] : 0.0;
          pg = fma(x[i], y[i], pg);
        }
      }
      const double gamma = group8_sum(pg);
      const double alpha = live ? nrm2[p] : 0.0, beta = live ? nrm2[q] : 0.0;
      // rotate when |gamma| > 1e-11 sqrt(alpha beta) (compared in squares): the eigenvalues are then good to about
      // 1e-22 and the vectors to 1e-11 over the relative gap, far beyond the fp32 outputs
      if (live && gamma != 0.0 && gamma * gamma > 1e-22 * (alpha * beta)) {
        if (sub == 0) rotated = 1;
        // The rotation angle only steers the iteration (any exact rotation keeps V orthogonal and the invariants
        // intact), so tan is computed in fp32 from the exponent-scaled pair (beta - alpha, 2 gamma); cos comes
        // from an fp32 reciprocal square root refined by two Newton steps in fp64, which makes c^2 + s^2 = 1 hold
        // to fp64 rounding. A rotation then leaves 1e-7 of the inner product instead of none, and the pair's
        // next visit removes that. The chain of dependent fp64 operations, which is the latency of a round,
        // shrinks to a third. Out-of-range exponents take the fp64 formula.
        const double d = beta - alpha, g2 = 2.0 * gamma;
        const double big = fmax(fabs(d), fabs(g2));
        const int ex = (int)((__double_as_longlong(big) >> 52) & 0x7ff);
        const double sc = __longlong_as_double((long long)(2046 - ex) << 52);       // 2^(1023 - ex)
        const float df = (float)(d * sc), gf = (float)(g2 * sc);
        double c, sn, tg;
        if (ex >= 1 && ex <= 2045 && fabsf(gf) > 1e-30f) {
          const float zf = df / gf, az = fabsf(zf);
          // t = sign(zeta) / (|zeta| + sqrt(1 + zeta^2)): the root of t^2 + 2 zeta t - 1 = 0 of smaller magnitude
          const float tf = (az > 1e15f) ? 0.5f / zf : copysignf(1.0f / (az + sqrtf(fmaf(zf, zf, 1.0f))), zf);
          const double t = (double)tf;
          const double w = fma(t, t, 1.0), h = 0.5 * w;            // w in [1, 2]
          double yv = (double)rsqrtf((float)w);
          yv = yv * fma(-h * yv, yv, 1.5);
          yv = yv * fma(-h * yv, yv, 1.5);
          c = yv; sn = yv * t;
          tg = t * gamma;
        } else {
          const double zeta = d / g2;
          const double w = 1.0 + zeta * zeta;
          const double root = w * rsqrt(w);                          // sqrt(1 + zeta^2)
          const double t = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + root);
          c = rsqrt(1.0 + t * t); sn = c * t;
          tg = t * gamma;
        }
        if (sub == 0) { nrm2[p] = alpha - tg; nrm2[q] = beta + tg; }
        double* vp = V + p * ls; double* vq = V + q * ls;
#pragma unroll
        for (int i = 0; i < JAC_NR; ++i) {
          const int r = sub + 8 * i;
          if (i < nr && r < l) {
            ap[r] = c * x[i] - sn * y[i]; aq[r] = sn * x[i] + c * y[i];
            if (track_v) {
              const double a = vp[r], b = vq[r];
              vp[r] = c * a - sn * b; vq[r] = sn * a + c * b;
            }
          }
        }
      }
      __syncthreads();
    }
    if (!rotated) break;
    __syncthreads();
  }
  if (tid == 0 && sweep >= max_sweeps && status) atomicOr(&status[bz], 2);
  // eigenvalues
  if (warp < 32) {
    for (int j = warp; j < l; j += (blockDim.x >> 5)) {
      const double* aj = A + j * ls; const double* vj = V + j * ls;
      const double a0 = (lane < l) ? aj[lane] : 0.0, a1 = (lane + 32 < l) ? aj[lane + 32] : 0.0;
      const double v0 = (lane < l) ? vj[lane] : 0.0, v1 = (lane + 32 < l) ? vj[lane + 32] : 0.0;
      const double nrm = sqrt(warp_sum(a0 * a0 + a1 * a1));
      const double rq = warp_sum(a0 * v0 + a1 * v1);
      if (lane == 0) lam[j] = signed_input ? ((rq >= 0.0) ? nrm : -nrm) : nrm;
      if (!track_v) {
        // v_j = a_j / lambda_j; a column that vanished (rank-deficient input) keeps its unit vector, which only
        // ever meets a zero singular value
        const double inv = (nrm > 1e-150) ? 1.0 / nrm : 0.0;
        if (nrm > 1e-150) {
          if (lane < l) V[j * ls + lane] = a0 * inv;
          if (lane + 32 < l) V[j * ls + lane + 32] = a1 * inv;
        }
      }
    }
  }
  __syncthreads();
  if (tid < l) {
    // (a NaN compares false with everything: it ranks as magnitude -1, after every number, so that `order` is a
    // permutation whatever the input holds)
    double mine = fabs(lam[tid]);
    if (!(mine == mine)) mine = -1.0;
    int rank = 0;
    for (int i = 0; i < l; ++i) {
      double o = fabs(lam[i]);
      if (!(o == o)) o = -1.0;
      if (o > mine || (o == mine && i < tid)) ++rank;
    }
    order[rank] = tid;
  }
  __syncthreads();
  for (int e = tid; e < l * l; e += blockDim.x) {
    const int r = e / l, cc = e % l;
    const int src = order[cc];
    const double v = V[src * ls + r];
    const double lm = lam[src];
    const double sv = signed_input ? lm : sqrt(lm > 0.0 ? lm : 0.0);
    if (E) E[(long long)bz * l * l + e] = (float)v;
    if (Es) Es[(long long)bz * l * l + e] = (fabs(sv) > 1e-300) ? (float)(v / sv) : 0.f;
    if (r == 0 && s_out) s_out[(long long)bz * l + cc] = (float)sv;
  }
}

cudaError_t jacobi_eig_launch(const double* partial, int nchunk, int batch, int l, int signed_input, float* s_out,
                              float* E, float* Es, int* status, cudaStream_t st, long long* launches, int max_sweeps) {
  const size_t smem = 2 * (size_t)MAX_L * (MAX_L + 1) * sizeof(double);
  cudaFuncSetAttribute(jacobi_eig_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  jacobi_eig_kernel<<<batch, JAC_THREADS, smem, st>>>(partial, nchunk, l, signed_input, s_out, E, Es, status,
                                                      max_sweeps > 0 ? max_sweeps : 40);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Frobenius partial sums of a [b, count] array (bf16 or fp32): partial[b, nblk] in fp64.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) frob_partial_kernel(const void* __restrict__ X, int dtype, long long count,
                                                           int nblk, double* __restrict__ partial) {
  __shared__ double red[8];
  const int bz = blockIdx.y, tid = threadIdx.x;
  const long long per = (count + nblk - 1) / nblk;
  const long long lo = (long long)blockIdx.x * per, hi = min(count, lo + per);
  const long long base = (long long)bz * count;
  double acc = 0.0;
  float f = 0.f;
  int n = 0;
  for (long long i = lo + tid; i < hi; i += 256) {
    const float v = ld_as_float(X, base + i, dtype);
    f = fmaf(v, v, f);
    if (++n == 16) { acc += (double)f; f = 0.f; n = 0; }
  }
  acc += (double)f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if ((tid & 31) == 0) red[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red[w];
    partial[(long long)bz * nblk + blockIdx.x] = t;
  }
}

cudaError_t frob_partial_launch(const void* X, int dtype, int batch, long long count, int nblk, double* partial,
                                cudaStream_t st, long long* launches) {
  frob_partial_kernel<<<dim3(nblk, batch), 256, 0, st>>>(X, dtype, count, nblk, partial);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// rho[b] = sqrt(sum of partials); one warp per matrix, lane-strided sums then a shuffle tree (fixed order);
// inv_rho[b] = 1/rho (0 and status bit 4 when rho is 0 or not finite)
__global__ void rho_finalize_kernel(const double* __restrict__ partial, int nper, int batch, float* __restrict__ rho,
                                    float* __restrict__ inv_rho, float* __restrict__ inv_rho2,
                                    int* __restrict__ status) {
  const int bz = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (bz >= batch) return;
  double t = 0.0;
  for (int i = lane; i < nper; i += 32) t += partial[(long long)bz * nper + i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if (lane != 0) return;
  const double r = sqrt(t);
  const bool ok = (r > 0.0) && isfinite(r);
  if (rho) rho[bz] = (float)r;
  if (inv_rho) inv_rho[bz] = ok ? (float)(1.0 / r) : 0.f;
  if (inv_rho2) inv_rho2[bz] = ok ? (float)(1.0 / t) : 0.f;
  if (!ok && status) atomicOr(&status[bz], 4);
}

cudaError_t rho_finalize_launch(const double* partial, int nper, int batch, float* rho, float* inv_rho,
                                float* inv_rho2, int* status, cudaStream_t st, long long* launches) {
  rho_finalize_kernel<<<(batch + 3) / 4, 128, 0, st>>>(partial, nper, batch, rho, inv_rho, inv_rho2, status);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Frobenius partial sums with 16-byte loads: CTA (blk, batch) sums a contiguous run of whole 16-byte packets (fp32
// sums of at most 64 squares per thread, then fp64), partial[b, nblk]. The leftover elements of a matrix whose
// size is not a whole number of packets go to the last CTA. Needs a 16-byte aligned base and matrix stride.
template <typename T, int V>
__global__ void __launch_bounds__(256) frob_partial_vec_kernel(const T* __restrict__ X, long long count, int nblk,
                                                               double* __restrict__ partial) {
  struct alignas(16) Pack { T v[V]; };
  __shared__ double red[8];
  const int bz = blockIdx.y, tid = threadIdx.x;
  const T* Xb = X + (long long)bz * count;
  const long long nvec = count / V;
  const long long per = (nvec + nblk - 1) / nblk;
  const long long lo = (long long)blockIdx.x * per, hi = min(nvec, lo + per);
  double acc = 0.0;
  const Pack* P = reinterpret_cast<const Pack*>(Xb);
  long long i = lo + tid;
  // four packets per thread in flight
  for (; i + 3 * 256 < hi; i += 4 * 256) {
    Pack q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) q[u] = P[i + u * 256];
    float f = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int j = 0; j < V; ++j) { const float v = (float)q[u].v[j]; f = fmaf(v, v, f); }
    acc += (double)f;
  }
  for (; i < hi; i += 256) {
    const Pack q = P[i];
    float f = 0.f;
#pragma unroll
    for (int j = 0; j < V; ++j) { const float v = (float)q.v[j]; f = fmaf(v, v, f); }
    acc += (double)f;
  }
  if (blockIdx.x == nblk - 1) {
    for (long long e = nvec * V + tid; e < count; e += 256) { const float v = (float)Xb[e]; acc += (double)v * (double)v; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if ((tid & 31) == 0) red[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red[w];
    partial[(long long)bz * nblk + blockIdx.x] = t;
  }
}

cudaError_t frob_partial_vec_launch(const void* X, int dtype, int batch, long long count, int nblk, double* partial,
                                    cudaStream_t st, long long* launches) {
  const int es = (int)dtype_size(dtype);
  const bool aligned = (reinterpret_cast<uintptr_t>(X) & 15) == 0 && ((count * es) & 15) == 0;
  if (!aligned || dtype == F16) return frob_partial_launch(X, dtype, batch, count, nblk, partial, st, launches);
  if (dtype == BF16) frob_partial_vec_kernel<__nv_bfloat16, 8><<<dim3(nblk, batch), 256, 0, st>>>((const __nv_bfloat16*)X, count, nblk, partial);
  else frob_partial_vec_kernel<float, 4><<<dim3(nblk, batch), 256, 0, st>>>((const float*)X, count, nblk, partial);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// rho[b] from the identity ||A - U_k diag(s) V_k^T||_F^2 = ||A||_F^2 - sum_{i < keff} s_i^2 (triplets of Algorithm 3):
// one warp per matrix adds the partial sums of ||A||_F^2 (fixed order), lane 0 subtracts the squares in fp64.
// A difference below 1e-6 ||A||_F^2 is below what the fp32 singular values resolve: the residual counts as zero
// (status bit 4, 1/rho = 0), as does a non-finite one.
__global__ void rho_identity_kernel(const double* __restrict__ partial, int nper, int batch, const float* __restrict__ s,
                                    int ld_s, const int* __restrict__ keff, float* __restrict__ rho,
                                    float* __restrict__ inv_rho, float* __restrict__ inv_rho2, int* __restrict__ status) {
  const int bz = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (bz >= batch) return;
  double t = 0.0;
  for (int i = lane; i < nper; i += 32) t += partial[(long long)bz * nper + i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if (lane != 0) return;
  const double total = t;
  const int ke = keff[bz];
  for (int i = 0; i < ke; ++i) { const double v = (double)s[(long long)bz * ld_s + i]; t -= v * v; }
  const bool ok = isfinite(t) && t > 1e-6 * total;
  const double r = ok ? sqrt(t) : 0.0;
  if (rho) rho[bz] = (float)r;
  if (inv_rho) inv_rho[bz] = ok ? (float)(1.0 / r) : 0.f;
  if (inv_rho2) inv_rho2[bz] = ok ? (float)(1.0 / t) : 0.f;
  if (!ok && status) atomicOr(&status[bz], 4);
}

cudaError_t rho_identity_launch(const double* partial, int nper, int batch, const float* s, int ld_s, const int* keff,
                                float* rho, float* inv_rho, float* inv_rho2, int* status, cudaStream_t st,
                                long long* launches) {
  rho_identity_kernel<<<(batch + 3) / 4, 128, 0, st>>>(partial, nper, batch, s, ld_s, keff, rho, inv_rho, inv_rho2, status);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Non-finite results are reported, not returned silently: one CTA per matrix looks at the first 4096 elements and at
// 4096 more spread evenly over the matrix, and raises bit 16 of status[b] when one of them is Inf or NaN. A sample is
// enough: a non-finite entry of an iterate (non-finite input, or a value that left the range of the iterate's
// storage format) reaches the Gram matrix of the next step and from there every entry of the following iterate.
__global__ void __launch_bounds__(256) finite_probe_kernel(const void* __restrict__ X, int dtype, long long count,
                                                           int* __restrict__ status) {
  const int bz = blockIdx.x, tid = threadIdx.x;
  const long long base = (long long)bz * count;
  const long long head = min(count, (long long)4096);
  const long long stride = max((long long)1, count / 4096);
  bool bad = false;
  for (long long i = tid; i < head; i += 256) bad |= !isfinite(ld_as_float(X, base + i, dtype));
  for (long long j = tid; j < 4096 && j * stride < count; j += 256) bad |= !isfinite(ld_as_float(X, base + j * stride, dtype));
  if (__syncthreads_or(bad ? 1 : 0) && tid == 0) atomicOr(&status[bz], 16);
}

cudaError_t finite_probe_launch(const void* X, int dtype, int batch, long long count, int* status, cudaStream_t st,
                                long long* launches) {
  if (batch <= 0 || count <= 0) return cudaSuccess;
  finite_probe_kernel<<<batch, 256, 0, st>>>(X, dtype, count, status);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Out[b, rows, k] = In[b, rows, (ld_in)] * diag(coef): coef_t = c0 * s[b,t] * (use_inv ? inv_rho[b] : 1) + c1
__global__ void scale_cols_kernel(const float* __restrict__ In, long long in_bs, int ld_in, int rows, int k,
                                  const float* __restrict__ s, int ld_s, const float* __restrict__ inv_rho, float c0,
                                  float c1, float* __restrict__ Out, long long out_bs, int ld_out,
                                  const int* __restrict__ keff) {
  const int bz = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)rows * k) return;
  const int r = (int)(e / k), t = (int)(e % k);
  float sc = c0 * s[(long long)bz * ld_s + t] * (inv_rho ? inv_rho[bz] : 1.f) + c1;
  if (keff && t >= keff[bz]) sc = 0.f;     // column not deflated for this matrix (gate)
  Out[(long long)bz * out_bs + (long long)r * ld_out + t] = In[(long long)bz * in_bs + (long long)r * ld_in + t] * sc;
}

cudaError_t scale_cols_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int k, const float* s,
                              int ld_s, const float* inv_rho, float c0, float c1, float* Out, long long out_bs,
                              int ld_out, cudaStream_t st, long long* launches, const int* keff) {
  if (k <= 0) return cudaSuccess;
  const long long tot = (long long)rows * k;
  scale_cols_kernel<<<dim3((unsigned)((tot + 255) / 256), batch), 256, 0, st>>>(In, in_bs, ld_in, rows, k, s, ld_s,
                                                                               inv_rho, c0, c1, Out, out_bs, ld_out, keff);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Out[b, i] = scale[b] * In[b, i]  (type conversion allowed)
__global__ void scale_kernel(const void* __restrict__ In, int in_dt, void* __restrict__ Out, int out_dt,
                             long long count, const float* __restrict__ scale, int round_tf32, float mult) {
  const int bz = blockIdx.y;
  const float sc = (scale ? scale[bz] : 1.f) * mult;
  const long long base = (long long)bz * count;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x)
  {
    float v = sc * ld_as_float(In, base + i, in_dt);
    if (round_tf32) v = round_to_tf32(v);
    st_from_float(Out, base + i, out_dt, v);
  }
}

cudaError_t scale_launch(const void* In, int in_dt, void* Out, int out_dt, int batch, long long count,
                         const float* scale, cudaStream_t st, long long* launches, int round_tf32, float mult) {
  const int nblk = (int)min((long long)1184, (count + 255) / 256);
  scale_kernel<<<dim3(nblk, batch), 256, 0, st>>>(In, in_dt, Out, out_dt, count, scale, round_tf32, mult);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Counter-based Gaussian fill (the generator documented in the public header).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

__global__ void fill_gaussian_kernel(void* __restrict__ dst, long long count, int dtype, unsigned long long seed,
                                     long long per_stream, unsigned long long seed_stride) {
  // element e belongs to stream e / per_stream (seed + stream * seed_stride), index e % per_stream
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < count;
       e += (long long)gridDim.x * blockDim.x) {
    const unsigned long long stream = per_stream > 0 ? (unsigned long long)(e / per_stream) : 0ull;
    const unsigned long long idx = per_stream > 0 ? (unsigned long long)(e % per_stream) : (unsigned long long)e;
    const unsigned long long hs = mix64(seed + stream * seed_stride);
    const unsigned long long j = idx >> 1;
    const unsigned long long r1 = mix64(hs ^ (2ull * j)), r2 = mix64(hs ^ (2ull * j + 1ull));
    const double u1 = ((double)(r1 >> 11) + 1.0) * (1.0 / 9007199254740992.0);
    const double u2 = (double)(r2 >> 11) * (1.0 / 9007199254740992.0);
    const double rad = sqrt(-2.0 * log(u1));
    double sn, cs;
    sincos(6.283185307179586476925286766559 * u2, &sn, &cs);
    st_from_float(dst, e, dtype, (float)((idx & 1ull) ? rad * sn : rad * cs));
  }
}

cudaError_t fill_gaussian_launch(void* dst, long long count, int dtype, unsigned long long seed, long long per_stream,
                                 unsigned long long seed_stride, cudaStream_t st, long long* launches) {
  if (count <= 0) return cudaSuccess;
  const int nblk = (int)min((long long)2368, (count + 255) / 256);
  fill_gaussian_kernel<<<nblk, 256, 0, st>>>(dst, count, dtype, seed, per_stream, seed_stride);
  if (launches) ++*launches;
  return cudaGetLastError();
}

__global__ void fill_int_kernel(int* p, int n, int v) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}
cudaError_t fill_int_launch(int* p, int n, int v, cudaStream_t st, long long* launches) {
  if (n <= 0) return cudaSuccess;
  fill_int_kernel<<<(n + 255) / 256, 256, 0, st>>>(p, n, v);
  if (launches) ++*launches;
  return cudaGetLastError();
}

}  // namespace defl

namespace defl {
__global__ void or_status_kernel(int* status, int n, const int* word) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) status[i] |= *word;
}
cudaError_t or_status_launch(int* status, int n, const int* word, cudaStream_t st, long long* launches) {
  if (n <= 0) return cudaSuccess;
  or_status_kernel<<<(n + 255) / 256, 256, 0, st>>>(status, n, word);
  if (launches) ++*launches;
  return cudaGetLastError();
}
}  // namespace defl

// ---------------------------------------------------------------------------------------------
// Allocation-free batched Frobenius norm (see defl_frobenius_norms_noalloc in the public header).
// The partial sums that frob_partial_kernel normally writes into context-owned scratch go into a
// fixed file-scope device array instead, so the call needs no cudaMalloc at all.
// ---------------------------------------------------------------------------------------------
#include "../../include/defl.h"
#include <mutex>

namespace defl {
constexpr int NOALLOC_NBLK = 148;   // partial sums per matrix (one per CTA)
static __device__ __align__(256) double g_noalloc_partials[DEFL_NOALLOC_MAX_BATCH * NOALLOC_NBLK];

constexpr int NOALLOC_MAX_DEVICES = 64;
static double* g_noalloc_ptr[NOALLOC_MAX_DEVICES];   // device address of the array, per device
static std::mutex g_noalloc_mutex;
}  // namespace defl

extern "C" int defl_frobenius_norms_noalloc(const void* X, int dtype, int b, long long count, float* norms,
                                            void* cuda_stream) {
  using namespace defl;
  if (!X || !norms || b <= 0 || count <= 0 || (dtype != DEFL_BF16 && dtype != DEFL_F32)) return DEFL_ERR_ARG;
  if (b > DEFL_NOALLOC_MAX_BATCH) return DEFL_ERR_RANK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return DEFL_ERR_CUDA;
  double* scratch = nullptr;
  {
    // First call on this device: ask the runtime where this device's copy of the array lives. The
    // array's name is only a host-side handle here; a kernel must be given the looked-up address.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || !p) return DEFL_ERR_CUDA;
      g_noalloc_ptr[dev] = reinterpret_cast<double*>(p);
    }
    scratch = g_noalloc_ptr[dev];
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // every slot read by the second kernel is written by the first, so nothing needs clearing
  frob_partial_kernel<<<dim3(NOALLOC_NBLK, b), 256, 0, st>>>(X, dtype, count, NOALLOC_NBLK, scratch);
  if (cudaGetLastError() != cudaSuccess) return DEFL_ERR_CUDA;
  rho_finalize_kernel<<<(b + 3) / 4, 128, 0, st>>>(scratch, NOALLOC_NBLK, b, norms, nullptr, nullptr, nullptr);
  if (cudaGetLastError() != cudaSuccess) return DEFL_ERR_CUDA;
  return DEFL_OK;
}

// ---------------------------------------------------------------------------------------------
// Split-precision copies of fp32 panels for the tensor engine: x = hi + lo with hi = bf16(x),
// lo = bf16(x - hi) (about 16 significant bits together).
// ---------------------------------------------------------------------------------------------
namespace defl {

// hi, lo [b, rows, lp] from In [b, rows, l] (leading dimension ld_in); columns l..lp-1 are zero.
__global__ void split_panel_kernel(const float* __restrict__ In, long long in_bs, int ld_in, int rows, int l, int lp,
                                   __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  const int bz = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)rows * lp) return;
  const int r = (int)(e / lp), c = (int)(e % lp);
  const float x = (c < l) ? In[(long long)bz * in_bs + (long long)r * ld_in + c] : 0.f;
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  const long long o = (long long)bz * rows * lp + e;
  hi[o] = h;
  lo[o] = __float2bfloat16_rn(x - __bfloat162float(h));
}

cudaError_t split_panel_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int l, int lp,
                               __nv_bfloat16* hi, __nv_bfloat16* lo, cudaStream_t st, long long* launches) {
  const long long tot = (long long)rows * lp;
  split_panel_kernel<<<dim3((unsigned)((tot + 255) / 256), batch), 256, 0, st>>>(In, in_bs, ld_in, rows, l, lp, hi, lo);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Out [b, rows, 3*kp] (16-bit) = three column blocks of the (optionally column-scaled) panel In [b, rows, k]:
//   pattern 0: [hi | hi | lo]      pattern 1: [hi | lo | hi]
// so that  Out0 * Out1^T = hi hi^T + hi lo^T + lo hi^T  (the product of the two fp32 panels up to the lo*lo term).
// Column t is scaled by  mult * (c0 * s[b,t] * (inv_rho ? inv_rho[b] : 1) + c1 * (rho ? rho[b] : 1))  (without s: by mult alone).
// The two halves are bf16 or, with `f16`, IEEE half (the type of the product they enter); with `transposed` the
// copy is stored as [b, 3*kp, rows], the layout of an operand whose long side is contiguous.
template <bool F16, bool TRANSPOSED>
__global__ void split_concat3_kernel(const float* __restrict__ In, long long in_bs, int ld_in, int rows, int k, int kp,
                                     const float* __restrict__ s, int ld_s, const float* __restrict__ inv_rho, float c0,
                                     float c1, float mult, int pattern, uint16_t* __restrict__ Out,
                                     const int* __restrict__ keff, const float* __restrict__ rho) {
  const int bz = blockIdx.y;
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)rows * kp) return;
  // consecutive threads walk the contiguous direction of the output
  const int r = TRANSPOSED ? (int)(e % rows) : (int)(e / kp), t = TRANSPOSED ? (int)(e / rows) : (int)(e % kp);
  float x = 0.f;
  if (t < k && !(keff && t >= keff[bz])) {
    x = In[(long long)bz * in_bs + (long long)r * ld_in + t] * mult;
    if (s) x *= c0 * s[(long long)bz * ld_s + t] * (inv_rho ? inv_rho[bz] : 1.f) + c1 * (rho ? rho[bz] : 1.f);
  }
  uint16_t h, lw;
  if (F16) {
    const __half hh = __float2half_rn(x);
    h = __half_as_ushort(hh);
    lw = __half_as_ushort(__float2half_rn(x - __half2float(hh)));
  } else {
    const __nv_bfloat16 hh = __float2bfloat16_rn(x);
    h = __bfloat16_as_ushort(hh);
    lw = __bfloat16_as_ushort(__float2bfloat16_rn(x - __bfloat162float(hh)));
  }
  uint16_t* ob = Out + (long long)bz * rows * (3LL * kp);
  const long long step = TRANSPOSED ? (long long)kp * rows : (long long)kp;      // distance between the three blocks
  uint16_t* o = TRANSPOSED ? ob + (long long)t * rows + r : ob + (long long)r * (3LL * kp) + t;
  o[0] = h;
  o[step] = pattern ? lw : h;
  o[2 * step] = pattern ? h : lw;
}

cudaError_t split_concat3_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int k, int kp,
                                 const float* s, int ld_s, const float* inv_rho, float c0, float c1, int pattern,
                                 __nv_bfloat16* Out, cudaStream_t st, long long* launches, const int* keff, int f16,
                                 int transposed, float mult, const float* rho) {
  const long long tot = (long long)rows * kp;
  const dim3 grid((unsigned)((tot + 255) / 256), batch);
  uint16_t* o = reinterpret_cast<uint16_t*>(Out);
  if (f16 && transposed) split_concat3_kernel<true, true><<<grid, 256, 0, st>>>(In, in_bs, ld_in, rows, k, kp, s, ld_s, inv_rho, c0, c1, mult, pattern, o, keff, rho);
  else if (f16) split_concat3_kernel<true, false><<<grid, 256, 0, st>>>(In, in_bs, ld_in, rows, k, kp, s, ld_s, inv_rho, c0, c1, mult, pattern, o, keff, rho);
  else if (transposed) split_concat3_kernel<false, true><<<grid, 256, 0, st>>>(In, in_bs, ld_in, rows, k, kp, s, ld_s, inv_rho, c0, c1, mult, pattern, o, keff, rho);
  else split_concat3_kernel<false, false><<<grid, 256, 0, st>>>(In, in_bs, ld_in, rows, k, kp, s, ld_s, inv_rho, c0, c1, mult, pattern, o, keff, rho);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// Matrices whose residual counts as zero (status bit 4: 1/rho = 0) get the padded head alone as filter input,
// X0 = scale * P[:, :keff] W[:, :keff]^T; every other matrix is left untouched (its CTAs return at once).
__global__ void __launch_bounds__(256) zero_residual_entry_kernel(const int* __restrict__ status, const float* __restrict__ P,
                                                                  const float* __restrict__ W, const int* __restrict__ keff,
                                                                  int m, int n, int k, float scale, void* __restrict__ X0,
                                                                  int dtype) {
  const int bz = blockIdx.y;
  if (!(status[bz] & 4)) return;
  const float* Pb = P + (long long)bz * m * k;
  const float* Wb = W + (long long)bz * n * k;
  const int ke = keff ? min(keff[bz], k) : k;
  const long long tot = (long long)m * n;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < tot; e += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(e / n), j = (int)(e % n);
    float t = 0.f;
    for (int q = 0; q < ke; ++q) t = fmaf(Pb[(long long)i * k + q], Wb[(long long)j * k + q], t);
    st_from_float(X0, (long long)bz * tot + e, dtype, scale * t);
  }
}

cudaError_t zero_residual_entry_launch(const int* status, const float* P, const float* W, const int* keff, int batch, int m,
                                       int n, int k, float scale, void* X0, int dtype, cudaStream_t st, long long* launches) {
  zero_residual_entry_kernel<<<dim3(64, batch), 256, 0, st>>>(status, P, W, keff, m, n, k, scale, X0, dtype);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// The deflation gate of Algorithms 1 and 2 on the estimated magnitudes s[b, 0..] (descending in magnitude):
//   tau <= 0: keff = window (deflate exactly the requested number);
//   tau > 0 : if |s_window| < tau |s_1| then keff = #{i < kmax : |s_i| > tau |s_1|}, else keff = 0.
__global__ void gate_kernel(const float* __restrict__ s, int ld_s, int batch, int window, int kmax, float tau,
                            int* __restrict__ keff) {
  const int bz = blockIdx.x * blockDim.x + threadIdx.x;
  if (bz >= batch) return;
  const float* sb = s + (long long)bz * ld_s;
  int k = window;
  if (tau > 0.f && window > 0) {
    const float s1 = fabsf(sb[0]);
    k = 0;
    if (fabsf(sb[window - 1]) < tau * s1)
      for (int i = 0; i < kmax; ++i) if (fabsf(sb[i]) > tau * s1) k = i + 1;
  }
  keff[bz] = k;
}

cudaError_t gate_launch(const float* s, int ld_s, int batch, int window, int kmax, float tau, int* keff, cudaStream_t st,
                        long long* launches) {
  gate_kernel<<<(batch + 127) / 128, 128, 0, st>>>(s, ld_s, batch, window, kmax, tau, keff);
  if (launches) ++*launches;
  return cudaGetLastError();
}

}  // namespace defl

// ---------------------------------------------------------------------------------------------
// Fused panel pass for CholeskyQR2 and the triplet products: for panel In[b, rows, l]
//   Out = In * Mtx[:, :kout]   (Mtx null: Out = In), written as fp32 and/or as bf16 hi + lo,
//   and/or the Gram partials of Out (fp32 products over 128-row tiles, tiles added in fp64).
// One CTA walks its share of the rows in 128-row tiles; register-blocked 4 x 8 outputs per thread.
// In-place (Out == In) is safe: a tile is read completely before it is written.
// ---------------------------------------------------------------------------------------------
namespace defl {

constexpr int FUSED_TILE = 128;
constexpr int FUSED_TS = MAX_L + 4;

// Rows are split over CTAs in whole 128-row tiles. The split is chosen so that all CTAs of the launch are resident
// at once (two per SM with this kernel's registers): a fixed 512-row split gave 624 CTAs for 592 places on
// the 48 x 6400-row panels, i.e. a second wave for 32 CTAs, and left two thirds of the GPU idle on 1600-row panels.
// At least two tiles per CTA, so the count never exceeds gram_num_chunks(rows), which sizes the partials buffer.
int fused_num_chunks(int rows, int batch) {
  static int sms = 0;
  if (sms <= 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      sms = 148;
  }
  const int places = sms * 2;
  const int tiles = (rows + FUSED_TILE - 1) / FUSED_TILE;
  int t = 2;
  while (t < tiles && (long long)((tiles + t - 1) / t) * batch > places) ++t;
  return (tiles + t - 1) / t;
}

__global__ void __launch_bounds__(256, 2) panel_fused_kernel(const float* In, long long in_bs, int ld_in, int rows, int l,
                                                          const float* __restrict__ Mtx, int ldm, int kout,
                                                          float* Out, long long out_bs, int ld_out,
                                                          __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                          int lp, double* __restrict__ partial, int nchunk) {
  extern __shared__ __align__(16) float fsm[];
  // row stride 68 floats: rows stay 16-byte aligned, so register blocks are fetched with 128-bit loads
  float (*tile)[FUSED_TS] = reinterpret_cast<float (*)[FUSED_TS]>(fsm);                          // [128][68]
  float (*ms)[FUSED_TS] = reinterpret_cast<float (*)[FUSED_TS]>(fsm + FUSED_TILE * FUSED_TS);    // [64][68]
  const int chunk = blockIdx.x, bz = blockIdx.y, tid = threadIdx.x;
  const float* Ib = In + (long long)bz * in_bs;
  const int wout = Mtx ? kout : l;      // width of Out
  if (Mtx) {
    const float* Mb = Mtx + (long long)bz * l * ldm;
    for (int e = tid; e < MAX_L * MAX_L; e += 256) {
      const int r = e / MAX_L, cc = e % MAX_L;
      ms[r][cc] = (r < l && cc < kout) ? Mb[r * ldm + cc] : 0.f;
    }
  }
  // product: thread (ty, tx) computes rows ty, ty + 32, ty + 64, ty + 96 and columns 4 tx .. 4 tx + 3, 32 + 4 tx .. + 3.
  // A warp's four ty values are then four consecutive tile rows (68 floats apart: different banks) and its eight
  // tx values read 128 contiguous bytes of the staged matrix: one shared-memory wavefront per 16-byte load. (With
  // rows 4 ty + i and columns 8 tx + j the same loads took two wavefronts each, and the product was bound by them.)
  const int ty = tid >> 3, tx = tid & 7;
  // Gram: the upper block triangle of W = In^T In (or Out^T Out) in blocks of 4 rows x 8 columns; the threads form
  // `ngrp` groups of `nblk` (one block each), group g takes the rows g, g + ngrp, ... of every tile. fp32 sums
  // per thread (at most rows-per-CTA / ngrp terms), added up over the groups in fp64 at the end, in a fixed order.
  const int nb4 = (wout + 3) >> 2, nb8 = (wout + 7) >> 3;
  int nblk = 0;
  for (int j = 0; j < nb8; ++j) nblk += min(nb4, 2 * j + 2);
  const int ngrp = min(16, 256 / nblk);
  const int grp = tid / nblk;
  const bool gram_on = partial != nullptr && grp < ngrp;
  int bi = 0, bj = 0;          // this thread's block: rows 4 bi.., columns 8 bj.. of W
  {
    int rem = tid - grp * nblk;
    while (bj < nb8 - 1 && rem >= min(nb4, 2 * bj + 2)) { rem -= min(nb4, 2 * bj + 2); ++bj; }
    bi = rem;
  }
  float g8[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) g8[i][j] = 0.f;
  const int tiles = (rows + FUSED_TILE - 1) / FUSED_TILE;
  const int chunk_rows = ((tiles + nchunk - 1) / nchunk) * FUSED_TILE;
  const int r_begin = chunk * chunk_rows, r_end = min(rows, r_begin + chunk_rows);
  for (int r0 = r_begin; r0 < r_end; r0 += FUSED_TILE) {
    __syncthreads();
    if ((ld_in & 3) == 0 && (l & 3) == 0 && ((reinterpret_cast<uintptr_t>(Ib) & 15) == 0)) {
      // 16 threads per row (one float4 each, up to 64 columns), 16 rows per pass: no index division, and all
      // eight loads of a thread are issued before the first use
      const int c4 = tid & 15, rr0 = tid >> 4;
      const bool col_ok = c4 * 4 < l;
      float4 buf[FUSED_TILE / 16];
#pragma unroll
      for (int it = 0; it < FUSED_TILE / 16; ++it) {
        const int rr = rr0 + it * 16;
        buf[it] = (col_ok && r0 + rr < r_end) ? *reinterpret_cast<const float4*>(Ib + (long long)(r0 + rr) * ld_in + c4 * 4)
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
      }
      if (col_ok) {
#pragma unroll
        for (int it = 0; it < FUSED_TILE / 16; ++it) *reinterpret_cast<float4*>(&tile[rr0 + it * 16][c4 * 4]) = buf[it];
      }
    } else {
      const int lr = (l + 3) & ~3;      // columns l..lr-1 are zeroed: the product walks the row in blocks of four
      for (int e = tid; e < FUSED_TILE * lr; e += 256) {
        const int rr = e / lr, c = e % lr;
        tile[rr][c] = (c < l && r0 + rr < r_end) ? Ib[(long long)(r0 + rr) * ld_in + c] : 0.f;
      }
    }
    __syncthreads();
    if (Mtx) {
      float acc[4][8];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
      // Mtx rows beyond l and columns beyond kout were zeroed when it was staged, so blocks of four are safe
      for (int q = 0; q < l; q += 4) {
        float4 a4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a4[i] = *reinterpret_cast<const float4*>(&tile[ty + 32 * i][q]);
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
          const float4 b0 = *reinterpret_cast<const float4*>(&ms[q + qq][tx * 4]);
          const float4 b1 = *reinterpret_cast<const float4*>(&ms[q + qq][32 + tx * 4]);
          const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float av = (qq == 0) ? a4[i].x : (qq == 1) ? a4[i].y : (qq == 2) ? a4[i].z : a4[i].w;
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av, b[j], acc[i][j]);
          }
        }
      }
      __syncthreads();
      // (columns wout.. of the tile receive zeros: the staged matrix has zero columns there)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        *reinterpret_cast<float4*>(&tile[ty + 32 * i][tx * 4]) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        *reinterpret_cast<float4*>(&tile[ty + 32 * i][32 + tx * 4]) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
      }
      __syncthreads();
    }
    if (Out) {
      float* Ob = Out + (long long)bz * out_bs;
      if ((wout & 3) == 0 && (ld_out & 3) == 0 && ((reinterpret_cast<uintptr_t>(Ob) & 15) == 0)) {
        const int c4 = tid & 15, rr0 = tid >> 4;
        if (c4 * 4 < wout) {
#pragma unroll
          for (int it = 0; it < FUSED_TILE / 16; ++it) {
            const int rr = rr0 + it * 16;
            if (r0 + rr < r_end)
              *reinterpret_cast<float4*>(Ob + (long long)(r0 + rr) * ld_out + c4 * 4) = *reinterpret_cast<const float4*>(&tile[rr][c4 * 4]);
          }
        }
      } else {
        for (int e = tid; e < FUSED_TILE * wout; e += 256) {
          const int rr = e / wout, c = e % wout;
          if (r0 + rr < r_end) Ob[(long long)(r0 + rr) * ld_out + c] = tile[rr][c];
        }
      }
    }
    if (hi) {
      if ((lp & 3) == 0 && lp <= 64 && ((reinterpret_cast<uintptr_t>(hi) | reinterpret_cast<uintptr_t>(lo)) & 7) == 0) {
        // four values per thread: 8-byte stores of the hi and lo halves (tile columns wout..lp-1 may hold
        // leftovers of the input, so they are masked here)
        const int c4 = tid & 15, rr0 = tid >> 4;
        if (c4 * 4 < lp) {
#pragma unroll
          for (int it = 0; it < FUSED_TILE / 16; ++it) {
            const int rr = rr0 + it * 16;
            if (r0 + rr >= r_end) continue;
            const float4 x4 = *reinterpret_cast<const float4*>(&tile[rr][c4 * 4]);
            float x[4] = {x4.x, x4.y, x4.z, x4.w};
            __nv_bfloat16 h[4], lw[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (c4 * 4 + j >= wout) x[j] = 0.f;
              h[j] = __float2bfloat16_rn(x[j]);
              lw[j] = __float2bfloat16_rn(x[j] - __bfloat162float(h[j]));
            }
            const long long o = ((long long)bz * rows + r0 + rr) * lp + c4 * 4;
            uint2 hv, lv;
            hv.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
            hv.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
            lv.x = (uint32_t)__bfloat16_as_ushort(lw[0]) | ((uint32_t)__bfloat16_as_ushort(lw[1]) << 16);
            lv.y = (uint32_t)__bfloat16_as_ushort(lw[2]) | ((uint32_t)__bfloat16_as_ushort(lw[3]) << 16);
            *reinterpret_cast<uint2*>(hi + o) = hv;
            *reinterpret_cast<uint2*>(lo + o) = lv;
          }
        }
      } else {
        for (int e = tid; e < FUSED_TILE * lp; e += 256) {
          const int rr = e / lp, c = e % lp;
          if (r0 + rr >= r_end) continue;
          const float x = (c < wout) ? tile[rr][c] : 0.f;
          const __nv_bfloat16 h = __float2bfloat16_rn(x);
          const long long o = ((long long)bz * rows + r0 + rr) * lp + c;
          hi[o] = h;
          lo[o] = __float2bfloat16_rn(x - __bfloat162float(h));
        }
      }
    }
    if (gram_on) {
      const int nr = min(FUSED_TILE, r_end - r0);
      for (int rr = grp; rr < nr; rr += ngrp) {
        const float4 a0 = *reinterpret_cast<const float4*>(&tile[rr][bi * 4]);
        const float4 b0 = *reinterpret_cast<const float4*>(&tile[rr][bj * 8]);
        const float4 b1 = *reinterpret_cast<const float4*>(&tile[rr][bj * 8 + 4]);
        const float a[4] = {a0.x, a0.y, a0.z, a0.w};
        const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) g8[i][j] = fmaf(a[i], b[j], g8[i][j]);
      }
    }
  }
  if (partial) {
    // sum over the groups in fp64 (group order fixed: the result does not depend on timing), in the tile's memory
    // (rows padded to an odd stride: the blocks of a group lie 4 rows apart and the mirror reads walk a column, both
    // of which land on one shared-memory bank when a row is 48 doubles = 96 words)
    const int wr = wout | 1;
    double* red = reinterpret_cast<double*>(fsm);        // [wout][wr], upper blocks only
    __syncthreads();
    for (int e = tid; e < wout * wr; e += 256) red[e] = 0.0;
    __syncthreads();
    for (int g = 0; g < ngrp; ++g) {
      if (gram_on && grp == g) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int gi = bi * 4 + i, gj = bj * 8 + j;
            if (gi < wout && gj < wout) red[gi * wr + gj] += (double)g8[i][j];
          }
      }
      __syncthreads();
    }
    double* out = partial + ((long long)bz * nchunk + chunk) * wout * wout;
    for (int e = tid; e < wout * wout; e += 256) {
      const int gi = e / wout, gj = e - gi * wout;
      // blocks below the block diagonal were not computed: take the mirror image
      out[e] = ((gi >> 3) <= (gj >> 3)) ? red[gi * wr + gj] : red[gj * wr + gi];
    }
  }
}

cudaError_t panel_fused_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int l, const float* Mtx,
                               int ldm, int kout, float* Out, long long out_bs, int ld_out, __nv_bfloat16* hi,
                               __nv_bfloat16* lo, int lp, double* partial, cudaStream_t st, long long* launches) {
  const size_t smem = (size_t)(FUSED_TILE + MAX_L) * FUSED_TS * sizeof(float);
  cudaFuncSetAttribute(panel_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const int nchunk = fused_num_chunks(rows, batch);
  panel_fused_kernel<<<dim3(nchunk, batch), 256, smem, st>>>(In, in_bs, ld_in, rows, l, Mtx, ldm, kout, Out, out_bs, ld_out,
                                                            hi, lo, lp, partial, nchunk);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Momentum of a Muon step, element-wise in fp32: Mom <- mu Mom + Grad, stored in the momentum's type; when `look`
// is given it receives Grad + mu Mom' with Mom' the STORED (rounded) new momentum, i.e. the Nesterov look-ahead
// is a function of the optimizer state as it is kept in memory.
// ---------------------------------------------------------------------------------------------
template <typename T, int V>
__global__ void __launch_bounds__(256) momentum_vec_kernel(T* Mom, const T* __restrict__ Grad, T* look, long long nvec, float mu) {
  // V elements (16 bytes) per thread and trip
  struct alignas(16) Pack { T v[V]; };
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride) {
    const Pack g = reinterpret_cast<const Pack*>(Grad)[i];
    Pack m = reinterpret_cast<const Pack*>(Mom)[i];
    Pack l;
#pragma unroll
    for (int j = 0; j < V; ++j) {
      const float gf = (float)g.v[j];
      m.v[j] = (T)fmaf(mu, (float)m.v[j], gf);
      l.v[j] = (T)fmaf(mu, (float)m.v[j], gf);          // from the momentum as stored
    }
    reinterpret_cast<Pack*>(Mom)[i] = m;
    if (look) reinterpret_cast<Pack*>(look)[i] = l;
  }
}

__global__ void __launch_bounds__(256) momentum_kernel(void* Mom, const void* __restrict__ Grad, void* look, int dtype,
                                                       long long first, long long count, float mu) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = first + (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) {
    const float g = ld_as_float(Grad, i, dtype);
    st_from_float(Mom, i, dtype, fmaf(mu, ld_as_float(Mom, i, dtype), g));
    if (look) st_from_float(look, i, dtype, fmaf(mu, ld_as_float(Mom, i, dtype), g));
  }
}
cudaError_t momentum_launch(void* Mom, const void* Grad, void* look, int dtype, long long count, float mu, cudaStream_t st,
                            long long* launches) {
  if (count <= 0) return cudaSuccess;
  const bool aligned = ((reinterpret_cast<uintptr_t>(Mom) | reinterpret_cast<uintptr_t>(Grad) | reinterpret_cast<uintptr_t>(look)) & 15) == 0;
  const int per = (dtype == BF16) ? 8 : 4;
  const long long nvec = aligned ? count / per : 0;
  if (nvec > 0) {
    const int nblk = (int)min((long long)148 * 16, (nvec + 255) / 256);
    if (dtype == BF16)
      momentum_vec_kernel<__nv_bfloat16, 8><<<nblk, 256, 0, st>>>((__nv_bfloat16*)Mom, (const __nv_bfloat16*)Grad, (__nv_bfloat16*)look, nvec, mu);
    else
      momentum_vec_kernel<float, 4><<<nblk, 256, 0, st>>>((float*)Mom, (const float*)Grad, (float*)look, nvec, mu);
    if (launches) ++*launches;
  }
  if (nvec * per < count) {      // the unaligned or leftover part
    momentum_kernel<<<1, 256, 0, st>>>(Mom, Grad, look, dtype, nvec * per, count, mu);
    if (launches) ++*launches;
  }
  return cudaGetLastError();
}

}  // namespace defl
