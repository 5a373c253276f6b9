// Deflated PSD projection (Algorithm 2) of one symmetric fp32 matrix, as kernel launches on one stream:
//   block step Z~ = Z V, Rayleigh-Ritz on V^T Z~ (one-sided Jacobi core), Ritz vectors U = V E,
//   R = Z - sum_I lambda_i u_i u_i^T, Lanczos upper estimate of ||R||_2 (Appendix E.1, "Normalization scale"),
//   X0 = R/theta + (1/gamma) sum_I sign(lambda_i) u_i u_i^T, the composite odd filter g (tf32 tensor
//   cores, every product symmetric), P = (R + R g(X0))/2 + sum_{lambda_i > 0} lambda_i u_i u_i^T,
//   P <- (P + P^T)/2, V <- CholeskyQR2(Z~).
// The basis V is orthonormalised on entry, so a Gaussian start block is accepted.
#include "../../include/defl.h"
#include "common.cuh"
#include <cuda_fp16.h>
#include "panel.cuh"
#include "ctx.cuh"

#include <cstdio>
#include <cstring>

using namespace defl;

namespace defl {

// ---------------------------------------------------------------------------------------------
// y = A x for a dense row-major fp32 matrix: one warp per row, float4 loads, fixed-order reduction.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) symv_kernel(const float* __restrict__ A, const float* __restrict__ x,
                                                   float* __restrict__ y, int n, const int* __restrict__ skip) {
  if (skip && *skip) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool vec = (n & 3) == 0;
  for (int r = blockIdx.x * 8 + warp; r < n; r += gridDim.x * 8) {
    const float* row = A + (long long)r * n;
    float acc = 0.f;
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(row);
      const float4* x4 = reinterpret_cast<const float4*>(x);
      // four independent partial sums per lane, combined in a fixed order; eight 16-byte loads of the row in flight per
      // lane where the row is long enough (a warp walks its row in dependent trips, each one a trip to L2 or HBM: the
      // trip count, not the bandwidth, is what a matrix-vector product of this size takes)
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      const int n4 = n / 4;
      int i = lane;
      for (; i + 224 < n4; i += 256) {
        float4 pr[8], qr[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) pr[u] = r4[i + 32 * u];
#pragma unroll
        for (int u = 0; u < 8; ++u) qr[u] = __ldg(&x4[i + 32 * u]);
        // (the same order of additions as two trips of the four-load loop below)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 p0 = pr[4 * h], p1 = pr[4 * h + 1], p2 = pr[4 * h + 2], p3 = pr[4 * h + 3];
          const float4 q0 = qr[4 * h], q1 = qr[4 * h + 1], q2 = qr[4 * h + 2], q3 = qr[4 * h + 3];
          a0 = fmaf(p0.x, q0.x, a0); a0 = fmaf(p0.y, q0.y, a0); a0 = fmaf(p0.z, q0.z, a0); a0 = fmaf(p0.w, q0.w, a0);
          a1 = fmaf(p1.x, q1.x, a1); a1 = fmaf(p1.y, q1.y, a1); a1 = fmaf(p1.z, q1.z, a1); a1 = fmaf(p1.w, q1.w, a1);
          a2 = fmaf(p2.x, q2.x, a2); a2 = fmaf(p2.y, q2.y, a2); a2 = fmaf(p2.z, q2.z, a2); a2 = fmaf(p2.w, q2.w, a2);
          a3 = fmaf(p3.x, q3.x, a3); a3 = fmaf(p3.y, q3.y, a3); a3 = fmaf(p3.z, q3.z, a3); a3 = fmaf(p3.w, q3.w, a3);
        }
      }
      for (; i + 96 < n4; i += 128) {
        const float4 p0 = r4[i], p1 = r4[i + 32], p2 = r4[i + 64], p3 = r4[i + 96];
        const float4 q0 = __ldg(&x4[i]), q1 = __ldg(&x4[i + 32]), q2 = __ldg(&x4[i + 64]), q3 = __ldg(&x4[i + 96]);
        a0 = fmaf(p0.x, q0.x, a0); a0 = fmaf(p0.y, q0.y, a0); a0 = fmaf(p0.z, q0.z, a0); a0 = fmaf(p0.w, q0.w, a0);
        a1 = fmaf(p1.x, q1.x, a1); a1 = fmaf(p1.y, q1.y, a1); a1 = fmaf(p1.z, q1.z, a1); a1 = fmaf(p1.w, q1.w, a1);
        a2 = fmaf(p2.x, q2.x, a2); a2 = fmaf(p2.y, q2.y, a2); a2 = fmaf(p2.z, q2.z, a2); a2 = fmaf(p2.w, q2.w, a2);
        a3 = fmaf(p3.x, q3.x, a3); a3 = fmaf(p3.y, q3.y, a3); a3 = fmaf(p3.z, q3.z, a3); a3 = fmaf(p3.w, q3.w, a3);
      }
      for (; i < n4; i += 32) {
        const float4 a = r4[i], b = __ldg(&x4[i]);
        a0 = fmaf(a.x, b.x, a0); a0 = fmaf(a.y, b.y, a0); a0 = fmaf(a.z, b.z, a0); a0 = fmaf(a.w, b.w, a0);
      }
      acc = (a0 + a1) + (a2 + a3);
    } else {
      for (int i = lane; i < n; i += 32) acc = fmaf(row[i], __ldg(&x[i]), acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) y[r] = acc;
  }
}

// out[i] = sum over s of part[s * count + i], s in ascending order (fixed order: reproducible)
__global__ void __launch_bounds__(256) sum_slices_kernel(const float* __restrict__ part, int slices, long long count,
                                                         float* __restrict__ out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float t = 0.f;
  for (int s2 = 0; s2 < slices; ++s2) t += part[(long long)s2 * count + i];
  out[i] = t;
}
static cudaError_t sum_slices_launch(const float* part, int slices, long long count, float* out, cudaStream_t st,
                                     long long* launches) {
  sum_slices_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(part, slices, count, out);
  if (launches) ++*launches;
  return cudaGetLastError();
}

static cudaError_t symv_launch(const float* A, const float* x, float* y, int n, const int* skip, cudaStream_t st,
                               long long* launches) {
  int grid = (n + 7) / 8;
  if (grid > 148 * 8) grid = 148 * 8;
  symv_kernel<<<grid, 256, 0, st>>>(A, x, y, n, skip);
  if (launches) ++*launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Lanczos on R^2 with full reorthogonalisation (Appendix E.1, "Normalization scale"). One CTA does the vector work of a step:
//   alpha_j = q_j . w;  w -= Q_j (Q_j^T w) twice;  beta_j = ||w||;  q_{j+1} = w / beta_j
// State in device memory: Q[steps, n], T[steps, steps] (dense tridiagonal, fp64), done flag.
// ---------------------------------------------------------------------------------------------
struct LanczosState {
  float* Q;        // [steps, n]
  double* T;       // [steps, steps]
  float* w;        // [n] work vector (R R q_j)
  float* t;        // [n] work vector (R q_j)
  int* done;       // set when the recurrence broke down (beta ~ 0); later steps become no-ops
  double* beta_prev;
};

__device__ double block_sum(double v, double* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  double t = 0.0;
  for (int i = 0; i < nw; ++i) t += red[i];
  return t;
}

__global__ void __launch_bounds__(1024) lanczos_init_kernel(const float* __restrict__ v0, int n, int steps, LanczosState s) {
  __shared__ double red[32];
  double a = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) a += (double)v0[i] * (double)v0[i];
  const double nv = sqrt(block_sum(a, red));
  for (int i = threadIdx.x; i < n; i += blockDim.x) s.Q[i] = (nv > 0.0) ? (float)((double)v0[i] / nv) : 0.f;
  for (int i = threadIdx.x; i < steps * steps; i += blockDim.x) s.T[i] = 0.0;
  if (threadIdx.x == 0) { *s.done = (nv > 0.0) ? 0 : 1; *s.beta_prev = 0.0; }
}

__global__ void __launch_bounds__(1024) lanczos_step_kernel(int j, int n, int steps, LanczosState s) {
  __shared__ double red[32];
  __shared__ double coef[DEFL_LANCZOS_STEPS];
  if (*s.done) return;
  const float* q = s.Q + (long long)j * n;
  double a = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) a += (double)q[i] * (double)s.w[i];
  a = block_sum(a, red);
  if (threadIdx.x == 0) s.T[j * steps + j] = a;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int pass = 0; pass < 2; ++pass) {
    // c = Q_j^T w, one warp per basis vector, then w -= Q_j c
    for (int p = warp; p <= j; p += nw) {
      const float* qp = s.Q + (long long)p * n;
      double d = 0.0;
      for (int i = lane; i < n; i += 32) d += (double)qp[i] * (double)s.w[i];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      if (lane == 0) coef[p] = d;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      double wi = (double)s.w[i];
      for (int p = 0; p <= j; ++p) wi -= coef[p] * (double)s.Q[(long long)p * n + i];
      s.w[i] = (float)wi;
    }
    __syncthreads();
  }
  double b = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) b += (double)s.w[i] * (double)s.w[i];
  b = sqrt(block_sum(b, red));
  if (j + 1 == steps) return;
  const double a0 = s.T[0];
  if (!(b > 1e-12 * fabs(a0))) {
    __syncthreads();
    if (threadIdx.x == 0) *s.done = 1;
    return;
  }
  if (threadIdx.x == 0) { s.T[j * steps + j + 1] = b; s.T[(j + 1) * steps + j] = b; }
  float* qn = s.Q + (long long)(j + 1) * n;
  for (int i = threadIdx.x; i < n; i += blockDim.x) qn[i] = (float)((double)s.w[i] / b);
}

// The same step with the work vector in registers (n <= 1024 * EPT): all j + 1 projections of a pass are reduced
// together (warp shuffles, then one pass over the per-warp partial sums in warp order), two block barriers per pass
// instead of a dependent chain of loops over global memory. alpha_j is the j-th projection of the first pass.
// The vectors and the per-warp sums are fp32 (the vectors are stored in fp32 anyway); fp64 is kept for adding up
// the 32 per-warp sums, the tridiagonal entries and the norm. With fp64 products and shuffles throughout, one CTA
// spent 22 us per step on fp64 instruction issue alone.
template <int EPT>
__global__ void __launch_bounds__(1024) lanczos_step_reg_kernel(int j, int n, int steps, LanczosState s) {
  __shared__ double part[32][DEFL_LANCZOS_STEPS];
  __shared__ double coef[DEFL_LANCZOS_STEPS];
  __shared__ double red[32];
  if (*s.done) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float wv[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) { const int i = tid + e * 1024; wv[e] = (i < n) ? s.w[i] : 0.f; }
  for (int pass = 0; pass < 2; ++pass) {
    for (int p = 0; p <= j; ++p) {
      const float* qp = s.Q + (long long)p * n;
      float d = 0.f;
#pragma unroll
      for (int e = 0; e < EPT; ++e) { const int i = tid + e * 1024; if (i < n) d = fmaf(qp[i], wv[e], d); }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      if (lane == 0) part[warp][p] = (double)d;
    }
    __syncthreads();
    if (tid <= j) {
      double t = 0.0;
      for (int w2 = 0; w2 < 32; ++w2) t += part[w2][tid];
      coef[tid] = t;
      if (pass == 0 && tid == j) s.T[j * steps + j] = t;
    }
    __syncthreads();
    for (int p = 0; p <= j; ++p) {
      const float* qp = s.Q + (long long)p * n;
      const float cp = (float)coef[p];
#pragma unroll
      for (int e = 0; e < EPT; ++e) { const int i = tid + e * 1024; if (i < n) wv[e] = fmaf(-cp, qp[i], wv[e]); }
    }
  }
  float bf = 0.f;
#pragma unroll
  for (int e = 0; e < EPT; ++e) bf = fmaf(wv[e], wv[e], bf);
  const double b = sqrt(block_sum((double)bf, red));
#pragma unroll
  for (int e = 0; e < EPT; ++e) { const int i = tid + e * 1024; if (i < n) s.w[i] = wv[e]; }
  if (j + 1 == steps) return;
  const double a0 = s.T[0];
  if (!(b > 1e-12 * fabs(a0))) {
    __syncthreads();
    if (tid == 0) *s.done = 1;
    return;
  }
  if (tid == 0) { s.T[j * steps + j + 1] = b; s.T[(j + 1) * steps + j] = b; }
  float* qn = s.Q + (long long)(j + 1) * n;
  const float inv_b = (float)(1.0 / b);
#pragma unroll
  for (int e = 0; e < EPT; ++e) { const int i = tid + e * 1024; if (i < n) qn[i] = wv[e] * inv_b; }
}

// ---------------------------------------------------------------------------------------------
// Largest eigenpair of the Lanczos matrix (symmetric tridiagonal, dense fp64 storage [steps, steps], rows after a
// breakdown all zero), by one warp: the eigenvalue by multi-section on the Sturm count (32 shifts per round, one
// per lane), the eigenvector by inverse iteration (elimination with row exchanges, pivots floored at eps ||T||).
// Only the leading unreduced block takes part: the Krylov space ends where an off-diagonal entry is zero, and the
// entries of the vector beyond it are exact zeros. Outputs rho[0] and column 0 of E (fp32, [steps, steps] row-major).
// A general symmetric eigensolver on this 20 x 20 matrix cost a fifth of the whole scale estimate.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) tridiag_top_kernel(const double* __restrict__ T, int steps, float* __restrict__ rho,
                                                         float* __restrict__ E) {
  constexpr int MS = DEFL_LANCZOS_STEPS;
  __shared__ double al[MS], be[MS], y[MS];
  const int lane = threadIdx.x;
  if (lane < steps) {
    al[lane] = T[lane * steps + lane];
    be[lane] = (lane + 1 < steps) ? T[lane * steps + lane + 1] : 0.0;
    E[lane * steps] = 0.f;
  }
  __syncwarp();
  int m = 1;
  while (m < steps && be[m - 1] != 0.0) ++m;                 // size of the leading unreduced block
  // Gershgorin interval and the scale of the matrix
  double lo = al[0], hi = al[0], tn = 0.0;
  for (int i = 0; i < m; ++i) {
    const double r = (i > 0 ? fabs(be[i - 1]) : 0.0) + (i + 1 < m ? fabs(be[i]) : 0.0);
    lo = fmin(lo, al[i] - r); hi = fmax(hi, al[i] + r);
    tn = fmax(tn, fabs(al[i]) + r);
  }
  const double eps = 2.220446049250313e-16;
  const double pivmin = fmax(tn * eps * eps, 1e-300);
  double a = lo - eps * tn - pivmin, b = hi + eps * tn + pivmin;       // count(a) < m = count(b)
  for (int round = 0; round < 16; ++round) {
    const double x = a + (b - a) * ((double)(lane + 1) / 33.0);
    // number of eigenvalues of the block below x: negative terms of the Sturm recurrence
    int cnt = 0;
    double q = 1.0;
    for (int i = 0; i < m; ++i) {
      q = al[i] - x - (i > 0 ? be[i - 1] * be[i - 1] / q : 0.0);
      if (fabs(q) < pivmin) q = -pivmin;
      cnt += q < 0.0;
    }
    const unsigned full = __ballot_sync(0xffffffffu, cnt >= m);         // shifts above every eigenvalue
    const int first = full ? __ffs(full) - 1 : 32;
    const double nb = (first < 32) ? __shfl_sync(0xffffffffu, x, first) : b;
    const double na = (first > 0) ? __shfl_sync(0xffffffffu, x, first - 1) : a;
    a = na; b = nb;
    if (b - a <= 2.0 * eps * fmax(fabs(a), fabs(b)) + 2.0 * pivmin) break;
  }
  const double lam = 0.5 * (a + b);
  if (lane == 0) {
    rho[0] = (float)lam;
    if (m == 1) y[0] = 1.0;
    else {
      // inverse iteration from the vector of ones (the off-diagonal entries of a Lanczos matrix are positive, so the
      // wanted vector has entries of one sign and is not orthogonal to it)
      double d[MS], du[MS], du2[MS], dl[MS], z[MS];
      const double floor_p = eps * tn;
      for (int i = 0; i < m; ++i) z[i] = 1.0;
      for (int iter = 0; iter < 3; ++iter) {
        for (int i = 0; i < m; ++i) { d[i] = al[i] - lam; du[i] = (i + 1 < m) ? be[i] : 0.0; dl[i] = du[i]; du2[i] = 0.0; }
        for (int i = 0; i + 1 < m; ++i) {
          if (fabs(d[i]) >= fabs(dl[i])) {
            if (fabs(d[i]) < floor_p) d[i] = (d[i] < 0.0) ? -floor_p : floor_p;
            const double f = dl[i] / d[i];
            d[i + 1] -= f * du[i];
            z[i + 1] -= f * z[i];
          } else {
            // rows i and i + 1 change places
            const double f = d[i] / dl[i];
            d[i] = dl[i];
            const double t = d[i + 1];
            d[i + 1] = du[i] - f * t;
            du[i] = t;
            if (i + 2 < m) { du2[i] = du[i + 1]; du[i + 1] = -f * du2[i]; }
            const double zt = z[i];
            z[i] = z[i + 1];
            z[i + 1] = zt - f * z[i + 1];
          }
        }
        if (fabs(d[m - 1]) < floor_p) d[m - 1] = (d[m - 1] < 0.0) ? -floor_p : floor_p;
        z[m - 1] /= d[m - 1];
        z[m - 2] = (z[m - 2] - du[m - 2] * z[m - 1]) / d[m - 2];
        for (int i = m - 3; i >= 0; --i) z[i] = (z[i] - du[i] * z[i + 1] - du2[i] * z[i + 2]) / d[i];
        double big = 0.0;
        for (int i = 0; i < m; ++i) big = fmax(big, fabs(z[i]));
        double nn = 0.0;
        for (int i = 0; i < m; ++i) { z[i] = (big > 0.0) ? z[i] / big : ((i == 0) ? 1.0 : 0.0); nn += z[i] * z[i]; }
        const double inv = rsqrt(nn);
        for (int i = 0; i < m; ++i) z[i] *= inv;
      }
      for (int i = 0; i < m; ++i) y[i] = z[i];
    }
  }
  __syncwarp();
  if (lane < m) E[lane * steps] = (float)y[lane];
}

// v = sum_p E[p][0] q_p (the Ritz vector of the largest Ritz value); E is [steps, steps] row-major fp32; rows of Q that
// carry a zero coefficient (those after a breakdown, never written) are not read
__global__ void lanczos_ritz_kernel(int n, int steps, const float* __restrict__ Q, const float* __restrict__ E,
                                    float* __restrict__ v) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  double a = 0.0;
  for (int p = 0; p < steps; ++p) {
    const float e = E[p * steps];
    if (e != 0.f) a += (double)e * (double)Q[(long long)p * n + i];
  }
  v[i] = (float)a;
}

// theta = sqrt(max(rho, 0) + ||w - rho v||), inv_theta = 1/theta (0 + status bit when theta is not a positive number)
__global__ void __launch_bounds__(1024) lanczos_theta_kernel(int n, const float* __restrict__ rho_p,
                                                             const float* __restrict__ v, const float* __restrict__ w,
                                                             float* theta, float* inv_theta, int* status) {
  __shared__ double red[32];
  const double rho = (double)rho_p[0];
  double a = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const double d = (double)w[i] - rho * (double)v[i];
    a += d * d;
  }
  a = sqrt(block_sum(a, red));
  if (threadIdx.x == 0) {
    const double th = sqrt((rho > 0.0 ? rho : 0.0) + a);
    const bool ok = th > 0.0 && isfinite(th);
    theta[0] = (float)th;
    inv_theta[0] = ok ? (float)(1.0 / th) : 0.f;
    if (!ok && status) atomicOr(status, 4);
  }
}

// P <- (P + P^T)/2 in place, 32 x 32 tiles through shared memory; tile pair (bi <= bj) per CTA
__global__ void __launch_bounds__(256) symmetrise_kernel(float* __restrict__ P, int n) {
  __shared__ float ta[32][33], tb[32][33];
  const int bi = blockIdx.y, bj = blockIdx.x;
  if (bj < bi) return;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int i = bi * 32 + r, j = bj * 32 + tx;
    ta[r][tx] = (i < n && j < n) ? P[(long long)i * n + j] : 0.f;
    const int i2 = bj * 32 + r, j2 = bi * 32 + tx;
    tb[r][tx] = (i2 < n && j2 < n) ? P[(long long)i2 * n + j2] : 0.f;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int i = bi * 32 + r, j = bj * 32 + tx;
    if (i < n && j < n) P[(long long)i * n + j] = 0.5f * (ta[r][tx] + tb[tx][r]);
    const int i2 = bj * 32 + r, j2 = bi * 32 + tx;
    if (bi != bj && i2 < n && j2 < n) P[(long long)i2 * n + j2] = 0.5f * (tb[r][tx] + ta[tx][r]);
  }
}

// hi = tf32(x) (round to nearest), lo = tf32(x - hi)
__global__ void split_tf32_kernel(const float* __restrict__ X, float* __restrict__ hi, float* __restrict__ lo, long long count) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
    const float x = X[i];
    const float h = round_to_tf32(x);
    hi[i] = h;
    lo[i] = round_to_tf32(x - h);
  }
}

// out[t] = f(lam[t]) per column scale helpers: mode 0: lambda, 1: sign(lambda)/gamma, 2: max(lambda, 0), 4: 1/gamma,
// 3: lambda^(-1/p) - root_scale z_pad (the head of an inverse root minus what the iteration left on the padded
// direction; a value that is not positive gives 0 and the non-finite status bit); negated if neg
__global__ void ritz_scale_kernel(const float* __restrict__ lam, int k, int mode, float gamma, int neg, float* __restrict__ out,
                                  const int* __restrict__ keff, const float* __restrict__ root_scale, float z_pad, int p,
                                  int* __restrict__ status) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= k) return;
  if (t >= keff[0]) { out[t] = 0.f; return; }     // not in the deflated set (gate)
  const float l = lam[t];
  float v = l;
  if (mode == 1) v = (l > 0.f ? 1.f : (l < 0.f ? -1.f : 0.f)) / gamma;
  else if (mode == 2) v = l > 0.f ? l : 0.f;
  else if (mode == 4) v = 1.f / gamma;
  else if (mode == 3) {
    if (l > 0.f && isfinite(l)) v = (float)(pow((double)l, -1.0 / (double)p) - (double)root_scale[0] * (double)z_pad);
    else { v = 0.f; if (status) atomicOr(status, DEFL_ST_NONFINITE); }
  }
  out[t] = neg ? -v : v;
}

// root_scale = theta^(-1/p) (0 when theta is not a positive number: the status bit is already set by the estimate)
__global__ void root_scale_kernel(const float* __restrict__ theta, int p, float* __restrict__ out) {
  const double th = (double)theta[0];
  out[0] = (th > 0.0 && isfinite(th)) ? (float)pow(th, -1.0 / (double)p) : 0.f;
}

// T = a I + b M for n x n fp32 matrices (the step matrix of the coupled Newton iteration), optionally rounded to tf32
__global__ void __launch_bounds__(256) affine_identity_kernel(const float* __restrict__ M, float a, float b,
                                                              float* __restrict__ T, int n, int round_tf32) {
  const long long total = (long long)n * n;
  const long long stride = (long long)gridDim.x * blockDim.x;
  if ((n & 3) == 0) {
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total / 4; q += stride) {
      const float4 m4 = reinterpret_cast<const float4*>(M)[q];
      const long long e = q * 4;
      const int i = (int)(e / n), j = (int)(e - (long long)i * n);
      float v[4] = {b * m4.x, b * m4.y, b * m4.z, b * m4.w};
      if (i >= j && i < j + 4) v[i - j] += a;
      if (round_tf32) {
#pragma unroll
        for (int t = 0; t < 4; ++t) v[t] = round_to_tf32(v[t]);
      }
      reinterpret_cast<float4*>(T)[q] = make_float4(v[0], v[1], v[2], v[3]);
    }
  } else {
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
      const int i = (int)(e / n), j = (int)(e - (long long)i * n);
      float v = b * M[e] + ((i == j) ? a : 0.f);
      T[e] = round_tf32 ? round_to_tf32(v) : v;
    }
  }
}

struct PsdWs {
  float* R; float* Xa; float* Xb; float* W; float* Tt;   // [n,n]
  float* Zt;        // [n,K]  Z V
  float* Vo;        // [n,K]  orthonormalised incoming basis
  float* U;         // [n,K]  Ritz vectors (leading k used)
  float* Us;        // [n,K]  scaled copy
  double* gram;     // [nchunk, K, K]
  float* Rinv; float* E; float* Es; float* lam; float* coef;   // [K,K] x3, [K], [K]
  float* Q; double* T; float* lw; float* lt; float* lv; float* lE; float* lrho;   // Lanczos state
  int* done; double* beta_prev;
  double* npart; float* theta; float* inv_theta; float* dummy; float* rscale;
  int* status;
  int* keff;        // [1] size of the deflated set (gate)
  float* start;     // [n] generated Lanczos start vector
  size_t bytes;
};

struct Carver2 {
  char* base; size_t off;
  explicit Carver2(void* p) : base(reinterpret_cast<char*>(p)), off(0) {}
  template <typename T> T* take(size_t count) {
    T* r = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off = align_up(off + count * sizeof(T), 256);
    return r;
  }
};

static PsdWs carve_psd(void* base, int n, int K) {
  Carver2 cv(base);
  PsdWs w;
  const size_t nn = (size_t)n * n;
  const int Ke = K > 0 ? K : 1;
  const int S = DEFL_LANCZOS_STEPS;
  w.R = cv.take<float>(nn); w.Xa = cv.take<float>(nn); w.Xb = cv.take<float>(nn);
  w.W = cv.take<float>(nn); w.Tt = cv.take<float>(nn);
  w.Zt = cv.take<float>((size_t)n * Ke); w.Vo = cv.take<float>((size_t)n * Ke);
  w.U = cv.take<float>((size_t)n * Ke); w.Us = cv.take<float>((size_t)n * Ke);
  w.gram = cv.take<double>((size_t)gram_num_chunks(n) * Ke * Ke);
  w.Rinv = cv.take<float>((size_t)Ke * Ke); w.E = cv.take<float>((size_t)Ke * Ke); w.Es = cv.take<float>((size_t)Ke * Ke);
  w.lam = cv.take<float>(Ke); w.coef = cv.take<float>(Ke);
  w.Q = cv.take<float>((size_t)S * n); w.T = cv.take<double>(S * S);
  w.lw = cv.take<float>(n); w.lt = cv.take<float>(n); w.lv = cv.take<float>(n);
  w.lE = cv.take<float>(S * S); w.lrho = cv.take<float>(S);
  w.done = cv.take<int>(1); w.beta_prev = cv.take<double>(1);
  w.npart = cv.take<double>(1184);
  w.theta = cv.take<float>(1); w.inv_theta = cv.take<float>(1); w.dummy = cv.take<float>(S * S); w.rscale = cv.take<float>(1);
  w.status = cv.take<int>(1);
  w.keff = cv.take<int>(1);
  w.start = cv.take<float>(n);
  w.bytes = cv.off;
  return w;
}

// Scale estimate of the symmetric matrix A (n x n): theta, inv_theta in device memory.
static int estimate_scale(defl_ctx* c, const float* A, int n, int norm_mode, const float* start, const PsdWs& w) {
  if (norm_mode == DEFL_NORM_FROBENIUS) {
    const int nblk = 296;
    if (ctx_fail(c, frob_partial_launch(A, F32, 1, (long long)n * n, nblk, w.npart, c->stream, &c->launches), "frobenius"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, rho_finalize_launch(w.npart, nblk, 1, w.theta, w.inv_theta, nullptr, w.status, c->stream, &c->launches), "theta"))
      return DEFL_ERR_CUDA;
    return DEFL_OK;
  }
  int steps = DEFL_LANCZOS_STEPS;
  if (steps > n) steps = n;
  LanczosState s;
  s.Q = w.Q; s.T = w.T; s.w = w.lw; s.t = w.lt; s.done = w.done; s.beta_prev = w.beta_prev;
  lanczos_init_kernel<<<1, 1024, 0, c->stream>>>(start, n, steps, s);
  ++c->launches;
  if (ctx_fail(c, cudaGetLastError(), "lanczos init")) return DEFL_ERR_CUDA;
  for (int j = 0; j < steps; ++j) {
    if (ctx_fail(c, symv_launch(A, w.Q + (size_t)j * n, w.lt, n, w.done, c->stream, &c->launches), "symv")) return DEFL_ERR_CUDA;
    if (ctx_fail(c, symv_launch(A, w.lt, w.lw, n, w.done, c->stream, &c->launches), "symv")) return DEFL_ERR_CUDA;
    if (n <= 4096) lanczos_step_reg_kernel<4><<<1, 1024, 0, c->stream>>>(j, n, steps, s);
    else if (n <= 8192) lanczos_step_reg_kernel<8><<<1, 1024, 0, c->stream>>>(j, n, steps, s);
    else lanczos_step_kernel<<<1, 1024, 0, c->stream>>>(j, n, steps, s);
    ++c->launches;
    if (ctx_fail(c, cudaGetLastError(), "lanczos step")) return DEFL_ERR_CUDA;
  }
  // largest Ritz pair of the (zero-padded) tridiagonal matrix
  tridiag_top_kernel<<<1, 32, 0, c->stream>>>(w.T, steps, w.lrho, w.lE);
  ++c->launches;
  if (ctx_fail(c, cudaGetLastError(), "ritz")) return DEFL_ERR_CUDA;
  lanczos_ritz_kernel<<<(n + 255) / 256, 256, 0, c->stream>>>(n, steps, w.Q, w.lE, w.lv);
  ++c->launches;
  if (ctx_fail(c, cudaGetLastError(), "ritz vector")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, symv_launch(A, w.lv, w.lt, n, nullptr, c->stream, &c->launches), "symv")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, symv_launch(A, w.lt, w.lw, n, nullptr, c->stream, &c->launches), "symv")) return DEFL_ERR_CUDA;
  lanczos_theta_kernel<<<1, 1024, 0, c->stream>>>(n, w.lrho, w.lv, w.lw, w.theta, w.inv_theta, w.status);
  ++c->launches;
  if (ctx_fail(c, cudaGetLastError(), "theta")) return DEFL_ERR_CUDA;
  return DEFL_OK;
}

// C = aux_scale * aux + alpha * U diag(coef) U^T  (rank-k symmetric update, exact fp32 products)
static int rank_update(defl_ctx* c, const PsdWs& w, int n, int K, int k, int coef_mode, float gamma, int neg,
                       const float* aux, float aux_scale, const float* aux_scale_dev, float* C, int round_tf32 = 0,
                       float z_pad = 0.f, int root_p = 1) {
  ritz_scale_kernel<<<1, 64, 0, c->stream>>>(w.lam, k, coef_mode, gamma, neg, w.coef, w.keff, w.rscale, z_pad, root_p, w.status);
  ++c->launches;
  if (ctx_fail(c, cudaGetLastError(), "ritz scale")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, scale_cols_launch(w.U, 0, K, 1, n, k, w.coef, K, nullptr, 1.f, 0.f, w.Us, 0, K, c->stream, &c->launches), "U diag"))
    return DEFL_ERR_CUDA;
  GemmDesc g = gemm_desc_zero();
  g.batch = 1; g.M = n; g.N = n; g.K[0] = k;
  g.A[0] = w.U; g.sa_i[0] = K; g.sa_k[0] = 1; g.in_dtype = F32;
  g.B[0] = w.Us; g.sb_k[0] = 1; g.sb_j[0] = K; g.b_dtype = F32;
  g.aux = aux; g.ld_aux = n; g.aux_dtype = F32;
  g.C = C; g.ldc = n; g.out_dtype = F32;
  g.epilogue = EPI_AUX_PLUS; g.aux_scale = aux_scale; g.aux_scale_dev = aux_scale_dev; g.alpha = 1.f;
  g.round_tf32 = round_tf32;
  return run_gemm(c, g, DEFL_ENGINE_SIMT, "rank-k update");
}

// ---------------------------------------------------------------------------------------------
// Three-block ADMM for SDPs with the constraints diag(X) = b (Appendix E.1, "ADMM for Standard-Form SDP"): element-wise kernels around
// the projection. A(X) = diag(X), A*(y) = Diag(y), A A* = I.
// ---------------------------------------------------------------------------------------------
// y_i = b_i / sigma - (X_ii / sigma + S_ii - C_ii)
__global__ void admm_y_kernel(const float* __restrict__ C, const float* __restrict__ X, const float* __restrict__ S,
                              const float* __restrict__ b, float* __restrict__ y, int n, float inv_sigma) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const long long d = (long long)i * n + i;
  y[i] = b[i] * inv_sigma - (X[d] * inv_sigma + S[d] - C[d]);
}

// Z = C - Diag(y) - X / sigma
__global__ void __launch_bounds__(256) admm_z_kernel(const float* __restrict__ C, const float* __restrict__ X,
                                                     const float* __restrict__ y, float* __restrict__ Z, int n,
                                                     float inv_sigma) {
  const long long total4 = (long long)n * n / 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total4; q += stride) {
    const float4 c4 = reinterpret_cast<const float4*>(C)[q], x4 = reinterpret_cast<const float4*>(X)[q];
    const long long e = q * 4;
    const int i = (int)(e / n), j = (int)(e - (long long)i * n);
    float z[4] = {c4.x - x4.x * inv_sigma, c4.y - x4.y * inv_sigma, c4.z - x4.z * inv_sigma, c4.w - x4.w * inv_sigma};
    if (i >= j && i < j + 4) z[i - j] -= y[i];
    reinterpret_cast<float4*>(Z)[q] = make_float4(z[0], z[1], z[2], z[3]);
  }
}

// X <- X + sigma (S + Diag(y) - C), and per-CTA partial sums (fp64, fixed order) of
//   [0] ||Diag(y) + S - C||_F^2   [1] <C, X_new>   [2] sum_i (X_new_ii - b_i)^2
__global__ void __launch_bounds__(256) admm_x_kernel(const float* __restrict__ C, const float* __restrict__ S,
                                                     const float* __restrict__ y, const float* __restrict__ b,
                                                     float* __restrict__ X, int n, float sigma,
                                                     double* __restrict__ partial) {
  __shared__ double red[3][8];
  const long long total4 = (long long)n * n / 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  double dres = 0.0, obj = 0.0, pres = 0.0;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total4; q += stride) {
    const float4 c4 = reinterpret_cast<const float4*>(C)[q], s4 = reinterpret_cast<const float4*>(S)[q];
    float4 x4 = reinterpret_cast<float4*>(X)[q];
    const long long e = q * 4;
    const int i = (int)(e / n), j = (int)(e - (long long)i * n);
    float r[4] = {s4.x - c4.x, s4.y - c4.y, s4.z - c4.z, s4.w - c4.w};
    const bool has_diag = (i >= j && i < j + 4);
    if (has_diag) r[i - j] += y[i];
    float xn[4] = {x4.x + sigma * r[0], x4.y + sigma * r[1], x4.z + sigma * r[2], x4.w + sigma * r[3]};
    const float cc[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      dres += (double)r[t] * (double)r[t];
      obj += (double)cc[t] * (double)xn[t];
    }
    if (has_diag) { const double d = (double)xn[i - j] - (double)b[i]; pres += d * d; }
    reinterpret_cast<float4*>(X)[q] = make_float4(xn[0], xn[1], xn[2], xn[3]);
  }
  double v[3] = {dres, obj, pres};
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int t = 0; t < 3; ++t) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[t] += __shfl_down_sync(0xffffffffu, v[t], o);
    if (lane == 0) red[t][warp] = v[t];
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    double t = 0.0;
    for (int w2 = 0; w2 < 8; ++w2) t += red[threadIdx.x][w2];
    partial[(long long)blockIdx.x * 3 + threadIdx.x] = t;
  }
}

// the three eigenvalue-free KKT terms of the iteration (Appendix E.4, "Experimental Details"), from the partial sums and b^T y, ||b||, ||C||_F
__global__ void admm_residual_kernel(const double* __restrict__ partial, int nblk, const float* __restrict__ b,
                                     const float* __restrict__ y, int n, double norm_b, double norm_c,
                                     float* __restrict__ out3) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  double dres = 0.0, obj = 0.0, pres = 0.0, by = 0.0;
  for (int i = 0; i < nblk; ++i) { dres += partial[3 * i]; obj += partial[3 * i + 1]; pres += partial[3 * i + 2]; }
  for (int i = 0; i < n; ++i) by += (double)b[i] * (double)y[i];
  out3[0] = (float)(sqrt(pres) / (1.0 + norm_b));
  out3[1] = (float)(sqrt(dres) / (1.0 + norm_c));
  out3[2] = (float)(fabs(obj - by) / (1.0 + fabs(obj) + fabs(by)));
}

// sum of squares of a float array in one CTA (norms of b and C, once per call)
__global__ void __launch_bounds__(1024) sumsq_kernel(const float* __restrict__ x, long long count, double* out) {
  __shared__ double red[32];
  double a = 0.0;
  for (long long i = threadIdx.x; i < count; i += blockDim.x) a += (double)x[i] * (double)x[i];
  a = block_sum(a, red);
  if (threadIdx.x == 0) *out = a;
}

}  // namespace defl

extern "C" {

size_t defl_psd_workspace_bytes(int n, int K) {
  if (n <= 0 || K < 0) return 0;
  return carve_psd(nullptr, n, K).bytes;
}

// Algorithm 2 (root_p = 0), or the same deflation around the coupled Newton iteration for the inverse p-th root
// (root_p = p; T is then the number of its steps and no coefficients are read)
static int psd_core(defl_ctx* c, const void* Xv, void* Pv, int n, int k, float* warm_basis, int K,
                    const float* coeff_schedule, int T, const defl_opts* opts, const defl_info* info, int root_p) {
  if (!c || !Xv || !Pv || n <= 0 || k < 0 || K < 0 || T < 0) return DEFL_ERR_ARG;
  if (K > 0 && !warm_basis) return DEFL_ERR_ARG;
  if (root_p == 0 && T > 0 && !coeff_schedule) return DEFL_ERR_ARG;
  if (k > K || K > DEFL_MAX_L || K >= n || T > DEFL_MAX_STEPS) return DEFL_ERR_RANK;
  const float* Z = reinterpret_cast<const float*>(Xv);
  float* P = reinterpret_cast<float*>(Pv);
  {
    const char* z0 = reinterpret_cast<const char*>(Xv);
    const char* p0 = reinterpret_cast<const char*>(Pv);
    const size_t bytes = (size_t)n * n * sizeof(float);
    if (z0 < p0 + bytes && p0 < z0 + bytes) return DEFL_ERR_ARG;
  }
  const int norm_mode = opts ? opts->norm_mode : DEFL_NORM_LANCZOS;
  if (norm_mode != DEFL_NORM_LANCZOS && norm_mode != DEFL_NORM_FROBENIUS) return DEFL_ERR_ARG;
  const float gamma = (opts && opts->gamma > 0.f) ? opts->gamma : 1.1f;
  const int engine_opt = opts ? opts->engine : DEFL_ENGINE_AUTO;
  if (engine_opt < 0 || engine_opt > 2) return DEFL_ERR_ARG;
  // the filter products run on the tensor cores (tf32) unless the fp32 engine is requested
  const int engine = (engine_opt == DEFL_ENGINE_SIMT) ? DEFL_ENGINE_SIMT : DEFL_ENGINE_TENSOR;
  const int sym = (opts && opts->exploit_symmetry) ? 1 : 0;
  const bool deflate = (k > 0) && !(opts && opts->warmup);
  const float tau = opts ? opts->tau : 0.f;
  // with the gate the deflated set is {i : |lambda_i| > tau |lambda_1|} among all K Ritz values; without it, the first k
  const int kcols = (deflate && tau > 0.f) ? K : k;
  // iterates that feed tf32 products are stored already rounded to nearest tf32: the tensor core would
  // otherwise truncate them, which biases every product towards zero
  const int tf32_round = (engine == DEFL_ENGINE_TENSOR) ? 1 : 0;
  // FP16 filter (Appendix E.2, "Composite Minimax Filter": the filter is used in half precision): iterates in IEEE half, kind::f16 products
  const bool half = opts && opts->half_filter;
  if (half && (root_p != 0 || engine != DEFL_ENGINE_TENSOR || (n & 7))) return DEFL_ERR_UNSUPPORTED;

  cudaSetDevice(c->device);
  int rc = ctx_reserve(c, carve_psd(nullptr, n, K).bytes);
  if (rc) return rc;
  PsdWs w = carve_psd(c->ws, n, K);
  ctx_profile_begin(c);
  c->err[0] = 0;
  ctx_stage_mark(c);
  if (ctx_fail(c, fill_int_launch(w.status, 1, 0, c->stream, &c->launches), "status")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, cudaMemsetAsync(c->wait_status, 0, sizeof(int), c->stream), "status word")) return DEFL_ERR_CUDA;

  // ---- stage 0: block step and Rayleigh-Ritz (lines 1-2) -------------------------------------------
  if (K > 0) {
    if (ctx_fail(c, cudaMemcpyAsync(w.Vo, warm_basis, (size_t)n * K * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy V"))
      return DEFL_ERR_CUDA;
    if ((rc = orthonormalise(c, w.Vo, 1, n, K, w.gram, w.Rinv, w.status))) return rc;
    GemmDesc g = gemm_desc_zero();
    g.batch = 1; g.M = n; g.N = K; g.K[0] = n;
    g.A[0] = Z; g.sa_i[0] = n; g.sa_k[0] = 1; g.in_dtype = F32;
    g.B[0] = w.Vo; g.sb_k[0] = K; g.sb_j[0] = 1; g.b_dtype = F32;
    g.C = w.Zt; g.ldc = K; g.out_dtype = F32; g.epilogue = EPI_STORE;
    // a tall product with a narrow output has few tiles (n/64): the inner dimension is cut into `cuts` slices,
    // taken as a batch into partial products (in the n x n scratch the filter uses later) and summed in slice order
    int cuts = 1;
    while (cuts < 16 && n % (2 * cuts * 16) == 0 && (long long)(n / 64 + 1) * cuts < 4LL * c->num_sms && 2LL * cuts * K <= n) cuts *= 2;
    if (cuts > 1) {
      const int kc = n / cuts;
      g.batch = cuts; g.K[0] = kc;
      g.batch_a[0] = kc;                       // slice s of Z: columns s kc ..
      g.batch_b[0] = (long long)kc * K;        // slice s of V: rows s kc ..
      g.C = w.W; g.batch_c = (long long)n * K;
    }
    if ((rc = run_gemm(c, g, DEFL_ENGINE_SIMT, "Z V"))) return rc;
    if (cuts > 1 &&
        ctx_fail(c, sum_slices_launch(w.W, cuts, (long long)n * K, w.Zt, c->stream, &c->launches), "sum slices"))
      return DEFL_ERR_CUDA;
    // H = V^T Z~ (symmetrised inside the eigensolver), H = E diag(lambda) E^T, sorted by |lambda|
    if (ctx_fail(c, gram_partial_launch(w.Vo, 0, 1, n, K, K, w.gram, c->stream, &c->launches, w.Zt), "V^T Z V")) return DEFL_ERR_CUDA;
    if (ctx_fail(c, jacobi_eig_launch(w.gram, gram_num_chunks(n), 1, K, 1, w.lam, w.E, nullptr, w.status, c->stream, &c->launches), "ritz"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, panel_apply_launch(w.Vo, 0, K, w.E, K, 1, n, K, K, w.U, 0, K, c->stream, &c->launches), "U = V E"))
      return DEFL_ERR_CUDA;
  }
  ctx_stage_mark(c);

  // ---- stage 1: R = Z - sum_I lambda_i u_i u_i^T (line 5) -------------------------------------------
  const float* Rm = Z;
  if (deflate) {
    if (ctx_fail(c, gate_launch(w.lam, K, 1, k, K, tau, w.keff, c->stream, &c->launches), "gate")) return DEFL_ERR_CUDA;
    if ((rc = rank_update(c, w, n, K, kcols, 0, gamma, 1, Z, 1.f, nullptr, w.R))) return rc;
    Rm = w.R;
  }
  ctx_stage_mark(c);

  // ---- stage 2: scale (line 6 / line 9) --------------------------------------------------------------
  const float* start = (opts && opts->lanczos_start) ? opts->lanczos_start : w.start;
  if (norm_mode == DEFL_NORM_LANCZOS && !(opts && opts->lanczos_start)) {
    if (ctx_fail(c, fill_gaussian_launch(w.start, n, F32, opts ? opts->seed : 0ull, 0, 0ull, c->stream, &c->launches), "start vector"))
      return DEFL_ERR_CUDA;
  }
  if ((rc = estimate_scale(c, Rm, n, norm_mode, start, w))) return rc;
  ctx_stage_mark(c);

  // ---- stage 3: X0 = R/theta + (1/gamma) sum_I sign(lambda_i) u_i u_i^T (line 7) ---------------------
  float* bufs[2] = {w.Xa, w.Xb};
  int cur = 0;
  if (deflate) {
    // (an inverse root pads at +1/gamma whatever the sign: a value that is not positive is reported, not followed)
    if ((rc = rank_update(c, w, n, K, kcols, root_p ? 4 : 1, gamma, 0, Rm, 1.f, w.inv_theta, bufs[cur], tf32_round))) return rc;
  } else {
    if (ctx_fail(c, scale_launch(Rm, F32, bufs[cur], F32, 1, (long long)n * n, w.inv_theta, c->stream, &c->launches, tf32_round), "normalise"))
      return DEFL_ERR_CUDA;
  }
  ctx_stage_mark(c);

  // ---- stage 4: g = p_T o ... o p_1 on the symmetric X0: W = X^2, Tt = a I + b W + c W^2, X <- X Tt ------
  float* root_z = nullptr;       // inverse root: Z_T
  if (root_p) {
    // Coupled Newton iteration on M_0 = X0, Z_0 = I: T_t = ((p+1) I - M_t)/p, Z_{t+1} = Z_t T_t, M_{t+1} = T_t^p M_t.
    // Every iterate is a polynomial in X0, so every product is a symmetric matrix: the tiles on and above the
    // diagonal are computed and mirrored, as in the filter of the projection. Z_1 = T_0 is a copy; the last step
    // does not update M. Buffers: M and two spares among {Xa, Xb, Tt}, T_t in W, Z alternating between the residual's
    // buffer (free once X0 exists) and the output, ending in the former.
    float* M = bufs[cur];
    float* spare[2] = {bufs[cur ^ 1], w.Tt};
    float* Tm = w.W;
    const int swaps = T > 1 ? T - 1 : 0;
    float* zc = (swaps & 1) ? P : w.R;
    float* zn = (swaps & 1) ? w.R : P;
    const long long nn = (long long)n * n;
    const int ablk = (int)((nn / 4 + 255) / 256 < 1184 ? (nn / 4 + 255) / 256 + 1 : 1184);
    auto product = [&](const float* Aop, const float* Bop, float* Cout, const char* what) {
      GemmDesc g = gemm_desc_zero();
      g.batch = 1; g.in_dtype = F32; g.b_dtype = F32; g.out_dtype = F32;
      g.M = n; g.N = n; g.K[0] = n;
      g.A[0] = Aop; g.sa_i[0] = n; g.sa_k[0] = 1;
      g.B[0] = Bop; g.sb_k[0] = 1; g.sb_j[0] = n;          // symmetric: rows as columns
      g.C = Cout; g.ldc = n; g.epilogue = EPI_STORE; g.symmetric = 1; g.round_tf32 = tf32_round;
      return run_gemm(c, g, gemm_tc_supported(g) ? engine : DEFL_ENGINE_SIMT, what);
    };
    if (T == 0) {
      affine_identity_kernel<<<ablk, 256, 0, c->stream>>>(M, 1.f, 0.f, zc, n, 0);
      ++c->launches;
      if (ctx_fail(c, cudaGetLastError(), "identity")) return DEFL_ERR_CUDA;
    }
    for (int t = 0; t < T; ++t) {
      affine_identity_kernel<<<ablk, 256, 0, c->stream>>>(M, (float)(root_p + 1) / (float)root_p, -1.f / (float)root_p, Tm, n, tf32_round);
      ++c->launches;
      if (ctx_fail(c, cudaGetLastError(), "step matrix")) return DEFL_ERR_CUDA;
      if (t == 0) {
        if (ctx_fail(c, cudaMemcpyAsync(zc, Tm, (size_t)nn * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "Z_1"))
          return DEFL_ERR_CUDA;
      } else {
        if ((rc = product(zc, Tm, zn, "Z T"))) return rc;
        float* sw = zc; zc = zn; zn = sw;
      }
      if (t + 1 == T) break;
      if (root_p == 1) {
        if ((rc = product(Tm, M, spare[0], "T M"))) return rc;
        float* old = M; M = spare[0]; spare[0] = old;
      } else if (root_p == 2) {
        if ((rc = product(Tm, Tm, spare[0], "T^2"))) return rc;
        if ((rc = product(spare[0], M, spare[1], "T^2 M"))) return rc;
        float* old = M; M = spare[1]; spare[1] = old;
      } else {
        if ((rc = product(Tm, Tm, spare[0], "T^2"))) return rc;
        if ((rc = product(spare[0], spare[0], spare[1], "T^4"))) return rc;
        if ((rc = product(spare[1], M, spare[0], "T^4 M"))) return rc;
        float* old = M; M = spare[0]; spare[0] = old;
      }
    }
    root_z = zc;
  }
  if (!root_p && half && T > 0) {
    // half-precision buffers inside the fp32 scratch that is free here: the two iterates share the other iterate
    // buffer, W and Tt share the fp32 W; the result returns to fp32 (rounded to tf32) for the reconstruction
    const size_t nn = (size_t)n * n;
    __half* H[2] = {reinterpret_cast<__half*>(bufs[cur ^ 1]), reinterpret_cast<__half*>(bufs[cur ^ 1]) + nn};
    __half* HW = reinterpret_cast<__half*>(w.W);
    __half* HT = HW + nn;
    if (ctx_fail(c, scale_launch(bufs[cur], F32, H[0], F16, 1, (long long)nn, nullptr, c->stream, &c->launches, 0), "to half"))
      return DEFL_ERR_CUDA;
    int hc = 0;
    for (int t = 0; t < T; ++t) {
      const float ca = coeff_schedule[3 * t], cb = coeff_schedule[3 * t + 1], cc = coeff_schedule[3 * t + 2];
      GemmDesc g = gemm_desc_zero();
      g.batch = 1; g.in_dtype = F16; g.b_dtype = F16; g.out_dtype = F16;
      g.M = n; g.N = n; g.K[0] = n;
      g.A[0] = H[hc]; g.sa_i[0] = n; g.sa_k[0] = 1;
      g.B[0] = H[hc]; g.sb_k[0] = 1; g.sb_j[0] = n;          // X symmetric: rows as columns
      g.C = HW; g.ldc = n; g.epilogue = EPI_STORE; g.symmetric = 1;
      if ((rc = run_gemm(c, g, DEFL_ENGINE_TENSOR, "X^2 (half)"))) return rc;
      g.A[0] = HW; g.B[0] = HW; g.C = HT;
      g.aux = HW; g.ld_aux = n; g.aux_dtype = F16;
      g.epilogue = EPI_POLY; g.pa = ca; g.pb = cb; g.pc = cc;
      if ((rc = run_gemm(c, g, DEFL_ENGINE_TENSOR, "polynomial (half)"))) return rc;
      g.A[0] = H[hc]; g.B[0] = HT; g.C = H[hc ^ 1]; g.aux = nullptr;
      g.epilogue = EPI_STORE; g.symmetric = 1;              // the iterate stays exactly symmetric (see below)
      if ((rc = run_gemm(c, g, DEFL_ENGINE_TENSOR, "apply (half)"))) return rc;
      hc ^= 1;
    }
    if (ctx_fail(c, scale_launch(H[hc], F16, bufs[cur], F32, 1, (long long)nn, nullptr, c->stream, &c->launches, tf32_round), "from half"))
      return DEFL_ERR_CUDA;
  }
  for (int t = 0; t < ((half || root_p) ? 0 : T); ++t) {
    const float ca = coeff_schedule[3 * t], cb = coeff_schedule[3 * t + 1], cc = coeff_schedule[3 * t + 2];
    const float* X = bufs[cur];
    float* Xn = bufs[cur ^ 1];
    GemmDesc g = gemm_desc_zero();
    g.batch = 1; g.in_dtype = F32; g.b_dtype = F32; g.out_dtype = F32;
    g.M = n; g.N = n; g.K[0] = n;
    g.A[0] = X; g.sa_i[0] = n; g.sa_k[0] = 1;
    g.B[0] = X; g.sb_k[0] = 1; g.sb_j[0] = n;          // X symmetric: rows as columns
    g.C = w.W; g.ldc = n; g.epilogue = EPI_STORE; g.symmetric = sym; g.round_tf32 = tf32_round;
    if ((rc = run_gemm(c, g, gemm_tc_supported(g) ? engine : DEFL_ENGINE_SIMT, "X^2"))) return rc;
    g.A[0] = w.W; g.B[0] = w.W; g.C = w.Tt;
    g.aux = w.W; g.ld_aux = n; g.aux_dtype = F32;
    g.epilogue = EPI_POLY; g.pa = ca; g.pb = cb; g.pc = cc;
    if ((rc = run_gemm(c, g, gemm_tc_supported(g) ? engine : DEFL_ENGINE_SIMT, "polynomial"))) return rc;
    g.A[0] = X; g.B[0] = w.Tt; g.C = Xn; g.aux = nullptr;
    // X Tt is symmetric only up to rounding, and the iterate must be EXACTLY symmetric: the products above take
    // X^T for X (rows as columns), which is the Gram X X^T, and an antisymmetric error N that anticommutes with
    // sign(X) then comes back as 2N after every step (X' = S + 3N/2 - S N S / 2). So the upper tiles are computed
    // and mirrored, whatever exploit_symmetry says; the skew part of the rounding turns into a symmetric error of
    // the same size, which the iteration does not amplify.
    g.epilogue = EPI_STORE; g.symmetric = 1;
    if ((rc = run_gemm(c, g, gemm_tc_supported(g) ? engine : DEFL_ENGINE_SIMT, "apply"))) return rc;
    cur ^= 1;
  }
  ctx_stage_mark(c);

  // ---- stage 5 (inverse root): out = theta^(-1/p) (Z - z_pad U U^T) + U diag(lambda^(-1/p)) U^T, symmetrised ----
  if (root_p) {
    root_scale_kernel<<<1, 1, 0, c->stream>>>(w.theta, root_p, w.rscale);
    ++c->launches;
    if (ctx_fail(c, cudaGetLastError(), "root scale")) return DEFL_ERR_CUDA;
    if (deflate) {
      // what the scalar iteration makes of the padding value 1/gamma (fp64 on the host: T steps)
      double m = 1.0 / (double)gamma, z = 1.0;
      for (int t = 0; t < T; ++t) {
        const double tt = ((double)(root_p + 1) - m) / (double)root_p;
        z *= tt;
        for (int q = 0; q < root_p; ++q) m *= tt;
      }
      if ((rc = rank_update(c, w, n, K, kcols, 3, gamma, 0, root_z, 1.f, w.rscale, P, 0, (float)z, root_p))) return rc;
    } else {
      if (ctx_fail(c, scale_launch(root_z, F32, P, F32, 1, (long long)n * n, w.rscale, c->stream, &c->launches, 0), "scale"))
        return DEFL_ERR_CUDA;
    }
    symmetrise_kernel<<<dim3((n + 31) / 32, (n + 31) / 32), 256, 0, c->stream>>>(P, n);
    ++c->launches;
    if (ctx_fail(c, cudaGetLastError(), "symmetrise")) return DEFL_ERR_CUDA;
    // the iteration diverges on an eigenvalue of X0 that is not positive (an indefinite input, or a basis that has not
    // settled: a Ritz pair with residual r leaves R indefinite by about -|r|^2 / (r^T A r / |r|^2)): report it
    if (ctx_fail(c, finite_probe_launch(P, F32, 1, (long long)n * n, w.status, c->stream, &c->launches), "finite probe"))
      return DEFL_ERR_CUDA;
  }
  // ---- stage 5: P = (R + R g(X0))/2 + sum_{lambda_i > 0} lambda_i u_i u_i^T, symmetrised (lines 8, 12) ----
  if (!root_p) {
    GemmDesc g = gemm_desc_zero();
    g.batch = 1; g.in_dtype = F32; g.b_dtype = F32; g.out_dtype = F32;
    g.M = n; g.N = n; g.K[0] = n;
    g.A[0] = Rm; g.sa_i[0] = n; g.sa_k[0] = 1;
    g.B[0] = bufs[cur]; g.sb_k[0] = 1; g.sb_j[0] = n;   // g(X0) symmetric up to rounding
    if (tf32_round && gemm_tc_supported(g)) {
      // R carries the large entries of this product: feed it as two tf32 terms R = R_hi + R_lo (two K
      // segments against the same g) so that the tensor core does not truncate it
      split_tf32_kernel<<<1184, 256, 0, c->stream>>>(Rm, w.W, w.Tt, (long long)n * n);
      ++c->launches;
      if (ctx_fail(c, cudaGetLastError(), "split R")) return DEFL_ERR_CUDA;
      g.nseg = 2; g.K[1] = n;
      g.A[0] = w.W; g.A[1] = w.Tt; g.sa_i[1] = n; g.sa_k[1] = 1;
      g.B[1] = bufs[cur]; g.sb_k[1] = 1; g.sb_j[1] = n;
    }
    g.aux = Rm; g.ld_aux = n; g.aux_dtype = F32;
    g.C = P; g.ldc = n;
    g.epilogue = EPI_AUX_PLUS; g.aux_scale = 0.5f; g.alpha = 0.5f;
    if ((rc = run_gemm(c, g, gemm_tc_supported(g) ? engine : DEFL_ENGINE_SIMT, "R g(X0)"))) return rc;
    if (deflate) {
      if ((rc = rank_update(c, w, n, K, kcols, 2, gamma, 0, P, 1.f, nullptr, P))) return rc;
    }
    symmetrise_kernel<<<dim3((n + 31) / 32, (n + 31) / 32), 256, 0, c->stream>>>(P, n);
    ++c->launches;
    if (ctx_fail(c, cudaGetLastError(), "symmetrise")) return DEFL_ERR_CUDA;
  }
  ctx_stage_mark(c);

  // ---- stage 6: V <- CholeskyQR(Z~) (line 11) ----------------------------------------------------------
  if (K > 0) {
    if ((rc = orthonormalise(c, w.Zt, 1, n, K, w.gram, w.Rinv, w.status))) return rc;
    if (ctx_fail(c, cudaMemcpyAsync(warm_basis, w.Zt, (size_t)n * K * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy V"))
      return DEFL_ERR_CUDA;
  }
  ctx_stage_mark(c);

  if (info) {
    if (info->s && K > 0 &&
        ctx_fail(c, cudaMemcpyAsync(info->s, w.lam, (size_t)K * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy lambda"))
      return DEFL_ERR_CUDA;
    if (info->rho &&
        ctx_fail(c, cudaMemcpyAsync(info->rho, w.theta, sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy theta"))
      return DEFL_ERR_CUDA;
    if (info->k_used) {
      if (!deflate && ctx_fail(c, fill_int_launch(w.keff, 1, 0, c->stream, &c->launches), "k_used")) return DEFL_ERR_CUDA;
      if (ctx_fail(c, cudaMemcpyAsync(info->k_used, w.keff, sizeof(int), cudaMemcpyDeviceToDevice, c->stream), "copy k_used"))
        return DEFL_ERR_CUDA;
    }
    if (info->status) {
      if (ctx_fail(c, or_status_launch(w.status, 1, c->wait_status, c->stream, &c->launches), "status")) return DEFL_ERR_CUDA;
      if (ctx_fail(c, cudaMemcpyAsync(info->status, w.status, sizeof(int), cudaMemcpyDeviceToDevice, c->stream), "copy status"))
        return DEFL_ERR_CUDA;
    }
  }
  return DEFL_OK;
}


int defl_psd_project(defl_ctx* c, const void* Xv, void* Pv, int n, int k, float* warm_basis, int K,
                     const float* coeff_schedule, int T, const defl_opts* opts, const defl_info* info) {
  return psd_core(c, Xv, Pv, n, k, warm_basis, K, coeff_schedule, T, opts, info, 0);
}

int defl_inv_root(defl_ctx* c, const void* Av, void* outv, int n, int p, int k, float* warm_basis, int K, int steps,
                  const defl_opts* opts, const defl_info* info) {
  if (p != 1 && p != 2 && p != 4) return DEFL_ERR_ARG;
  return psd_core(c, Av, outv, n, k, warm_basis, K, nullptr, steps, opts, info, p);
}

int defl_admm_diag_sdp(defl_ctx* c, const void* Cv, const float* b, int n, float sigma, int iters, int warmup_iters,
                       void* Xv, void* Sv, float* y, int k, float* warm_basis, int K, const float* coeff_schedule,
                       int T, const defl_opts* opts, float* residuals) {
  if (!c || !Cv || !b || !Xv || !Sv || !y || n <= 0 || (n & 3) || iters < 0 || !(sigma > 0.f)) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  const float* C = reinterpret_cast<const float*>(Cv);
  float* X = reinterpret_cast<float*>(Xv);
  float* S = reinterpret_cast<float*>(Sv);
  // scratch of this loop: Z [n,n], partial sums, residual history on the device; the context keeps it with the
  // staging buffers of the host-buffer entry point (the projection uses the workspace proper)
  const int nblk = c->num_sms * 4;
  const size_t zbytes = (size_t)n * n * sizeof(float);
  const size_t extra = align_up((size_t)nblk * 3 * sizeof(double), 256) + align_up((size_t)(iters > 0 ? iters : 1) * 3 * sizeof(float), 256) + 256;
  const size_t need = zbytes > extra ? zbytes : extra;
  {
    const size_t bytes = need;
    if (bytes > c->stage_bytes) {
      cudaDeviceSynchronize();
      if (c->stage_in) cudaFree(c->stage_in);
      if (c->stage_out) cudaFree(c->stage_out);
      c->stage_in = c->stage_out = nullptr;
      c->stage_bytes = 0;
      if (ctx_fail(c, cudaMalloc(&c->stage_in, bytes), "cudaMalloc(ADMM scratch)")) return DEFL_ERR_CUDA;
      if (ctx_fail(c, cudaMalloc(&c->stage_out, bytes), "cudaMalloc(ADMM scratch)")) return DEFL_ERR_CUDA;
      c->stage_bytes = bytes;
    }
  }
  float* Z = reinterpret_cast<float*>(c->stage_in);
  char* aux = reinterpret_cast<char*>(c->stage_out);
  double* partial = reinterpret_cast<double*>(aux);
  float* hist = reinterpret_cast<float*>(aux + align_up((size_t)nblk * 3 * sizeof(double), 256));
  double* norms = reinterpret_cast<double*>(aux + align_up((size_t)nblk * 3 * sizeof(double), 256) +
                                            align_up((size_t)(iters > 0 ? iters : 1) * 3 * sizeof(float), 256));
  sumsq_kernel<<<1, 1024, 0, c->stream>>>(b, n, norms);
  sumsq_kernel<<<1, 1024, 0, c->stream>>>(C, (long long)n * n, norms + 1);
  c->launches += 2;
  double hn[2] = {0.0, 0.0};
  if (ctx_fail(c, cudaMemcpyAsync(hn, norms, sizeof(hn), cudaMemcpyDeviceToHost, c->stream), "norms") ||
      ctx_fail(c, cudaStreamSynchronize(c->stream), "synchronize"))
    return DEFL_ERR_CUDA;
  const double norm_b = sqrt(hn[0]), norm_c = sqrt(hn[1]);
  const float inv_sigma = 1.f / sigma;
  defl_opts o;
  if (opts) o = *opts; else memset(&o, 0, sizeof(o));
  for (int it = 0; it < iters; ++it) {
    admm_y_kernel<<<(n + 255) / 256, 256, 0, c->stream>>>(C, X, S, b, y, n, inv_sigma);
    admm_z_kernel<<<nblk, 256, 0, c->stream>>>(C, X, y, Z, n, inv_sigma);
    c->launches += 2;
    if (ctx_fail(c, cudaGetLastError(), "ADMM y, Z")) return DEFL_ERR_CUDA;
    o.warmup = (it < warmup_iters) ? 1 : (opts ? opts->warmup : 0);
    const int rc = defl_psd_project(c, Z, S, n, k, warm_basis, K, coeff_schedule, T, &o, nullptr);
    if (rc) return rc;
    admm_x_kernel<<<nblk, 256, 0, c->stream>>>(C, S, y, b, X, n, sigma, partial);
    admm_residual_kernel<<<1, 32, 0, c->stream>>>(partial, nblk, b, y, n, norm_b, norm_c, hist + 3 * it);
    c->launches += 2;
    if (ctx_fail(c, cudaGetLastError(), "ADMM X")) return DEFL_ERR_CUDA;
  }
  if (residuals && iters > 0) {
    if (ctx_fail(c, cudaMemcpyAsync(residuals, hist, (size_t)iters * 3 * sizeof(float), cudaMemcpyDeviceToHost, c->stream), "residuals") ||
        ctx_fail(c, cudaStreamSynchronize(c->stream), "synchronize"))
      return DEFL_ERR_CUDA;
  }
  return DEFL_OK;
}

}  // extern "C"
