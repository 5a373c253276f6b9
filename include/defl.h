/* defl.h -- C ABI of the B200 (sm_100a) spectrally deflated matrix filter.
 *
 * The library wraps an unchanged fixed-depth polynomial filter (Eq. 1) in spectral deflation
 * (Section 2): estimate the dominant singular/eigen components, subtract them, normalise the
 * residual, run the filter, restore the components (Eq. 3). Two primitives are exported:
 *   defl_polar_batched  -- Algorithm 3 (batched randomized SVD) + Algorithm 1 (deflated polar factor)
 *   defl_psd_project    -- Algorithm 2 (deflated PSD projection with a warm-started basis)
 *   defl_inv_root       -- the same deflation around a fixed-depth inverse matrix root (Conclusion)
 * plus the batched randomized SVD on its own, a counter-based Gaussian fill and diagnostics.
 *
 * Conventions
 *   - Every matrix pointer is DEVICE memory unless the comment says "host". Matrices are
 *     row-major and contiguous; a batch is b matrices back to back.
 *   - The caller owns every buffer it passes; the library never frees or keeps a caller pointer
 *     after the call returns. A context owns its own scratch memory and grows it (cudaMalloc)
 *     when a call needs more than it holds, so repeated calls of one shape allocate once.
 *   - All work is enqueued on the context's stream and the call returns without synchronising
 *     (the only exception: growing the scratch memory synchronises the device).
 *   - Return value: 0 = OK, < 0 = caller error, nothing was launched (see defl_status_string).
 *     Numerical events (Cholesky breakdown, Jacobi sweep cap, zero residual, a non-finite result, a
 *     device-side wait that ran out) are reported per matrix in defl_info.status, never by a trap.
 *   - There is no CPU fallback: without a CUDA device every compute entry point returns
 *     DEFL_ERR_CUDA.
 */
#ifndef DEFL_H_
#define DEFL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* storage types of G / out */
#define DEFL_BF16 0 /* bf16 storage of inputs and outputs, 16-bit tensor-core products, fp32 accumulation */
#define DEFL_F32 1  /* fp32 storage; polar path: fp32 FMA products; PSD filter: tf32 tensor-core products */
#define DEFL_F16 2  /* IEEE half: the FP16 filter of the PSD projection (opts->half_filter) and defl_debug_gemm only */

/* where the head is restored (polar) */
#define DEFL_RESTORE_PADDED 0 /* Algorithm 1: X0 = R/||R||_F + U_k V_k^T / gamma, out = N^L(X0) */
#define DEFL_RESTORE_ADD 1    /* Eq. 3:       X0 = R/||R||_F,                   out = N^L(X0) + U_k V_k^T */

/* normalisation scale of the symmetric residual (PSD) */
#define DEFL_NORM_LANCZOS 0   /* Appendix E.1, "Normalization scale": 20-step Lanczos upper estimate of ||R||_2 */
#define DEFL_NORM_FROBENIUS 1 /* ||R||_F, a looser valid upper bound */

/* which product engine runs the large matrix products */
#define DEFL_ENGINE_AUTO 0   /* tensor cores whenever the shape and type allow */
#define DEFL_ENGINE_SIMT 1   /* fp32 FMA tiles (reference engine inside the library) */
#define DEFL_ENGINE_TENSOR 2 /* tcgen05 tiles; error if the shape is not supported */

/* return codes */
#define DEFL_OK 0
#define DEFL_ERR_ARG (-1)       /* null pointer, non-positive size, aliasing, bad enum */
#define DEFL_ERR_RANK (-2)      /* k + oversample leaves no room: need k < min(m,n) and l <= DEFL_MAX_L */
#define DEFL_ERR_CUDA (-3)      /* a CUDA runtime call failed (no device, launch error, out of memory) */
#define DEFL_ERR_UNSUPPORTED (-4) /* the requested engine cannot run this shape/type */

/* per-matrix status bits in defl_info.status */
#define DEFL_ST_CHOL_SHIFT 1   /* a Cholesky pivot was not positive; factorised with a diagonal shift */
#define DEFL_ST_JACOBI_CAP 2   /* the Jacobi eigensolver hit its sweep cap */
#define DEFL_ST_ZERO_RESIDUAL 4 /* ||R||_F was zero, not finite, or (bf16 storage, where it is taken as
                                  sqrt(||G||_F^2 - sum s_i^2)) below 1e-3 ||G||_F: residual treated as zero */
#define DEFL_ST_DEVICE_WAIT 8  /* a bounded device-side wait ran out; the output is not valid */
#define DEFL_ST_NONFINITE 16   /* the result of this matrix holds Inf or NaN: its input did, or an iterate left the range
                                  of its storage format (scaled IEEE half iterates overflow beyond about 2e3, which a
                                  normalised input reaches only with a schedule that diverges); polar calls only */

#define DEFL_MAX_L 64 /* largest sketch width k + oversample (and PSD basis width K) */
#define DEFL_MAX_STEPS 32 /* largest filter depth L (or T) */
#define DEFL_MAX_TERMS 6  /* most coefficients per filter step (Eq. 5 with d = 5) */
#define DEFL_LANCZOS_STEPS 20

typedef struct defl_ctx defl_ctx; /* opaque: device, stream, scratch memory */

typedef struct defl_opts {
  const float* sketch;   /* device, Omega[b, min(m,n), l] fp32 (Algorithm 3 line 2); NULL: drawn from `seed`
                            with defl_fill_gaussian's generator, stream index = matrix index */
  uint64_t seed;
  int restore_mode;      /* DEFL_RESTORE_* */
  float gamma;           /* padding margin gamma >= 1 (Algorithm 1 / 2); <= 0 means 1.01 */
  int norm_mode;         /* DEFL_NORM_* (PSD only) */
  const float* lanczos_start; /* device, [n] fp32 start vector of the Lanczos run; NULL: drawn from `seed` */
  int warmup;            /* PSD: non-zero = gate off, return the undeflated projection of Eq. 7 but still
                            advance the basis (the paper keeps the gate off while the basis stabilises) */
  int engine;            /* DEFL_ENGINE_* */
  int exploit_symmetry;  /* non-zero: compute only the upper tiles of X X^T and of A^2 and mirror them */
  float tau;             /* deflation gate of Algorithms 1 and 2. <= 0 (default): deflate exactly k components.
                            > 0: with s the k estimated magnitudes, deflate only if s_k < tau * s_1, and then the
                            components with s_i > tau * s_1 (PSD: among all K Ritz values); otherwise the call
                            reduces to the undeflated filter for that matrix. Decided per matrix on the device. */
  int half_filter;       /* PSD only, non-zero: the T filter steps run in IEEE half precision (iterates stored in
                            half, tensor-core products with fp32 accumulation), the precision the paper's SDP runs
                            use for the filter (Appendix E.2, "Composite Minimax Filter"). Everything around the filter stays fp32/tf32.
                            Needs n a multiple of 8 and the tensor engine. */
  int bf16_iterates;     /* polar path with bf16 input: storage type of the filter's iterates X_t, A_t, B_t (input,
                            output and every other stage are unchanged). 0 (default): IEEE half scaled by 32 in the
                            first two filter steps (same tensor-core rate, three more mantissa bits: the rounding of
                            the early iterates is what limits accuracy) and in every step up to the last one that
                            shares its pass over X with a neighbour (see defl_polar_batched: "two steps per pass"),
                            bf16 in the later ones (less power, i.e. more clock under a power cap); with
                            DEFL_RESTORE_ADD scaled half in every step (that mode is about ten times more sensitive
                            to the storage rounding). 1: bf16 in every step (and one pass over X per step), the
                            storage the paper's training runs use; NOT within the library's 3e-2 accuracy bar on wide
                            matrices with slowly decaying spectra (1600 x 6400, sigma_i = 200/i, k = 32: 4.2e-2 relative
                            Frobenius error against an fp64 evaluation of the same algorithm; square and faster
                            decaying cases stay below 3e-2). 2: scaled half in every step. */
  int poly_terms;        /* polar calls: coefficients per filter step in coeff_schedule. 0 or 3 (default): the quintic
                            (a, b, c) of Eq. 2. 2: a cubic (a, b). 4 .. DEFL_MAX_TERMS: the degree-(2d+1) map of Eq. 5,
                            X <- a_0 X + a_1 (X X^T) X + ... + a_d (X X^T)^d X with d = poly_terms - 1 (4 = the
                            degree-seven member); the schedule is then [L][poly_terms]. The polynomial in the Gram
                            matrix is formed by Horner steps, one more short-side product per degree beyond the quintic. */
} defl_opts;

typedef struct defl_info {
  float* s;      /* device, [b, l]: all l estimated singular values, descending (PSD: [K] Ritz values by
                    decreasing magnitude); may be NULL */
  float* rho;    /* device, [b]: ||R||_F used for normalisation (PSD: [1], the scale theta-hat); may be NULL */
  int* status;   /* device, [b]: DEFL_ST_* bits (PSD: [1]); may be NULL */
  int* k_used;   /* device, [b]: number of components actually deflated (PSD: [1]); may be NULL */
} defl_info;

/* Context. `device` is a CUDA ordinal. defl_create makes no assumption about the current device
 * and restores it. Not thread safe: one context per host thread or external locking.
 * Environment overrides are read here, once, and never on the call path: DEFL_TC_BN, DEFL_TC_TILE_M, DEFL_TC_STAGES,
 * DEFL_TC_KSUB, DEFL_TC_PAIR, DEFL_TC_PAIR_MIN_N, DEFL_TC_DYNAMIC, DEFL_TC_AUX_PREFETCH, DEFL_TC_DEBUG (tile forms of
 * the tensor engine, for experiments and tests), DEFL_TC_WAIT_MS (limit of the device-side waits, default 2000),
 * DEFL_NO_TRANSPOSED_APPLY, DEFL_NO_PAIRED_STEPS (one pass over X per filter step everywhere), DEFL_HOST_CHUNKS,
 * DEFL_JACOBI_SWEEPS (sweep cap of the Jacobi core, default 40). */
int defl_create(defl_ctx** out, int device);
int defl_destroy(defl_ctx* ctx);
int defl_set_stream(defl_ctx* ctx, void* cuda_stream); /* cudaStream_t; NULL = default stream */

/* Bytes of context scratch a polar / PSD call of this shape needs (what the context will hold; a polar call with
 * opts->poly_terms > 3 takes one more buffer of b * min(m,n)^2 elements). */
size_t defl_polar_workspace_bytes(int b, int m, int n, int dtype, int k, int oversample);
size_t defl_psd_workspace_bytes(int n, int K);

/* The paper gives the estimation window and the oversampling as ratios of the short side (Algorithm 3, line 1:
 * r = ceil(w m), r' = min{m, r + ceil(delta m)}; Algorithm 2: r = ceil(w n), K = ceil(w' n)). These two calls turn
 * the ratios into the counts the compute calls take: *k = r, *oversample = r' - r (polar, m the short side of an
 * m x n matrix; r is capped at m - 1), and *k = r, *K = ceil(w' n) (PSD; r is capped at K). Host arithmetic only.
 * With opts->tau > 0 the window is what the gate looks at and k_used reports how many of the r were deflated.
 * Returns DEFL_ERR_RANK when the widths exceed DEFL_MAX_L (the counts are still written), DEFL_ERR_ARG for negative
 * ratios, non-positive sizes or null pointers. */
int defl_polar_window(int m, int n, float w, float delta, int* k, int* oversample);
int defl_psd_window(int n, float w, float w_prime, int* k, int* K);

/* Deflated polar factor of a batch (Algorithm 3 then Algorithm 1, fixed-k reading).
 *   G    [b,m,n] dtype, not modified.         out [b,m,n] dtype, must not overlap G.
 *   k            number of triplets deflated; k = 0 runs the plain filter X0 = G/||G||_F (Algorithm 1, else-branch).
 *   oversample   extra sketch columns p; l = min(min(m,n), k+p) columns are sketched (Algorithm 3 line 1).
 *   power_iters  J subspace iterations (Algorithm 3 lines 4-6).
 *   coeff_schedule  host, [L][3] = (a_t, b_t, c_t) of X <- a X + b (X X^T) X + c (X X^T)^2 X (Eq. 2), applied
 *                for t = 1..L in order ([L][opts->poly_terms] for the other degrees of Eq. 5). L = 0 returns X0.
 * Wide matrices (m < n) are handled as the transpose without moving data (polar(M^T) = polar(M)^T).
 * Two steps per pass: each step is evaluated through the short-side Gram matrix A_t = X_t X_t^T and B_t = a I + b A_t +
 * c A_t^2 as X_{t+1} = B_t X_t (Eq. 2). On the bf16 tensor path, when the long side is at least twice the short one,
 * two consecutive quintic steps share one pass over X: since B_t is a polynomial in A_t, A_{t+1} = B_t^2 A_t needs no
 * product with X, and X_{t+2} = (B_{t+1} B_t) X_t: one Gram and one apply product of ms^2 ml each and five ms^3
 * products instead of two of each big product and two small ones; the same composite polynomial, another order of
 * evaluation. Both steps are kept in scaled IEEE half, and a pair starts at step t only where |a_t| <= 4.5 and
 * |b_{t+1} + 2 c_{t+1}| <= 1 (the two gains with which the rounding of the stored A_t reaches the result; Muon's and
 * the classical quintic qualify, the steep steps of a per-step minimax schedule do not). Not with the fp32 engine, not
 * with opts->bf16_iterates = 1, not for the other degrees of Eq. 5.
 * Errors: DEFL_ERR_ARG, DEFL_ERR_RANK (k >= min(m,n) or l > DEFL_MAX_L or L > DEFL_MAX_STEPS), DEFL_ERR_CUDA,
 * DEFL_ERR_UNSUPPORTED. opts and info may be NULL. */
int defl_polar_batched(defl_ctx* ctx, const void* G, void* out, int b, int m, int n, int dtype,
                       int k, int oversample, int power_iters,
                       const float* coeff_schedule, int L,
                       const defl_opts* opts, const defl_info* info);

/* The same call for HOST buffers: G_host and out_host are host memory (pinned memory makes the copies
 * asynchronous and fast). The library copies G to device staging memory it owns, runs defl_polar_batched,
 * copies the result back and synchronises before returning, so out_host is ready on return. The batch goes
 * through in a few chunks of whole matrices, the copies of one chunk overlapping the computation of another on
 * streams the context owns; every matrix gets the result (and the sketch) it would get from one
 * defl_polar_batched call on the whole batch. opts->sketch, if given, is still device memory. Same errors as
 * defl_polar_batched. */
int defl_polar_batched_host(defl_ctx* ctx, const void* G_host, void* out_host, int b, int m, int n, int dtype,
                            int k, int oversample, int power_iters,
                            const float* coeff_schedule, int L, const defl_opts* opts);

/* One Deflated Muon step for a group of same-shape matrices (Section 3, "Muon with deflation": the polar-factor
 * routine inside Muon is replaced by Algorithm 3 + Algorithm 1, once per shape group; Section 1, "Two
 * applications": W <- W - lambda polar(M) with M the momentum matrix). In this order, all on the context's stream:
 *   Mom <- mu * Mom + Grad              (skipped when Grad is NULL: Mom is then taken as it is)
 *   D    = Mom, or Grad + mu * Mom when `nesterov` is non-zero (Mom here is the new momentum as stored)
 *   W   <- (1 - lr * weight_decay) * W - lr * scale * F(D)
 * where F is exactly what defl_polar_batched computes (same k, oversample, power_iters, schedule, opts, info).
 * The weight update is the epilogue of the last filter product (and of the restore product in ADD mode): F(D) is
 * never written to memory. The paper fixes only the last line with lr = lambda, scale = 1, weight_decay = 0; the
 * momentum rule, Nesterov form, decoupled weight decay and `scale` are the usual Muon conventions, stated here
 * because the paper takes them from the Muon references.
 *   W    device, [b,m,n] row-major, type w_dtype (DEFL_BF16 | DEFL_F32), updated in place
 *   Mom  device, [b,m,n], type dtype, updated in place;  Grad  device, [b,m,n], type dtype, not modified, or NULL
 * L >= 1 is required (the update rides on the last product). Scratch: the context's workspace plus two buffers of
 * b*m*n elements of `dtype` that it keeps. Errors as defl_polar_batched; DEFL_ERR_ARG also for nesterov without
 * Grad. */
int defl_muon_step_batched(defl_ctx* ctx, void* W, int w_dtype, void* Mom, const void* Grad, int b, int m, int n,
                           int dtype, float lr, float mu, int nesterov, float weight_decay, float scale,
                           int k, int oversample, int power_iters, const float* coeff_schedule, int L,
                           const defl_opts* opts, const defl_info* info);

/* Batched randomized SVD alone (Algorithm 3) in the caller's orientation:
 *   G ~ P diag(s) W^T with P [b,m,l], s [b,l] descending, W [b,n,l], all fp32; l = min(min(m,n), k+oversample).
 * Any of P, s, W may be NULL. The sketch comes from opts as above. */
int defl_brsvd_batched(defl_ctx* ctx, const void* G, int b, int m, int n, int dtype,
                       int k, int oversample, int power_iters,
                       float* P, float* s, float* W, const defl_opts* opts, int* status);

/* Deflated PSD projection (Algorithm 2, fixed-k reading) of one symmetric matrix.
 *   X  [n,n] fp32 symmetric, not modified.   P [n,n] fp32, exactly symmetric on return, must not overlap X.
 *   warm_basis [n,K] fp32 with orthonormal columns, IN/OUT: on return the orthonormalised Z V (line 9).
 *   k  Ritz pairs of largest magnitude to deflate (k <= K); k = 0 or opts->warmup: Eq. 7.
 *   coeff_schedule host, [T][3]: the composite odd filter g = p_T o ... o p_1, p_t(x) = a x + b x^3 + c x^5.
 * The only state carried between calls is warm_basis, which the caller owns. */
int defl_psd_project(defl_ctx* ctx, const void* X, void* P, int n, int k,
                     float* warm_basis, int K,
                     const float* coeff_schedule, int T,
                     const defl_opts* opts, const defl_info* info);

/* Deflated inverse matrix root  out ~ A^(-1/p)  of one symmetric positive definite matrix (Conclusion: inverse
 * matrix roots, the preconditioners of Shampoo-type optimizers, are named as the next instance of the framework; the
 * paper gives no algorithm for it, so each step below is the one it defines for its own instances):
 *   1. block step A V, Rayleigh-Ritz on the tracked basis, the k leading eigenpairs (lambda_i, u_i) removed:
 *      R = A - sum lambda_i u_i u_i^T                                        (Algorithm 2, lines 1-5)
 *   2. theta = Lanczos upper estimate of ||R||_2 (Appendix E.1, "Normalization scale");
 *      X0 = R / theta + (1/gamma) sum u_i u_i^T                              (Algorithm 2, line 7; Algorithm 1, line 4)
 *   3. `steps` steps of the coupled Newton iteration, matrix products only:
 *      T_t = ((p+1) I - M_t) / p,  Z_{t+1} = Z_t T_t,  M_{t+1} = T_t^p M_t,  M_0 = X0, Z_0 = I
 *   4. out = theta^(-1/p) (Z - z_pad sum u_i u_i^T) + sum lambda_i^(-1/p) u_i u_i^T, symmetrised, where z_pad is the
 *      value the scalar iteration gives the padding 1/gamma: the head is restored exactly (Eq. 3 in padded form)
 *   5. warm_basis <- orthonormalised A V                                     (Algorithm 2, line 9)
 *   A  [n,n] fp32 symmetric positive definite, not modified.  out [n,n] fp32, exactly symmetric on return, must not
 *   overlap A.  warm_basis [n,K] fp32 with orthonormal columns, IN/OUT (K = 0: no deflation).  p in {1, 2, 4}.
 *   k <= K eigenpairs to remove; k = 0 or opts->warmup: the plain normalised iteration.  steps <= DEFL_MAX_STEPS.
 * The basis must have settled before eigenpairs are removed (run the first calls with opts->warmup, as the paper does
 * for the projection): a Ritz pair (lambda, u) with residual r = A u - lambda u leaves R indefinite, with an eigenvalue
 * near -|r|^2 / a, a = r^T A r / |r|^2; the padding keeps X0 positive definite while |r|^2 < a theta / gamma, and on an
 * eigenvalue that is not positive the iteration diverges. A result that is not finite sets DEFL_ST_NONFINITE.
 * Products on the tensor cores in tf32 (iterates stored rounded to tf32) unless opts->engine = DEFL_ENGINE_SIMT
 * (exact fp32 products). Read from opts: gamma (default 1.1), engine, warmup, tau (gate on the Ritz values, as in
 * defl_psd_project), norm_mode, lanczos_start, seed, exploit_symmetry. info: s = the K Ritz values by decreasing
 * magnitude, rho = theta, k_used, status (a removed Ritz value that is not positive sets DEFL_ST_NONFINITE and leaves
 * that direction at the iteration's value: the matrix is not positive definite there).
 * Errors: DEFL_ERR_ARG (null pointers, overlap, p not in {1,2,4}, steps < 0), DEFL_ERR_RANK (k > K, K > DEFL_MAX_L,
 * K >= n, steps > DEFL_MAX_STEPS), DEFL_ERR_CUDA. */
int defl_inv_root(defl_ctx* ctx, const void* A, void* out, int n, int p, int k,
                  float* warm_basis, int K, int steps,
                  const defl_opts* opts, const defl_info* info);

/* Three-block ADMM for a standard-form SDP whose constraints are diag(X) = b (max-cut type):
 *   min <C, X>  s.t.  diag(X) = b, X PSD;   A(X) = diag(X), A*(y) = Diag(y), A A* = I.
 * One iteration (Appendix E.1, "ADMM for Standard-Form SDP": the ADMM iteration; the S-update is Algorithm 2 through defl_psd_project):
 *   y <- b / sigma - diag(X / sigma + S - C)
 *   Z  = C - Diag(y) - X / sigma;        S <- projection of Z on the PSD cone (deflated, basis carried along)
 *   X <- X + sigma (S + Diag(y) - C)
 * After every iteration the three eigenvalue-free KKT terms of Appendix E.4, "Experimental Details" are evaluated on the device:
 *   residuals[3 it + 0] = ||diag(X) - b||_2 / (1 + ||b||_2)
 *   residuals[3 it + 1] = ||Diag(y) + S - C||_F / (1 + ||C||_F)
 *   residuals[3 it + 2] = |<C, X> - b^T y| / (1 + |<C, X>| + |b^T y|)
 *   C  device, [n,n] fp32 symmetric, not modified;  b  device, [n] fp32;  n a multiple of 4
 *   X, S  device, [n,n] fp32, IN/OUT: the iterates (zeros for a cold start);  y  device, [n] fp32, OUT
 *   warm_basis, K, k, coeff_schedule, T, opts: as defl_psd_project; the first `warmup_iters` iterations run with
 *   the gate off (opts->warmup), as the paper does while the basis settles
 *   residuals  HOST, [iters][3] fp32, written before the call returns (may be NULL); the call synchronises the
 *   stream twice (norms of b and C at the start, the residual history at the end)
 * Scratch besides the projection's workspace: two buffers of n*n fp32 the context keeps. Errors as
 * defl_psd_project; DEFL_ERR_ARG also for n not a multiple of 4 or sigma <= 0. */
int defl_admm_diag_sdp(defl_ctx* ctx, const void* C, const float* b, int n, float sigma, int iters, int warmup_iters,
                       void* X, void* S, float* y, int k, float* warm_basis, int K,
                       const float* coeff_schedule, int T, const defl_opts* opts, float* residuals);

/* Counter-based standard-normal fill (the sketch of Algorithm 3 when none is passed):
 *   h(x): x += 0x9E3779B97F4A7C15; x = (x ^ x>>30) * 0xBF58476D1CE4E5B9; x = (x ^ x>>27) * 0x94D049BB133111EB; x ^ x>>31
 *   j = idx/2; r1 = h(h(seed) ^ 2j); r2 = h(h(seed) ^ (2j+1)); u1 = ((r1>>11)+1) 2^-53; u2 = (r2>>11) 2^-53
 *   value(idx) = sqrt(-2 ln u1) * (idx even ? cos(2 pi u2) : sin(2 pi u2)), evaluated in fp64, rounded to dtype.
 * dst is device memory of `count` elements of dtype (DEFL_BF16 or DEFL_F32). */
int defl_fill_gaussian(defl_ctx* ctx, void* dst, size_t count, int dtype, uint64_t seed);

/* Batched Frobenius norms without any allocation (no counterpart in the paper; it is the normalisation
 * scale ||M||_F of Eq. 1 offered on its own). Written for callers that cannot allocate device memory when
 * they call: code running inside another allocator's critical section or with all device memory already
 * handed to a pool, and latency-critical loops where cudaMalloc's implicit device synchronisation is not
 * acceptable. It needs no context and calls no cudaMalloc, cudaFree or allocating library routine: the
 * partial sums live in a fixed array inside the library (DEFL_NOALLOC_MAX_BATCH x 148 doubles, about
 * 300 KB, held by every GPU that loads the library until the process exits).
 *   X      device, [b, count] of dtype (DEFL_BF16 or DEFL_F32), b matrices of `count` elements each
 *   norms  device, [b] fp32, receives ||X[i]||_F
 *   cuda_stream  cudaStream_t to enqueue on (NULL = default stream); the call does not synchronise
 * Works on the CURRENT device. The first call on each device looks up that device's address of the array
 * (a host-side query, no allocation); make that first call before starting any stream capture.
 * All calls on a device share the array, so two calls whose kernels may overlap on the GPU (different
 * streams, no ordering between them) race; calls on one stream are safe. Nothing needs clearing between
 * calls: every slot that is read has just been written.
 * Errors: DEFL_ERR_ARG (null pointer, b <= 0, count <= 0, bad dtype), DEFL_ERR_RANK (b > DEFL_NOALLOC_MAX_BATCH;
 * split the batch), DEFL_ERR_CUDA. */
#define DEFL_NOALLOC_MAX_BATCH 256
int defl_frobenius_norms_noalloc(const void* X, int dtype, int b, long long count, float* norms, void* cuda_stream);

/* Diagnostics: one batched product C[b,M,N] = alpha * opA(A) opB(B) through a chosen engine, used by the
 * tests to check the tensor-core tile engine against the fp32 engine (no counterpart in the paper).
 * A element (i,kk) is A[i*sa_i + kk*sa_k], B element (kk,j) is B[kk*sb_k + j*sb_j]; C is row-major [M,N].
 * in_dtype / out_dtype are DEFL_BF16 or DEFL_F32; strides in elements. exploit_symmetry: bit 0 = the product is
 * symmetric (upper tiles computed and mirrored); bit 1 = the product is written transposed, C row-major [N,M]
 * (tensor engine only; DEFL_ERR_UNSUPPORTED otherwise); bit 2 = test of the bounded waits (tensor engine, outputs
 * of at most 128 rows): the first pipeline step of every CTA's first tile is never copied, so the wait for it runs
 * out after the context's wait limit, C is not written and defl_device_wait_status reports DEFL_ST_DEVICE_WAIT. */
int defl_debug_gemm(defl_ctx* ctx, int engine, int batch, int M, int N, int K,
                    const void* A, long long sa_i, long long sa_k, long long batch_a,
                    const void* B, long long sb_k, long long sb_j, long long batch_b,
                    void* C, int in_dtype, int out_dtype, float alpha, int exploit_symmetry);

/* Stage timing: when enabled, the context records CUDA events between the stages of each call;
 * defl_get_stage_ms synchronises the stream and writes up to `cap` stage durations (ms) of the last
 * call, returning how many stages there were. Polar stages: 0 randomized SVD (Algorithm 3),
 * 1 deflate + normalise, 2 filter, 3 restore. PSD stages: 0 block step + Rayleigh-Ritz, 1 deflate,
 * 2 Lanczos scale, 3 initialisation, 4 filter, 5 reconstruction, 6 basis update. */
int defl_set_profiling(defl_ctx* ctx, int enabled);
int defl_get_stage_ms(defl_ctx* ctx, float* ms, int cap);
/* The same durations added up over the last `ncalls` calls of the context (at most 64 are kept), so that a timed
 * loop can be split into stages afterwards without a synchronisation between its calls. */
int defl_get_stage_ms_sum(defl_ctx* ctx, float* ms, int cap, int ncalls);

/* Number of kernels the library launched on this context since creation. */
long long defl_launch_count(defl_ctx* ctx);

/* The tensor engine's wait word of this context: every device-side wait of its kernels (on a copy, on a free
 * pipeline stage, on an accumulator) is bounded; one that runs out sets DEFL_ST_DEVICE_WAIT in this word, the kernel
 * stops waiting, lets its copies land, frees its tensor memory and returns. defl_polar_batched, defl_psd_project
 * and the calls built on them clear the word when they start and fold it into defl_info.status when they end; this
 * call is for the others (defl_debug_gemm). It synchronises the context's stream, returns the word (>= 0, or a
 * negative DEFL_ERR_*), and clears it when `clear` is non-zero. No counterpart in the paper. */
int defl_device_wait_status(defl_ctx* ctx, int clear);

const char* defl_status_string(int code);
const char* defl_last_error(defl_ctx* ctx); /* text of the last CUDA failure, "" if none */

#ifdef __cplusplus
}
#endif
#endif /* DEFL_H_ */
