// C ABI of the library: context, scratch memory, and the orchestration of the deflated polar factor
// (Algorithm 3 + Algorithm 1) as a sequence of kernel launches on one stream. The PSD projection
// lives in psd.cu. Nothing here computes on the host beyond choosing launch parameters.
#include "../../include/defl.h"
#include "common.cuh"
#include "panel.cuh"
#include "ctx.cuh"
#include <cstdlib>

#include <cstdio>
#include <cstring>
#include <new>

using namespace defl;

namespace defl {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool ctx_fail(defl_ctx* c, cudaError_t e, const char* where) {
  if (e == cudaSuccess) return false;
  snprintf(c->err, sizeof(c->err), "%s: %s", where, cudaGetErrorString(e));
  return true;
}

int ctx_reserve(defl_ctx* c, size_t bytes) {
  if (bytes <= c->ws_bytes) return DEFL_OK;
  if (c->ws) {
    cudaDeviceSynchronize();
    cudaFree(c->ws);
    c->ws = nullptr;
    c->ws_bytes = 0;
  }
  void* p = nullptr;
  if (ctx_fail(c, cudaMalloc(&p, bytes), "cudaMalloc(workspace)")) return DEFL_ERR_CUDA;
  c->ws = p;
  c->ws_bytes = bytes;
  return DEFL_OK;
}

void ctx_profile_begin(defl_ctx* c) {
  if (!c->profiling || !c->marks_ready) return;
  ++c->call_seq;
  c->n_marks[c->call_seq % DEFL_PROFILE_CALLS] = 0;
}

void ctx_stage_mark(defl_ctx* c) {
  if (!c->profiling || !c->marks_ready || c->call_seq == 0) return;
  const int slot = (int)(c->call_seq % DEFL_PROFILE_CALLS);
  if (c->n_marks[slot] >= DEFL_MAX_MARKS) return;
  cudaEventRecord(c->marks[slot][c->n_marks[slot]++], c->stream);
}

// Which engine a product runs on. AUTO sends bf16 products to the tensor cores and keeps fp32
// products on exact fp32 FMA; ENGINE_TENSOR also sends fp32 products there (as tf32).
bool use_tensor_engine(const GemmDesc& g, int engine) {
  if (engine == DEFL_ENGINE_SIMT) return false;
  if (engine == DEFL_ENGINE_AUTO && g.in_dtype == F32) return false;
  return gemm_tc_supported(g);
}

// Run one product on the engine the options ask for. Returns a DEFL_* code.
int run_gemm(defl_ctx* c, const GemmDesc& g, int engine, const char* what) {
  const bool tc = use_tensor_engine(g, engine);
  if ((engine == DEFL_ENGINE_TENSOR || g.transpose_out) && !tc) {
    snprintf(c->err, sizeof(c->err), "%s: shape/type not supported by the tensor engine", what);
    return DEFL_ERR_UNSUPPORTED;
  }
  cudaError_t e;
  if (tc) e = gemm_tc_launch(g, c->stream, c->wait_status, c->num_sms, &c->launches, &c->tc_knobs, &c->tm_cache);
  else e = gemm_simt_launch(g, c->stream, &c->launches);
  if (ctx_fail(c, e, what)) return DEFL_ERR_CUDA;
  return DEFL_OK;
}

int partials_per_batch(defl_ctx* c, const GemmDesc& g, int engine) {
  if (use_tensor_engine(g, engine)) return gemm_tc_partials_per_batch(g, &c->tc_knobs);
  return gemm_simt_partials_per_batch(g);
}

struct Carver {
  char* base; size_t off;
  explicit Carver(void* p) : base(reinterpret_cast<char*>(p)), off(0) {}
  template <typename T> T* take(size_t count) {
    T* r = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off = align_up(off + count * sizeof(T), 256);
    return r;
  }
};

// Workspace layout of one polar call (also used, with a null base, to size it).
struct PolarWs {
  void* X;            // [b,m,n] dtype   second iterate buffer (the other one is `out`)
  void* Am; void* Bm; // [b,ms,ms] dtype  A_t = X X^T and B_t = a I + b A_t + c A_t^2
  void* Cm;           // [b,ms,ms] dtype  Horner intermediate of the higher-degree maps (poly_terms > 3), B_t^2 and B_{t+1} B_t of a paired step
  void* Dm;           // [b,ms,ms] dtype  A_{t+1} = B_t^2 A_t of a paired step
  float* Lp;          // [b,ml,l]  long-side panel  (Y, then Q)
  float* Sp;          // [b,ms,l]  short-side panel (A^T Q and its orthonormalisation; finally (Q^T A)^T)
  double* gram;       // [b,nchunk,l,l]
  float* Rinv; float* E; float* Es; float* sv;   // [b,l,l] x3, [b,l]
  float* Uk; float* Vk;   // [b,ml,k], [b,ms,k]  leading triplets in the tall orientation
  float* Ws;          // [b,n,k] scaled copy of the right factor
  double* npart;      // [b,nper] Frobenius partial sums
  float* rho; float* inv_rho; float* inv_rho2;   // [b]
  int* status;        // [b]
  int* keff;          // [b] components deflated per matrix (gate)
  float* sketch;      // [b,ms,l] when the library draws the sketch
  // split-precision bf16 copies for the tensor engine (bf16 storage only)
  __nv_bfloat16* Lhi; __nv_bfloat16* Llo;   // [b,ml,lp]
  __nv_bfloat16* Shi; __nv_bfloat16* Slo;   // [b,ms,lp]
  __nv_bfloat16* Pc; __nv_bfloat16* Wc;     // [b,m,3kp], [b,n,3kp]
  size_t bytes;
};

inline int round_up8(int x) { return (x + 7) & ~7; }

// Two filter steps per pass over X (see the filter stage) pay when the long side is at least twice the short one:
// per pair, three more ms^3 products against one Gram and one apply product of ms^2 ml each
static bool paired_steps_shape(int m, int n, int dtype) {
  const int ms = m < n ? m : n, ml = m < n ? n : m;
  return dtype == BF16 && ml >= 2 * ms;
}

PolarWs carve_polar(void* base, int b, int m, int n, int dtype, int k, int l, int terms = 3) {
  const int ms = m < n ? m : n, ml = m < n ? n : m;
  const size_t es = dtype_size(dtype);
  Carver cv(base);
  PolarWs w;
  w.X = cv.take<char>((size_t)b * m * n * es);
  w.Am = cv.take<char>((size_t)b * ms * ms * es);
  w.Bm = cv.take<char>((size_t)b * ms * ms * es);
  const bool pairable = paired_steps_shape(m, n, dtype);
  w.Cm = cv.take<char>((terms > 3 || pairable) ? (size_t)b * ms * ms * es : 1);
  w.Dm = cv.take<char>(pairable ? (size_t)b * ms * ms * es : 1);
  const int le = l > 0 ? l : 1, ke = k > 0 ? k : 1;
  w.Lp = cv.take<float>((size_t)b * ml * le);
  w.Sp = cv.take<float>((size_t)b * ms * le);
  w.gram = cv.take<double>((size_t)b * gram_num_chunks(ml) * le * le);
  w.Rinv = cv.take<float>((size_t)b * le * le);
  w.E = cv.take<float>((size_t)b * le * le);
  w.Es = cv.take<float>((size_t)b * le * le);
  w.sv = cv.take<float>((size_t)b * le);
  w.Uk = cv.take<float>((size_t)b * ml * ke);
  w.Vk = cv.take<float>((size_t)b * ms * ke);
  w.Ws = cv.take<float>((size_t)b * n * ke);
  // norm partials: enough for either engine's tiling of an m x n output
  const size_t nper = (size_t)((m + 63) / 64) * ((n + 15) / 16) * 4 + 1184;
  w.npart = cv.take<double>((size_t)b * nper);
  w.rho = cv.take<float>(b);
  w.inv_rho = cv.take<float>(b);
  w.inv_rho2 = cv.take<float>(b);
  w.status = cv.take<int>(b);
  w.keff = cv.take<int>(b);
  w.sketch = cv.take<float>((size_t)b * ms * le);
  const int lp = round_up8(le), kp = round_up8(ke);
  const bool bf = (dtype == BF16);
  w.Lhi = cv.take<__nv_bfloat16>(bf ? (size_t)b * ml * lp : 1);
  w.Llo = cv.take<__nv_bfloat16>(bf ? (size_t)b * ml * lp : 1);
  w.Shi = cv.take<__nv_bfloat16>(bf ? (size_t)b * ms * lp : 1);
  w.Slo = cv.take<__nv_bfloat16>(bf ? (size_t)b * ms * lp : 1);
  w.Pc = cv.take<__nv_bfloat16>(bf ? (size_t)b * m * 3 * kp : 1);
  w.Wc = cv.take<__nv_bfloat16>(bf ? (size_t)b * n * 3 * kp : 1);
  w.bytes = cv.off;
  return w;
}

// CholeskyQR2 of the panel P[b, rows, l] in place: twice { W = P^T P; W = R^T R; P <- P R^-1 }.
int orthonormalise(defl_ctx* c, float* P, int b, int rows, int l, double* gram, float* Rinv, int* status,
                   __nv_bfloat16* hi, __nv_bfloat16* lo, int lp, int passes) {
  // CholeskyQR: Gram(P); R = chol; P <- P R^-1. With passes = 2 (CholeskyQR2) the second Gram is taken in the
  // same panel pass as the first solve. The last pass can also write P as bf16 hi + lo for the next
  // tensor-core product.
  const int nchunk = fused_num_chunks(rows, b);
  const long long bs = (long long)rows * l;
  if (ctx_fail(c, panel_fused_launch(P, bs, l, b, rows, l, nullptr, 0, l, nullptr, 0, 0, nullptr, nullptr, 0, gram,
                                     c->stream, &c->launches), "gram"))
    return DEFL_ERR_CUDA;
  if (ctx_fail(c, chol_inv_launch(gram, nchunk, b, l, Rinv, status, c->stream, &c->launches), "cholesky"))
    return DEFL_ERR_CUDA;
  if (passes >= 2) {
    if (ctx_fail(c, panel_fused_launch(P, bs, l, b, rows, l, Rinv, l, l, P, bs, l, nullptr, nullptr, 0, gram, c->stream,
                                       &c->launches), "apply + gram"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, chol_inv_launch(gram, nchunk, b, l, Rinv, status, c->stream, &c->launches), "cholesky"))
      return DEFL_ERR_CUDA;
  }
  if (ctx_fail(c, panel_fused_launch(P, bs, l, b, rows, l, Rinv, l, l, P, bs, l, hi, lo, lp, nullptr, c->stream,
                                     &c->launches), "apply"))
    return DEFL_ERR_CUDA;
  return DEFL_OK;
}

// Algorithm 3 on the batch: on return w.Lp = Q U_G (left vectors of A, all l), w.Sp... see below.
// Outputs: w.sv[b,l], w.Uk[b,ml,k_keep] and w.Vk[b,ms,k_keep] (leading k_keep triplets of A = G or G^T).
int run_brsvd(defl_ctx* c, const void* G, int b, int m, int n, int dtype, int l, int J, int k_keep,
              const float* sketch, const PolarWs& w, int engine) {
  const bool tall = m >= n;
  const int ms = tall ? n : m, ml = tall ? m : n;
  // element (i,j) of A (ml x ms): tall G[i*n+j]; wide G[j*n+i]
  const long long a_si = tall ? n : 1, a_sj = tall ? 1 : n;
  int rc;
  // Products with G on the tensor engine: the fp32 panel is split into bf16 hi + lo, both multiplied by the
  // same G tile and accumulated in fp32 (G is bf16 already). Falls back to the fp32 engine when the shape or
  // type does not fit (fp32 storage, strides not multiples of 16 bytes) or when that engine is requested.
  const int lp = round_up8(l);
  auto mul_G = [&](bool transposed, const float* Bp, float* Cp, bool presplit) {   // C = A B (ml x l) or A^T B (ms x l)
    const int M = transposed ? ms : ml, K = transposed ? ml : ms;
    GemmDesc g = gemm_desc_zero();
    g.batch = b; g.M = M; g.N = l; g.K[0] = K;
    g.A[0] = G; g.batch_a[0] = (long long)m * n; g.in_dtype = dtype;
    g.sa_i[0] = transposed ? a_sj : a_si; g.sa_k[0] = transposed ? a_si : a_sj;
    g.C = Cp; g.ldc = l; g.batch_c = (long long)M * l; g.out_dtype = F32;
    g.epilogue = EPI_STORE;
    if (dtype == BF16 && engine != DEFL_ENGINE_SIMT) {
      __nv_bfloat16* hi = transposed ? w.Lhi : w.Shi;
      __nv_bfloat16* lo = transposed ? w.Llo : w.Slo;
      GemmDesc t = g;
      t.B[0] = hi; t.B[1] = lo; t.b_split = 2; t.b_dtype = BF16;
      t.sb_k[0] = lp; t.sb_j[0] = 1; t.batch_b[0] = (long long)K * lp;
      if (gemm_tc_supported(t)) {
        if (!presplit &&
            ctx_fail(c, split_panel_launch(Bp, (long long)K * l, l, b, K, l, lp, hi, lo, c->stream, &c->launches), "split panel"))
          return (int)DEFL_ERR_CUDA;
        return run_gemm(c, t, DEFL_ENGINE_TENSOR, "G*panel (tensor)");
      }
    }
    g.B[0] = Bp; g.sb_k[0] = l; g.sb_j[0] = 1; g.batch_b[0] = (long long)K * l; g.b_dtype = F32;
    return run_gemm(c, g, DEFL_ENGINE_SIMT, "G*panel");
  };
  // after an orthonormalisation the panel's bf16 split already exists (written by its last pass)
  const bool split_out = (dtype == BF16 && engine != DEFL_ENGINE_SIMT);
  auto mul_A = [&](const float* Bp, float* Cp, bool presplit) { return mul_G(false, Bp, Cp, presplit); };
  auto mul_At = [&](const float* Bp, float* Cp, bool presplit) { return mul_G(true, Bp, Cp, presplit); };
  // The basis that defines B = Q^T A gets CholeskyQR2; the intermediate bases of the subspace iteration only
  // need to stay well conditioned, so one CholeskyQR pass (as Algorithm 3 prints it) is enough there: any
  // basis of the same span gives the same triplets.
  auto orth_long = [&](int passes) {
    return orthonormalise(c, w.Lp, b, ml, l, w.gram, w.Rinv, w.status, split_out ? w.Lhi : nullptr,
                          split_out ? w.Llo : nullptr, lp, passes);
  };
  auto orth_short = [&](int passes) {
    return orthonormalise(c, w.Sp, b, ms, l, w.gram, w.Rinv, w.status, split_out ? w.Shi : nullptr,
                          split_out ? w.Slo : nullptr, lp, passes);
  };
  if ((rc = mul_A(sketch, w.Lp, false))) return rc;                        // Y = A Omega
  if ((rc = orth_long(J == 0 ? 2 : 1))) return rc;                          // Q
  for (int j = 0; j < J; ++j) {
    if ((rc = mul_At(w.Lp, w.Sp, split_out))) return rc;                   // A^T Q
    if ((rc = orth_short(1))) return rc;
    if ((rc = mul_A(w.Sp, w.Lp, split_out))) return rc;                    // A Y
    if ((rc = orth_long(j + 1 == J ? 2 : 1))) return rc;
  }
  if ((rc = mul_At(w.Lp, w.Sp, split_out))) return rc;                     // (Q^T A)^T, [ms, l]
  // thin SVD of Q^T A through the Gram core: (Q^T A)(Q^T A)^T = E diag(s^2) E^T
  if (ctx_fail(c, panel_fused_launch(w.Sp, (long long)ms * l, l, b, ms, l, nullptr, 0, l, nullptr, 0, 0, nullptr, nullptr, 0,
                                     w.gram, c->stream, &c->launches), "gram core"))
    return DEFL_ERR_CUDA;
  if (ctx_fail(c, jacobi_eig_launch(w.gram, fused_num_chunks(ms, b), b, l, 0, w.sv, w.E, w.Es, w.status, c->stream,
                                    &c->launches, c->knobs.jacobi_sweeps), "jacobi"))
    return DEFL_ERR_CUDA;
  if (k_keep > 0) {
    // U = Q E (long side), V = (Q^T A)^T E diag(1/s) (short side); keep the leading k_keep columns
    if (ctx_fail(c, panel_fused_launch(w.Lp, (long long)ml * l, l, b, ml, l, w.E, l, k_keep, w.Uk, (long long)ml * k_keep,
                                       k_keep, nullptr, nullptr, 0, nullptr, c->stream, &c->launches), "U = Q E"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, panel_fused_launch(w.Sp, (long long)ms * l, l, b, ms, l, w.Es, l, k_keep, w.Vk, (long long)ms * k_keep,
                                       k_keep, nullptr, nullptr, 0, nullptr, c->stream, &c->launches), "V = B^T E / s"))
      return DEFL_ERR_CUDA;
  }
  return DEFL_OK;
}

const float* resolve_sketch(defl_ctx* c, const defl_opts* opts, int b, int ms, int l, const PolarWs& w, int* rc) {
  *rc = DEFL_OK;
  if (opts && opts->sketch) return opts->sketch;
  const unsigned long long seed = opts ? opts->seed : 0ull;
  if (ctx_fail(c, fill_gaussian_launch(w.sketch, (long long)b * ms * l, F32, seed, (long long)ms * l, 1ull, c->stream,
                                       &c->launches), "sketch"))
    *rc = DEFL_ERR_CUDA;
  return w.sketch;
}

}  // namespace defl

// ================================================================================================
extern "C" {

int defl_create(defl_ctx** out, int device) {
  if (!out) return DEFL_ERR_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return DEFL_ERR_CUDA;
  int prev = 0;
  cudaGetDevice(&prev);
  if (cudaSetDevice(device) != cudaSuccess) return DEFL_ERR_CUDA;
  defl_ctx* c = new (std::nothrow) defl_ctx();
  if (!c) return DEFL_ERR_CUDA;
  memset(c, 0, sizeof(*c));
  c->device = device;
  // every environment override is read here, once: nothing on the call path looks at the environment
  c->tc_knobs = tc_knobs_from_env();
  c->knobs.transposed_apply = getenv("DEFL_NO_TRANSPOSED_APPLY") ? 0 : 1;
  c->knobs.host_chunks = getenv("DEFL_HOST_CHUNKS") ? atoi(getenv("DEFL_HOST_CHUNKS")) : 0;
  c->knobs.jacobi_sweeps = getenv("DEFL_JACOBI_SWEEPS") ? atoi(getenv("DEFL_JACOBI_SWEEPS")) : 0;
  c->knobs.paired_steps = getenv("DEFL_NO_PAIRED_STEPS") ? 0 : 1;
  cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device);
  int ok = 1;
  if (cudaMalloc(&c->wait_status, 2 * sizeof(int)) != cudaSuccess) ok = 0;      // status word, tile counter
  if (ok) cudaMemset(c->wait_status, 0, 2 * sizeof(int));
  if (ok) {
    // identity tile of the tensor engine's identity segment (X0 = (G - head) / rho adds G in the accumulator)
    const size_t ib = 256 * 256 * sizeof(__nv_bfloat16);
    __nv_bfloat16* h = new (std::nothrow) __nv_bfloat16[256 * 256];
    if (!h || cudaMalloc(&c->ident_bf16, ib) != cudaSuccess) ok = 0;
    if (ok) {
      for (int i = 0; i < 256 * 256; ++i) h[i] = __float2bfloat16((i / 256 == i % 256) ? 1.f : 0.f);
      if (cudaMemcpy(c->ident_bf16, h, ib, cudaMemcpyHostToDevice) != cudaSuccess) ok = 0;
    }
    delete[] h;
  }
  if (!ok) {      // release whatever was created before the failure
    if (c->wait_status) cudaFree(c->wait_status);
    if (c->ident_bf16) cudaFree(c->ident_bf16);
    cudaSetDevice(prev);
    delete c;
    return DEFL_ERR_CUDA;
  }
  cudaSetDevice(prev);
  *out = c;
  return DEFL_OK;
}

int defl_destroy(defl_ctx* c) {
  if (!c) return DEFL_ERR_ARG;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  if (c->ws) cudaFree(c->ws);
  if (c->stage_in) cudaFree(c->stage_in);
  if (c->stage_out) cudaFree(c->stage_out);
  if (c->copy_ready) {
    cudaStreamDestroy(c->copy_in);
    cudaStreamDestroy(c->copy_out);
    for (int i = 0; i < DEFL_HOST_MAX_CHUNKS; ++i) { cudaEventDestroy(c->chunk_in[i]); cudaEventDestroy(c->chunk_done[i]); }
  }
  if (c->wait_status) cudaFree(c->wait_status);
  if (c->ident_bf16) cudaFree(c->ident_bf16);
  for (int r = 0; r < DEFL_PROFILE_CALLS; ++r)
    for (int i = 0; i < DEFL_MAX_MARKS; ++i)
      if (c->marks[r][i]) cudaEventDestroy(c->marks[r][i]);
  cudaSetDevice(prev);
  delete c;
  return DEFL_OK;
}

int defl_set_stream(defl_ctx* c, void* s) {
  if (!c) return DEFL_ERR_ARG;
  c->stream = reinterpret_cast<cudaStream_t>(s);
  return DEFL_OK;
}

size_t defl_polar_workspace_bytes(int b, int m, int n, int dtype, int k, int oversample) {
  if (b <= 0 || m <= 0 || n <= 0 || k < 0 || oversample < 0) return 0;
  const int ms = m < n ? m : n;
  int l = k > 0 ? k + oversample : 0;
  if (l > ms) l = ms;
  return carve_polar(nullptr, b, m, n, dtype, k, l).bytes;
}

int defl_set_profiling(defl_ctx* c, int enabled) {
  if (!c) return DEFL_ERR_ARG;
  if (enabled && !c->marks_ready) {
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(c->device);
    bool ok = true;
    for (int r = 0; ok && r < DEFL_PROFILE_CALLS; ++r)
      for (int i = 0; ok && i < DEFL_MAX_MARKS; ++i) ok = cudaEventCreate(&c->marks[r][i]) == cudaSuccess;
    cudaSetDevice(prev);
    if (!ok) { ctx_fail(c, cudaErrorUnknown, "events for stage timing"); return DEFL_ERR_CUDA; }
    c->marks_ready = true;
  }
  c->profiling = enabled != 0;
  return DEFL_OK;
}

int defl_get_stage_ms_sum(defl_ctx* c, float* ms, int cap, int ncalls) {
  if (!c || !ms || ncalls < 1) return DEFL_ERR_ARG;
  if (!c->marks_ready || c->call_seq == 0) return 0;
  if (ncalls > DEFL_PROFILE_CALLS) ncalls = DEFL_PROFILE_CALLS;
  if ((long long)ncalls > c->call_seq) ncalls = (int)c->call_seq;
  cudaStreamSynchronize(c->stream);
  int n = 0;
  for (int i = 0; i < cap; ++i) ms[i] = 0.f;
  for (int q = 0; q < ncalls; ++q) {
    const int slot = (int)((c->call_seq - q) % DEFL_PROFILE_CALLS);
    const int ns = c->n_marks[slot] - 1;
    if (ns > n) n = ns;
    for (int i = 0; i < ns && i < cap; ++i) {
      float t = 0.f;
      cudaEventElapsedTime(&t, c->marks[slot][i], c->marks[slot][i + 1]);
      ms[i] += t;
    }
  }
  return n < 0 ? 0 : n;
}

int defl_get_stage_ms(defl_ctx* c, float* ms, int cap) { return defl_get_stage_ms_sum(c, ms, cap, 1); }

long long defl_launch_count(defl_ctx* c) { return c ? c->launches : 0; }

int defl_device_wait_status(defl_ctx* c, int clear) {
  if (!c) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  int word = 0;
  if (ctx_fail(c, cudaStreamSynchronize(c->stream), "synchronize") ||
      ctx_fail(c, cudaMemcpy(&word, c->wait_status, sizeof(int), cudaMemcpyDeviceToHost), "read status word"))
    return DEFL_ERR_CUDA;
  if (clear && word && ctx_fail(c, cudaMemset(c->wait_status, 0, sizeof(int)), "clear status word")) return DEFL_ERR_CUDA;
  return word;
}

// Window sizes from the paper's ratios (host arithmetic only).
// (a ratio arrives as a float: 0.025f * 640 is 16.0000002, which must count as 16, so the product is taken two parts
// in a million short before it is rounded up)
static int ceil_ratio(float ratio, int dim) {
  const double v = (double)ratio * (double)dim * (1.0 - 2e-6);
  int c = (int)v;
  if ((double)c < v) ++c;
  return c;
}

int defl_polar_window(int m, int n, float w, float delta, int* k, int* oversample) {
  if (m <= 0 || n <= 0 || !(w >= 0.f) || !(delta >= 0.f) || !k || !oversample) return DEFL_ERR_ARG;
  const int ms = m < n ? m : n;
  int r = ceil_ratio(w, ms);
  if (r >= ms) r = ms - 1;                       // at least one component stays in the residual
  int rp = r + ceil_ratio(delta, ms);
  if (rp > ms) rp = ms;
  *k = r;
  *oversample = rp - r;
  return rp > DEFL_MAX_L ? DEFL_ERR_RANK : DEFL_OK;
}

int defl_psd_window(int n, float w, float w_prime, int* k, int* K) {
  if (n <= 0 || !(w >= 0.f) || !(w_prime >= 0.f) || !k || !K) return DEFL_ERR_ARG;
  int r = ceil_ratio(w, n), kk = ceil_ratio(w_prime, n);
  if (kk > n) kk = n;
  if (r > kk) r = kk;
  *k = r;
  *K = kk;
  return kk > DEFL_MAX_L ? DEFL_ERR_RANK : DEFL_OK;
}

const char* defl_status_string(int code) {
  switch (code) {
    case DEFL_OK: return "ok";
    case DEFL_ERR_ARG: return "bad argument (null pointer, non-positive size, overlap or bad enum)";
    case DEFL_ERR_RANK: return "rank/width out of range (need k < min(m,n), k+oversample <= 64, depth <= 32)";
    case DEFL_ERR_CUDA: return "CUDA runtime failure (see defl_last_error)";
    case DEFL_ERR_UNSUPPORTED: return "requested engine cannot run this shape or type";
    default: return "unknown status";
  }
}

const char* defl_last_error(defl_ctx* c) { return c ? c->err : ""; }

int defl_fill_gaussian(defl_ctx* c, void* dst, size_t count, int dtype, uint64_t seed) {
  if (!c || !dst || (dtype != DEFL_BF16 && dtype != DEFL_F32)) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  if (ctx_fail(c, fill_gaussian_launch(dst, (long long)count, dtype, seed, 0, 0ull, c->stream, &c->launches), "fill"))
    return DEFL_ERR_CUDA;
  return DEFL_OK;
}

int defl_debug_gemm(defl_ctx* c, int engine, int batch, int M, int N, int K, const void* A, long long sa_i,
                    long long sa_k, long long batch_a, const void* B, long long sb_k, long long sb_j, long long batch_b,
                    void* C, int in_dtype, int out_dtype, float alpha, int exploit_symmetry) {
  if (!c || !A || !B || !C || batch <= 0 || M <= 0 || N <= 0 || K <= 0) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  GemmDesc g = gemm_desc_zero();
  g.batch = batch; g.M = M; g.N = N; g.K[0] = K;
  g.A[0] = A; g.sa_i[0] = sa_i; g.sa_k[0] = sa_k; g.batch_a[0] = batch_a;
  g.B[0] = B; g.sb_k[0] = sb_k; g.sb_j[0] = sb_j; g.batch_b[0] = batch_b;
  g.in_dtype = in_dtype; g.b_dtype = in_dtype;
  g.C = C; g.ldc = N; g.batch_c = (long long)M * N; g.out_dtype = out_dtype;
  g.epilogue = EPI_STORE; g.alpha = alpha; g.symmetric = (exploit_symmetry & 1) ? 1 : 0;
  if (exploit_symmetry & 2) { g.transpose_out = 1; g.ldc = M; }
  if (exploit_symmetry & 4) g.debug_hold_stage = 1;
  return run_gemm(c, g, engine, "debug gemm");
}

int defl_brsvd_batched(defl_ctx* c, const void* G, int b, int m, int n, int dtype, int k, int oversample,
                       int power_iters, float* P, float* s, float* W, const defl_opts* opts, int* status) {
  if (!c || !G || b <= 0 || m <= 0 || n <= 0 || k <= 0 || oversample < 0 || power_iters < 0) return DEFL_ERR_ARG;
  if (dtype != DEFL_BF16 && dtype != DEFL_F32) return DEFL_ERR_ARG;
  const bool tall = m >= n;
  const int ms = tall ? n : m, ml = tall ? m : n;
  int l = k + oversample;
  if (l > ms) l = ms;
  if (l > DEFL_MAX_L) return DEFL_ERR_RANK;
  cudaSetDevice(c->device);
  const size_t need = carve_polar(nullptr, b, m, n, dtype, l, l).bytes;
  int rc = ctx_reserve(c, need);
  if (rc) return rc;
  PolarWs w = carve_polar(c->ws, b, m, n, dtype, l, l);
  const int engine = opts ? opts->engine : DEFL_ENGINE_AUTO;
  if (ctx_fail(c, fill_int_launch(w.status, b, 0, c->stream, &c->launches), "status")) return DEFL_ERR_CUDA;
  const float* sk = resolve_sketch(c, opts, b, ms, l, w, &rc);
  if (rc) return rc;
  if ((rc = run_brsvd(c, G, b, m, n, dtype, l, power_iters, l, sk, w, engine))) return rc;
  // tall: G = U S V^T with U on m rows; wide: A = G^T so the left factor of G is V
  const float* left = tall ? w.Uk : w.Vk;
  const float* right = tall ? w.Vk : w.Uk;
  if (P && ctx_fail(c, cudaMemcpyAsync(P, left, (size_t)b * m * l * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy P"))
    return DEFL_ERR_CUDA;
  if (W && ctx_fail(c, cudaMemcpyAsync(W, right, (size_t)b * n * l * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy W"))
    return DEFL_ERR_CUDA;
  if (s && ctx_fail(c, cudaMemcpyAsync(s, w.sv, (size_t)b * l * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy s"))
    return DEFL_ERR_CUDA;
  if (status && ctx_fail(c, cudaMemcpyAsync(status, w.status, (size_t)b * sizeof(int), cudaMemcpyDeviceToDevice, c->stream), "copy status"))
    return DEFL_ERR_CUDA;
  (void)ml;
  return DEFL_OK;
}

// Weight update fused into the last product of the chain: W <- keep * W + step * (result of Algorithm 1)
struct WeightUpdate {
  void* W;
  int w_dtype;
  float keep, step;
};

static int polar_core(defl_ctx* c, const void* G, void* out, int b, int m, int n, int dtype, int k, int oversample,
                      int power_iters, const float* coeff_schedule, int L, const defl_opts* opts,
                      const defl_info* info, const WeightUpdate* upd) {
  if (!c || !G || !out || b <= 0 || m <= 0 || n <= 0 || k < 0 || oversample < 0 || power_iters < 0 || L < 0)
    return DEFL_ERR_ARG;
  if (dtype != DEFL_BF16 && dtype != DEFL_F32) return DEFL_ERR_ARG;
  if (L > 0 && !coeff_schedule) return DEFL_ERR_ARG;
  if (upd && (L < 1 || !upd->W)) return DEFL_ERR_ARG;      // the update rides on the last filter product
  const size_t es = dtype_size(dtype);
  const size_t gbytes = (size_t)b * m * n * es;
  {
    const char* g0 = reinterpret_cast<const char*>(G);
    const char* o0 = reinterpret_cast<const char*>(out);
    if (g0 < o0 + gbytes && o0 < g0 + gbytes) return DEFL_ERR_ARG;
  }
  const bool tall = m >= n;     // tall: Gram on the n side, X <- X B; otherwise Gram on the m side, X <- B X
  const bool wide = m <= n;
  const int ms = m < n ? m : n, ml = m < n ? n : m;
  int l = k > 0 ? k + oversample : 0;
  if (l > ms) l = ms;
  if (k >= ms || l > DEFL_MAX_L || L > DEFL_MAX_STEPS) return DEFL_ERR_RANK;
  const int engine = opts ? opts->engine : DEFL_ENGINE_AUTO;
  const int mode = opts ? opts->restore_mode : DEFL_RESTORE_PADDED;
  if (mode != DEFL_RESTORE_PADDED && mode != DEFL_RESTORE_ADD) return DEFL_ERR_ARG;
  if (engine < 0 || engine > 2) return DEFL_ERR_ARG;
  const float gamma = (opts && opts->gamma > 0.f) ? opts->gamma : 1.01f;
  const int sym = (opts && opts->exploit_symmetry) ? 1 : 0;
  const float tau = opts ? opts->tau : 0.f;
  // Iterate type of the filter. bf16 inputs: X_t, A_t, B_t are kept in IEEE half, scaled by 32 (Y = 32 X, so
  // A' = Y Y^T = 1024 A and the step's coefficients become a, b/2^10, c/2^20; the last product scales back by 1/32).
  // Same tensor-core rate as bf16, three more mantissa bits: the rounding of the stored iterate is what limits
  // the bf16 path's accuracy on wide matrices with slowly decaying spectra. The power-of-two scale keeps small
  // entries (1/sqrt(mn) of a normalised residual, off-diagonal Gram entries) out of half's subnormal range, and
  // overflow would need a singular value above 8.
  // How many steps need it: the rounding of X_0 and of the first iterates is what costs accuracy (the small
  // singular values are still small there). Measured on the 48 x 1600 x 6400 workload against the oracle: half in
  // all five steps 5.5e-3, in the first four 6.5e-3, three 8.1e-3, two 1.07e-2, one 1.5e-2, none (bf16 throughout)
  // 4.2e-2. Half-precision products draw more power than bf16 ones, and under the board's power cap that is clock:
  // 23.3 ms per step with five half steps, 22.6 ms with two or one, 21.9 ms with none. Default: the first two
  // steps in half, the rest in bf16. opts->bf16_iterates = 1: bf16 throughout; = 2: half throughout.
  // ADD restore keeps half in every step: without the head inside X_0 all its singular values are small and stay
  // small for longer, and the same storage rounding costs about ten times more (a 636 x 75 case with six steps:
  // 2.8e-2 with half throughout, 8.2e-2 with two half steps, 1.7e-1 with bf16; padded restore 2.7e-3 / 9.8e-3 / 1.7e-2).
  int terms = (opts && opts->poly_terms) ? opts->poly_terms : 3;
  if (terms < 2 || terms > DEFL_MAX_TERMS) return DEFL_ERR_ARG;
  // a cubic is the quintic with a zero last coefficient
  float cubic_as_quintic[3 * DEFL_MAX_STEPS];
  if (terms == 2) {
    for (int t = 0; t < L; ++t) { cubic_as_quintic[3 * t] = coeff_schedule[2 * t]; cubic_as_quintic[3 * t + 1] = coeff_schedule[2 * t + 1]; cubic_as_quintic[3 * t + 2] = 0.f; }
    coeff_schedule = cubic_as_quintic;
    terms = 3;
  }
  const int it_mode = opts ? opts->bf16_iterates : 0;
  const bool half_iter = dtype == DEFL_BF16 && L > 0 && it_mode != 1;
  // the first `n_half` filter steps keep the iterate in scaled IEEE half, the rest in bf16
  // Paired steps (two filter steps per pass over X, both in scaled half: see the filter stage) on the tensor engine's
  // bf16 path when the shape pays for them; every step but an odd last one is then kept in half
  const bool pair_ok = c->knobs.paired_steps && half_iter && terms == 3 && engine != DEFL_ENGINE_SIMT &&
                       paired_steps_shape(m, n, dtype);
  // A pair starts at step t when a next step exists and two gains are moderate. The short-side step multiplies the
  // rounding of the stored A_t by about a_t^2 in the directions of small singular values (12 for Muon's quintic, 70 for
  // the steep first step of a per-step minimax schedule, which therefore stays a step of its own): |a_t| <= 4.5. And the
  // next polynomial is evaluated on an A_{t+1} that was not recomputed from the iterate, so its rounding reaches
  // B_{t+1} with the gain |b_{t+1} + 2 c_{t+1}| at the top of the spectrum (0.7 for Muon's quintic, 0.5 for the
  // classical one, 1.5-2 for the middle steps of a minimax schedule, where a pair left single singular values 0.1
  // off): <= 1. The walk is greedy from the first step.
  auto pair_starts = [&](int t) {
    if (!pair_ok || t + 1 >= L) return false;
    const float* c0 = coeff_schedule + (size_t)terms * t;
    const float* c1 = c0 + terms;
    return fabsf(c0[0]) <= 4.5f && fabsf(c1[1] + 2.f * c1[2]) <= 1.0f;
  };
  int n_half_rule = half_iter ? ((it_mode == 2 || mode == DEFL_RESTORE_ADD) ? L : (L < 2 ? L : 2)) : 0;
  int npass = 0;
  for (int t = 0; t < L; ++npass) {
    if (pair_starts(t)) { t += 2; if (t > n_half_rule) n_half_rule = t; }       // both steps of a pair in scaled half
    else t += 1;
  }
  const int n_half = n_half_rule;
  const int it_dtype = n_half > 0 ? (int)F16 : dtype;      // format and scale of X_0
  const float ys = n_half > 0 ? 32.f : 1.f;

  cudaSetDevice(c->device);
  int rc = ctx_reserve(c, carve_polar(nullptr, b, m, n, dtype, k, l, terms).bytes);
  if (rc) return rc;
  PolarWs w = carve_polar(c->ws, b, m, n, dtype, k, l, terms);
  ctx_profile_begin(c);
  c->err[0] = 0;
  ctx_stage_mark(c);
  if (ctx_fail(c, fill_int_launch(w.status, b, 0, c->stream, &c->launches), "status")) return DEFL_ERR_CUDA;
  // the engine's wait word reports this call only (the tile counter next to it stays as the kernels leave it: zero)
  if (ctx_fail(c, cudaMemsetAsync(c->wait_status, 0, sizeof(int), c->stream), "status word")) return DEFL_ERR_CUDA;

  // ---- stage 0: Algorithm 3 ------------------------------------------------------------------
  if (k > 0) {
    const float* sk = resolve_sketch(c, opts, b, ms, l, w, &rc);
    if (rc) return rc;
    if ((rc = run_brsvd(c, G, b, m, n, dtype, l, power_iters, k, sk, w, engine))) return rc;
  }
  ctx_stage_mark(c);

  // iterate buffers: the chain must end in `out`
  void* bufs[2] = {w.X, out};
  // X0 goes to bufs[cur]; every pass over X swaps the buffers, and the last one must write `out` (a paired step is one
  // pass for two filter steps)
  int cur = (npass % 2 == 0) ? 1 : 0;

  // ---- stage 1: R = G - P diag(s) W^T, rho = ||R||_F, X0 = R/rho (+ P W^T / gamma) ----------------
  const float* left = tall ? w.Uk : w.Vk;     // [b,m,k]
  const float* right = tall ? w.Vk : w.Uk;    // [b,n,k]
  const int kp = round_up8(k > 0 ? k : 1);
  if (k > 0) {
    // R = G - P diag(s) W^T as a rank-k product on the product engine with G read in the epilogue.
    // bf16 storage: the fp32 factors are split into bf16 hi + lo and the three significant cross terms are
    // laid side by side along K, [hi|hi|lo] x [hi|lo|hi]^T, one tensor-core product of depth 3k.
    // gate (Algorithm 1, lines 1-2): per matrix, how many of the k triplets are deflated; the columns beyond
    // that count are zeroed in the scaled right factor, which removes them from every product below
    if (ctx_fail(c, gate_launch(w.sv, l, b, k, k, tau, w.keff, c->stream, &c->launches), "gate")) return DEFL_ERR_CUDA;
    GemmDesc g = gemm_desc_zero();
    g.batch = b; g.M = m; g.N = n;
    g.aux = G; g.ld_aux = n; g.batch_aux = (long long)m * n; g.aux_dtype = dtype;
    bool tensor_defl = false;
    if (dtype == BF16 && engine != DEFL_ENGINE_SIMT) {
      g.K[0] = 3 * kp;
      g.A[0] = w.Pc; g.sa_i[0] = 3 * kp; g.sa_k[0] = 1; g.batch_a[0] = (long long)m * 3 * kp; g.in_dtype = BF16;
      g.B[0] = w.Wc; g.sb_k[0] = 1; g.sb_j[0] = 3 * kp; g.batch_b[0] = (long long)n * 3 * kp; g.b_dtype = BF16;
      tensor_defl = gemm_tc_supported(g);
    }
    const int deng = tensor_defl ? DEFL_ENGINE_TENSOR : DEFL_ENGINE_SIMT;
    if (tensor_defl) {
      if (ctx_fail(c, split_concat3_launch(left, (long long)m * k, k, b, m, k, kp, nullptr, 0, nullptr, 0.f, 0.f, 0, w.Pc,
                                           c->stream, &c->launches), "split P"))
        return DEFL_ERR_CUDA;
      // The triplets come from U = Q E and Q^T A = E diag(s) V^T (Algorithm 3, lines 7-9), so the residual's norm
      // needs no pass over R:  ||A - U_k diag(s) V_k^T||_F^2 = ||A||_F^2 - sum_{i<=k} s_i^2  for ANY orthonormal Q
      // (expand the square: the cross term is 2 tr(E_k^T Q^T A A^T Q E_k) = 2 sum s_i^2). ||G||_F^2 is one streaming
      // read of G in fixed-order fp64 partial sums; with the gate only the deflated columns are subtracted. The
      // difference is formed in fp64 from fp32 s_i: a residual below 1e-3 ||G||_F is not resolved and counts as zero.
      if (ctx_fail(c, frob_partial_vec_launch(G, dtype, b, (long long)m * n, FROB_VEC_BLOCKS, w.npart, c->stream, &c->launches), "frobenius"))
        return DEFL_ERR_CUDA;
      if (ctx_fail(c, rho_identity_launch(w.npart, FROB_VEC_BLOCKS, b, w.sv, l, w.keff, w.rho, w.inv_rho, w.inv_rho2, w.status,
                                          c->stream, &c->launches), "rho"))
        return DEFL_ERR_CUDA;
    } else {
      // fp32 products (fp32 storage, or shapes the tensor engine cannot take): the residual is formed and its squares
      // summed in the epilogue of a first pass, nothing stored
      if (ctx_fail(c, scale_cols_launch(right, (long long)n * k, k, b, n, k, w.sv, l, nullptr, 1.f, 0.f, w.Ws,
                                        (long long)n * k, k, c->stream, &c->launches, w.keff), "W diag(s)"))
        return DEFL_ERR_CUDA;
      g.K[0] = k;
      g.A[0] = left; g.sa_i[0] = k; g.sa_k[0] = 1; g.batch_a[0] = (long long)m * k; g.in_dtype = F32;
      g.B[0] = w.Ws; g.sb_k[0] = 1; g.sb_j[0] = k; g.batch_b[0] = (long long)n * k; g.b_dtype = F32;
      g.epilogue = EPI_RESID_NORM; g.partials = w.npart;
      g.partials_per_batch = partials_per_batch(c, g, deng);
      if ((rc = run_gemm(c, g, deng, "residual norm"))) return rc;
      if (ctx_fail(c, rho_finalize_launch(w.npart, g.partials_per_batch, b, w.rho, w.inv_rho, w.inv_rho2, w.status,
                                          c->stream, &c->launches), "rho"))
        return DEFL_ERR_CUDA;
    }
    // X0 = G/rho - P diag(s/rho - pad) W^T: pad = 1/gamma puts the head into X0 (Algorithm 1); with ADD restore the
    // head stays out (pad = 0) and joins the last filter product, or, when there is no filter step to carry it,
    // goes in at full weight (X0 + P W^T is the padded entry with gamma = 1)
    const float pad = (mode == DEFL_RESTORE_PADDED) ? 1.f / gamma : (L == 0 ? 1.f : 0.f);
    // Tensor engine, second form: X0 = (1/rho) [G - P diag(s - pad rho) W^T] with G itself added in the accumulator
    // (a second K segment: the tile's own columns of G against an identity tile, exact in bf16 x bf16 -> fp32), so
    // that the epilogue is the plain coalesced store scaled by the per-matrix 1/rho. Reading G element-wise in the
    // epilogue instead (the first form, kept for shapes whose rows the copy engine cannot address) is bound by
    // the epilogue warps' instruction issue, at a quarter of the memory bandwidth.
    bool ident_form = false;
    GemmDesc gi = g;
    if (tensor_defl) {
      gi.nseg = 2; gi.seg1_identity = 1;
      gi.A[1] = G; gi.sa_i[1] = n; gi.sa_k[1] = 1; gi.batch_a[1] = (long long)m * n;
      gi.B[1] = c->ident_bf16; gi.sb_k[1] = 1; gi.sb_j[1] = 256; gi.batch_b[1] = 0; gi.K[1] = 256;
      gi.aux = nullptr; gi.epilogue = EPI_STORE; gi.partials = nullptr;
      ident_form = gemm_tc_supported(gi);
    }
    if (ident_form) {
      if (ctx_fail(c, split_concat3_launch(right, (long long)n * k, k, b, n, k, kp, w.sv, l, nullptr, -1.f, pad, 1, w.Wc,
                                           c->stream, &c->launches, w.keff, 0, 0, 1.f, w.rho), "split W diag(coef)"))
        return DEFL_ERR_CUDA;
      gi.alpha = ys; gi.alpha_dev = w.inv_rho;
      gi.C = bufs[cur]; gi.ldc = n; gi.batch_c = (long long)m * n; gi.out_dtype = it_dtype;
      if ((rc = run_gemm(c, gi, DEFL_ENGINE_TENSOR, "deflate+normalise"))) return rc;
      // (a matrix whose residual counts as zero has 1/rho = 0 and came out as zeros: it gets the padded head alone)
      if (ctx_fail(c, zero_residual_entry_launch(w.status, left, right, w.keff, b, m, n, k, ys * pad, bufs[cur], it_dtype, c->stream,
                                                 &c->launches), "zero-residual entry"))
        return DEFL_ERR_CUDA;
    } else {
      if (tensor_defl) {
        if (ctx_fail(c, split_concat3_launch(right, (long long)n * k, k, b, n, k, kp, w.sv, l, w.inv_rho, -1.f, pad, 1, w.Wc,
                                             c->stream, &c->launches, w.keff), "split W diag(coef)"))
          return DEFL_ERR_CUDA;
      } else if (ctx_fail(c, scale_cols_launch(right, (long long)n * k, k, b, n, k, w.sv, l, w.inv_rho, -1.f, pad, w.Ws,
                                               (long long)n * k, k, c->stream, &c->launches, w.keff), "W diag(coef)")) {
        return DEFL_ERR_CUDA;
      }
      g.epilogue = EPI_AUX_PLUS; g.partials = nullptr;
      g.aux_scale = ys; g.aux_scale_dev = w.inv_rho; g.alpha = ys;
      g.C = bufs[cur]; g.ldc = n; g.batch_c = (long long)m * n; g.out_dtype = it_dtype;
      if ((rc = run_gemm(c, g, deng, "deflate+normalise"))) return rc;
    }
  } else {
    if (ctx_fail(c, frob_partial_vec_launch(G, dtype, b, (long long)m * n, FROB_VEC_BLOCKS, w.npart, c->stream, &c->launches), "frobenius"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, rho_finalize_launch(w.npart, FROB_VEC_BLOCKS, b, w.rho, w.inv_rho, w.inv_rho2, w.status, c->stream,
                                        &c->launches), "rho"))
      return DEFL_ERR_CUDA;
    if (ctx_fail(c, scale_launch(G, dtype, bufs[cur], it_dtype, b, (long long)m * n, w.inv_rho, c->stream, &c->launches, 0, ys), "normalise"))
      return DEFL_ERR_CUDA;
  }
  ctx_stage_mark(c);

  // ---- restore (Eq. 3) with ADD mode: out = N^L(X0) + P W^T rides on the LAST filter product as a second K segment
  // (depth k, or 3k for the split 16-bit copies), so the head is added in the accumulator and `out` makes no further
  // trip through memory. The factors are prepared here: in the type and scale of the last step's operands
  // (16-bit iterates: [hi|hi|lo] x [hi|lo|hi] copies, IEEE half or bf16, their product scaled like the iterate;
  // fp32: the factors themselves), the right one gated and laid out like the operand it accompanies.
  const bool fuse_restore = k > 0 && mode == DEFL_RESTORE_ADD && L > 0;
  const bool last_half = L > 0 && (L - 1) < n_half;            // the last step's operands are scaled IEEE half
  if (fuse_restore) {
    if (dtype == BF16) {
      const float ysl = last_half ? 32.f : 1.f;
      const float mp = last_half ? 8.f : 1.f;                  // powers of two: P W^T * ysl = (mp P)(ysl / mp W)^T exactly
      if (ctx_fail(c, split_concat3_launch(left, (long long)m * k, k, b, m, k, kp, nullptr, 0, nullptr, 0.f, 0.f, 0, w.Pc,
                                           c->stream, &c->launches, nullptr, last_half ? 1 : 0, 0, mp), "split P (restore)"))
        return DEFL_ERR_CUDA;
      if (ctx_fail(c, split_concat3_launch(right, (long long)n * k, k, b, n, k, kp, nullptr, 0, nullptr, 0.f, 0.f, 1, w.Wc,
                                           c->stream, &c->launches, w.keff, last_half ? 1 : 0, wide ? 1 : 0, ysl / mp),
                   "split W (restore)"))
        return DEFL_ERR_CUDA;
    } else if (ctx_fail(c, scale_cols_launch(right, (long long)n * k, k, b, n, k, w.sv, l, nullptr, 0.f, 1.f, w.Ws,
                                             (long long)n * k, k, c->stream, &c->launches, w.keff), "W (gated)")) {
      return DEFL_ERR_CUDA;
    }
  }
  // second K segment of the last apply product; `transposed_form`: the product is computed as its transpose
  auto add_restore_segment = [&](GemmDesc& q, bool transposed_form) {
    q.nseg = 2;
    if (dtype == BF16) {
      q.K[1] = 3 * kp;
      const void* Pr = w.Pc;      // [b, m, 3kp]
      const void* Wr = w.Wc;      // [b, 3kp, n] for a wide matrix, else [b, n, 3kp]
      if (!transposed_form) {
        q.A[1] = Pr; q.sa_i[1] = 3 * kp; q.sa_k[1] = 1; q.batch_a[1] = (long long)m * 3 * kp;
        q.B[1] = Wr; q.batch_b[1] = (long long)n * 3 * kp;
        if (wide) { q.sb_k[1] = n; q.sb_j[1] = 1; } else { q.sb_k[1] = 1; q.sb_j[1] = 3 * kp; }
      } else {
        q.A[1] = Wr; q.sa_i[1] = 1; q.sa_k[1] = n; q.batch_a[1] = (long long)n * 3 * kp;
        q.B[1] = Pr; q.sb_k[1] = 1; q.sb_j[1] = 3 * kp; q.batch_b[1] = (long long)m * 3 * kp;
      }
    } else {
      q.K[1] = k;
      q.A[1] = left; q.sa_i[1] = k; q.sa_k[1] = 1; q.batch_a[1] = (long long)m * k;
      q.B[1] = w.Ws; q.sb_k[1] = 1; q.sb_j[1] = k; q.batch_b[1] = (long long)n * k;
    }
  };

  // ---- stage 2: X <- a X + b (X X^T) X + c (X X^T)^2 X, L times, through the short-side Gram -------
  // Paired steps. X_{t+2} = B_{t+1} B_t X_t, and the Gram matrix of the step in between needs no pass over X:
  // A_{t+1} = X_{t+1} X_{t+1}^T = B_t A_t B_t = B_t^2 A_t (B_t is a polynomial in A_t). A pair costs one Gram product and
  // one apply product of ms^2 ml each plus five ms^3 products (A_t^2 in B_t, B_t^2, B_t^2 A_t, A_{t+1}^2 in B_{t+1},
  // B_{t+1} B_t) where two single steps cost two of each big product and two small ones. Only ONE step is taken on the
  // short side at a time, and only with the 11-bit storage: every further one would multiply the rounding of the
  // stored A by a^2 (about 12), which the small singular values do not survive.
  for (int t = 0; t < L;) {
    const bool paired = pair_starts(t);                              // (both steps are then in scaled half)
    const int tl = paired ? t + 1 : t;                               // the last step this pass over X covers
    const float* cf = coeff_schedule + (size_t)terms * t;       // a_0 .. a_{terms-1} of this step
    const void* X = bufs[cur];
    void* Xn = bufs[cur ^ 1];
    const bool hs = t < n_half, hn = tl + 1 < n_half;
    const int it_dtype = hs ? (int)F16 : dtype, nx_dtype = hn ? (int)F16 : dtype;     // this step's and the next one's
    const float ys = hs ? 32.f : 1.f, ys_next = hn ? 32.f : 1.f;
    GemmDesc g = gemm_desc_zero();
    g.batch = b; g.in_dtype = it_dtype; g.b_dtype = it_dtype; g.out_dtype = it_dtype;
    // A_t = X X^T (wide) or X^T X (tall), ms x ms, symmetric
    g.M = ms; g.N = ms; g.K[0] = ml;
    g.A[0] = X; g.B[0] = X; g.batch_a[0] = g.batch_b[0] = (long long)m * n;
    if (wide) { g.sa_i[0] = n; g.sa_k[0] = 1; g.sb_k[0] = 1; g.sb_j[0] = n; }
    else { g.sa_i[0] = 1; g.sa_k[0] = n; g.sb_k[0] = n; g.sb_j[0] = 1; }
    g.C = w.Am; g.ldc = ms; g.batch_c = (long long)ms * ms;
    g.epilogue = EPI_STORE; g.symmetric = sym;
    if ((rc = run_gemm(c, g, engine, "gram"))) return rc;
    // B_t = a_0 I + a_1 A_t + ... + a_d A_t^d by Horner steps. The innermost one forms a_{d-2} I + a_{d-1} A_t +
    // a_d A_t A_t in the epilogue of one product (the whole polynomial for the quintic); every further degree costs one
    // more product C <- a_j I + A_t C. With scaled iterates the stored Gram matrix is ys^2 A_t: the coefficients absorb
    // the powers, the intermediate polynomials are kept unscaled.
    const int nprod = terms - 2;
    const float iy2 = 1.f / (ys * ys);
    for (int q = 0; q < nprod; ++q) {
      void* dst = ((nprod - 1 - q) % 2 == 0) ? w.Bm : w.Cm;        // the last product lands in B_t
      const void* prev = (dst == w.Bm) ? w.Cm : w.Bm;
      g = gemm_desc_zero();
      g.batch = b; g.in_dtype = it_dtype; g.b_dtype = it_dtype; g.out_dtype = it_dtype;
      g.M = ms; g.N = ms; g.K[0] = ms;
      g.A[0] = w.Am; g.sa_i[0] = ms; g.sa_k[0] = 1; g.batch_a[0] = (long long)ms * ms;
      g.B[0] = (q == 0) ? w.Am : prev; g.sb_k[0] = 1; g.sb_j[0] = ms; g.batch_b[0] = (long long)ms * ms;   // symmetric: rows as columns
      g.C = dst; g.ldc = ms; g.batch_c = (long long)ms * ms;
      g.aux = w.Am; g.ld_aux = ms; g.batch_aux = (long long)ms * ms; g.aux_dtype = it_dtype;
      g.epilogue = EPI_POLY; g.symmetric = sym;
      if (q == 0) { g.pa = cf[terms - 3]; g.pb = cf[terms - 2] * iy2; g.pc = cf[terms - 1] * iy2 * iy2; }
      else { g.pa = cf[terms - 3 - q]; g.pb = 0.f; g.pc = iy2; }
      if ((rc = run_gemm(c, g, engine, "polynomial"))) return rc;
    }
    const void* Bap = w.Bm;          // what multiplies X: B_t, or B_{t+1} B_t
    if (paired) {
      const float* cf1 = coeff_schedule + (size_t)terms * (t + 1);
      auto small_product = [&](const void* L_, const void* R_, void* C_, const char* what) {
        GemmDesc q = gemm_desc_zero();
        q.batch = b; q.in_dtype = it_dtype; q.b_dtype = it_dtype; q.out_dtype = it_dtype;
        q.M = ms; q.N = ms; q.K[0] = ms;
        q.A[0] = L_; q.sa_i[0] = ms; q.sa_k[0] = 1; q.batch_a[0] = (long long)ms * ms;
        q.B[0] = R_; q.sb_k[0] = 1; q.sb_j[0] = ms; q.batch_b[0] = (long long)ms * ms;      // symmetric: rows as columns
        q.C = C_; q.ldc = ms; q.batch_c = (long long)ms * ms;
        q.epilogue = EPI_STORE; q.symmetric = sym;
        return run_gemm(c, q, engine, what);
      };
      if ((rc = small_product(w.Bm, w.Bm, w.Cm, "B^2"))) return rc;
      if ((rc = small_product(w.Cm, w.Am, w.Dm, "B^2 A"))) return rc;          // ys^2 A_{t+1}: the stored scale carries over
      g = gemm_desc_zero();
      g.batch = b; g.in_dtype = it_dtype; g.b_dtype = it_dtype; g.out_dtype = it_dtype;
      g.M = ms; g.N = ms; g.K[0] = ms;
      g.A[0] = w.Dm; g.sa_i[0] = ms; g.sa_k[0] = 1; g.batch_a[0] = (long long)ms * ms;
      g.B[0] = w.Dm; g.sb_k[0] = 1; g.sb_j[0] = ms; g.batch_b[0] = (long long)ms * ms;
      g.C = w.Am; g.ldc = ms; g.batch_c = (long long)ms * ms;                   // A_t is no longer needed
      g.aux = w.Dm; g.ld_aux = ms; g.batch_aux = (long long)ms * ms; g.aux_dtype = it_dtype;
      g.epilogue = EPI_POLY; g.symmetric = sym;
      g.pa = cf1[0]; g.pb = cf1[1] * iy2; g.pc = cf1[2] * iy2 * iy2;
      if ((rc = run_gemm(c, g, engine, "polynomial (second step)"))) return rc;
      if ((rc = small_product(w.Am, w.Bm, w.Cm, "B' B"))) return rc;
      Bap = w.Cm;
    }
    // X <- B_t X (wide) or X B_t (tall)
    g = gemm_desc_zero();
    g.batch = b; g.in_dtype = it_dtype; g.b_dtype = it_dtype; g.out_dtype = it_dtype;
    g.M = m; g.N = n;
    if (wide) {
      g.K[0] = m;
      g.A[0] = Bap; g.sa_i[0] = m; g.sa_k[0] = 1; g.batch_a[0] = (long long)m * m;
      g.B[0] = X; g.sb_k[0] = n; g.sb_j[0] = 1; g.batch_b[0] = (long long)m * n;
    } else {
      g.K[0] = n;
      g.A[0] = X; g.sa_i[0] = n; g.sa_k[0] = 1; g.batch_a[0] = (long long)m * n;
      g.B[0] = Bap; g.sb_k[0] = 1; g.sb_j[0] = n; g.batch_b[0] = (long long)n * n;   // B_t symmetric
    }
    g.C = Xn; g.ldc = n; g.batch_c = (long long)m * n;
    g.epilogue = EPI_STORE;
    g.out_dtype = nx_dtype; g.alpha = ys_next / ys;                   // the next step's format and scale
    if (tl == L - 1) { g.out_dtype = dtype; g.alpha = 1.f / ys; }      // the result leaves in the caller's type and scale
    const bool carry_head = fuse_restore && tl == L - 1;
    if (carry_head) add_restore_segment(g, false);
    if (wide && !(upd && tl == L - 1)) {
      // The tensor engine pads the product's rows to whole 256-row tiles, its columns only to 32: for a wide X
      // whose short side is not a multiple of 256 (1600 = 6.25 tiles) it is cheaper to compute (B X)^T = X^T B
      // (rows = the long side) and let the epilogue write the tile transposed, which is the same memory.
      GemmDesc gt = g;
      gt.M = n; gt.N = m;
      gt.A[0] = X; gt.sa_i[0] = 1; gt.sa_k[0] = n; gt.batch_a[0] = (long long)m * n;
      gt.B[0] = Bap; gt.sb_j[0] = m; gt.sb_k[0] = 1; gt.batch_b[0] = (long long)m * m;    // B_t symmetric
      if (carry_head) add_restore_segment(gt, true);
      gt.transpose_out = 1;
      const long long pad_rows = (long long)((m + 255) / 256) * 256 * ((n + 31) / 32 * 32);
      const long long pad_rows_t = (long long)((n + 255) / 256) * 256 * ((m + 31) / 32 * 32);
      if (m > 128 && pad_rows_t < pad_rows && use_tensor_engine(gt, engine) && c->knobs.transposed_apply) g = gt;
    }
    if (upd && tl == L - 1) {
      // last step of a Muon update: W <- keep W + step (B_L X [+ P W^T]) instead of storing the iterate
      g.C = upd->W; g.out_dtype = upd->w_dtype;
      g.aux = upd->W; g.ld_aux = n; g.batch_aux = (long long)m * n; g.aux_dtype = upd->w_dtype;
      g.epilogue = EPI_AUX_PLUS; g.alpha = upd->step / ys; g.aux_scale = upd->keep;
    }
    // (a forced tensor engine that cannot take the two-segment product, e.g. fp32 factors whose width is not a
    // multiple of four, runs this one product on the fp32 engine instead of failing)
    const int eng_apply = (carry_head && engine == DEFL_ENGINE_TENSOR && !use_tensor_engine(g, engine)) ? DEFL_ENGINE_SIMT : engine;
    if ((rc = run_gemm(c, g, eng_apply, "apply"))) return rc;
    cur ^= 1;
    t = tl + 1;
  }
  ctx_stage_mark(c);

  // (stage 3, the restore of Eq. 3, is part of the last filter product: see above)
  ctx_stage_mark(c);

  // a result that is not finite raises DEFL_ST_NONFINITE for its matrix
  if (ctx_fail(c, finite_probe_launch(upd ? upd->W : out, upd ? upd->w_dtype : dtype, b, (long long)m * n, w.status, c->stream,
                                      &c->launches), "finite probe"))
    return DEFL_ERR_CUDA;
  if (info) {
    if (info->s && l > 0 &&
        ctx_fail(c, cudaMemcpyAsync(info->s, w.sv, (size_t)b * l * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy s"))
      return DEFL_ERR_CUDA;
    if (info->rho &&
        ctx_fail(c, cudaMemcpyAsync(info->rho, w.rho, (size_t)b * sizeof(float), cudaMemcpyDeviceToDevice, c->stream), "copy rho"))
      return DEFL_ERR_CUDA;
    if (info->k_used) {
      if (k == 0 && ctx_fail(c, fill_int_launch(w.keff, b, 0, c->stream, &c->launches), "k_used")) return DEFL_ERR_CUDA;
      if (ctx_fail(c, cudaMemcpyAsync(info->k_used, w.keff, (size_t)b * sizeof(int), cudaMemcpyDeviceToDevice, c->stream), "copy k_used"))
        return DEFL_ERR_CUDA;
    }
    if (info->status) {
      // fold the engine's device-wait word into every matrix's status
      if (ctx_fail(c, or_status_launch(w.status, b, c->wait_status, c->stream, &c->launches), "status"))
        return DEFL_ERR_CUDA;
      if (ctx_fail(c, cudaMemcpyAsync(info->status, w.status, (size_t)b * sizeof(int), cudaMemcpyDeviceToDevice, c->stream), "copy status"))
        return DEFL_ERR_CUDA;
    }
  }
  return DEFL_OK;
}


int defl_polar_batched(defl_ctx* c, const void* G, void* out, int b, int m, int n, int dtype, int k, int oversample,
                       int power_iters, const float* coeff_schedule, int L, const defl_opts* opts,
                       const defl_info* info) {
  return polar_core(c, G, out, b, m, n, dtype, k, oversample, power_iters, coeff_schedule, L, opts, info, nullptr);
}

static int ensure_staging(defl_ctx* c, size_t bytes) {
  if (bytes <= c->stage_bytes) return DEFL_OK;
  cudaDeviceSynchronize();
  if (c->stage_in) cudaFree(c->stage_in);
  if (c->stage_out) cudaFree(c->stage_out);
  c->stage_in = c->stage_out = nullptr;
  c->stage_bytes = 0;
  if (ctx_fail(c, cudaMalloc(&c->stage_in, bytes), "cudaMalloc(staging)")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, cudaMalloc(&c->stage_out, bytes), "cudaMalloc(staging)")) return DEFL_ERR_CUDA;
  c->stage_bytes = bytes;
  return DEFL_OK;
}

int defl_muon_step_batched(defl_ctx* c, void* W, int w_dtype, void* Mom, const void* Grad, int b, int m, int n,
                           int dtype, float lr, float mu, int nesterov, float weight_decay, float scale, int k,
                           int oversample, int power_iters, const float* coeff_schedule, int L,
                           const defl_opts* opts, const defl_info* info) {
  if (!c || !W || !Mom || b <= 0 || m <= 0 || n <= 0) return DEFL_ERR_ARG;
  if ((dtype != DEFL_BF16 && dtype != DEFL_F32) || (w_dtype != DEFL_BF16 && w_dtype != DEFL_F32)) return DEFL_ERR_ARG;
  if (L < 1 || !coeff_schedule) return DEFL_ERR_ARG;
  if (nesterov && !Grad) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  const size_t count = (size_t)b * m * n;
  int rc = ensure_staging(c, count * dtype_size(dtype));
  if (rc) return rc;
  // momentum, then the matrix whose polar factor is taken: the stored momentum itself, or the Nesterov look-ahead
  const void* D = Mom;
  if (Grad) {
    void* look = nesterov ? c->stage_in : nullptr;
    if (ctx_fail(c, momentum_launch(Mom, Grad, look, dtype, (long long)count, mu, c->stream, &c->launches), "momentum"))
      return DEFL_ERR_CUDA;
    if (nesterov) D = look;
  }
  WeightUpdate upd;
  upd.W = W; upd.w_dtype = w_dtype; upd.keep = 1.f - lr * weight_decay; upd.step = -lr * scale;
  return polar_core(c, D, c->stage_out, b, m, n, dtype, k, oversample, power_iters, coeff_schedule, L, opts, info, &upd);
}

int defl_polar_batched_host(defl_ctx* c, const void* G_host, void* out_host, int b, int m, int n, int dtype, int k,
                            int oversample, int power_iters, const float* coeff_schedule, int L,
                            const defl_opts* opts) {
  if (!c || !G_host || !out_host || b <= 0 || m <= 0 || n <= 0) return DEFL_ERR_ARG;
  if (dtype != DEFL_BF16 && dtype != DEFL_F32) return DEFL_ERR_ARG;
  cudaSetDevice(c->device);
  const size_t bytes = (size_t)b * m * n * dtype_size(dtype);
  if (ensure_staging(c, bytes)) return DEFL_ERR_CUDA;
  // The batch is independent matrices: it goes through in chunks, the copy of chunk i+1 to the device and of
  // chunk i-1 back to the host running (on streams of their own) while chunk i is computed. Few chunks: the small
  // kernels of the range finder take about the same time for 12 matrices as for 48.
  int chunks = b >= 24 ? 3 : (b >= 8 ? 2 : 1);
  if (c->knobs.host_chunks >= 1) chunks = c->knobs.host_chunks;
  if (chunks > DEFL_HOST_MAX_CHUNKS) chunks = DEFL_HOST_MAX_CHUNKS;
  if (chunks > b) chunks = b;
  if (!c->copy_ready) {
    bool ok = cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < DEFL_HOST_MAX_CHUNKS; ++i)
      ok = cudaEventCreateWithFlags(&c->chunk_in[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&c->chunk_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { ctx_fail(c, cudaErrorUnknown, "streams for the host-buffer path"); return DEFL_ERR_CUDA; }
    c->copy_ready = 1;
  }
  const size_t per_matrix = (size_t)m * n * dtype_size(dtype);
  const int per = (b + chunks - 1) / chunks;
  const int ms = m < n ? m : n;
  int l = k > 0 ? k + oversample : 0;
  if (l > ms) l = ms;
  // the staging buffers may still be read by work the caller queued on the compute stream before this call
  if (ctx_fail(c, cudaEventRecord(c->chunk_done[0], c->stream), "record")) return DEFL_ERR_CUDA;
  if (ctx_fail(c, cudaStreamWaitEvent(c->copy_in, c->chunk_done[0], 0), "wait")) return DEFL_ERR_CUDA;
  for (int i = 0; i < chunks; ++i) {
    const int b0 = i * per, bc = (b - b0 < per) ? b - b0 : per;
    if (bc <= 0) { chunks = i; break; }
    const size_t off = (size_t)b0 * per_matrix;
    if (ctx_fail(c, cudaMemcpyAsync((char*)c->stage_in + off, (const char*)G_host + off, (size_t)bc * per_matrix,
                                    cudaMemcpyHostToDevice, c->copy_in), "H2D")) return DEFL_ERR_CUDA;
    if (ctx_fail(c, cudaEventRecord(c->chunk_in[i], c->copy_in), "record")) return DEFL_ERR_CUDA;
  }
  int rc = DEFL_OK;
  for (int i = 0; i < chunks && rc == DEFL_OK; ++i) {
    const int b0 = i * per, bc = (b - b0 < per) ? b - b0 : per;
    const size_t off = (size_t)b0 * per_matrix;
    defl_opts o;
    if (opts) o = *opts; else memset(&o, 0, sizeof(o));
    // matrix b0 + j of the batch keeps the sketch it would get in one call: its slice of Omega, or stream b0 + j
    if (o.sketch) o.sketch += (size_t)b0 * ms * l; else o.seed += (uint64_t)b0;
    if (ctx_fail(c, cudaStreamWaitEvent(c->stream, c->chunk_in[i], 0), "wait")) { rc = DEFL_ERR_CUDA; break; }
    rc = defl_polar_batched(c, (char*)c->stage_in + off, (char*)c->stage_out + off, bc, m, n, dtype, k, oversample,
                            power_iters, coeff_schedule, L, &o, nullptr);
    if (rc) break;
    if (ctx_fail(c, cudaEventRecord(c->chunk_done[i], c->stream), "record") ||
        ctx_fail(c, cudaStreamWaitEvent(c->copy_out, c->chunk_done[i], 0), "wait") ||
        ctx_fail(c, cudaMemcpyAsync((char*)out_host + off, (char*)c->stage_out + off, (size_t)bc * per_matrix,
                                    cudaMemcpyDeviceToHost, c->copy_out), "D2H"))
      rc = DEFL_ERR_CUDA;
  }
  // everything queued so far finishes before the call returns, also after an error
  const cudaError_t e1 = cudaStreamSynchronize(c->copy_in), e2 = cudaStreamSynchronize(c->stream),
                    e3 = cudaStreamSynchronize(c->copy_out);
  if (rc) return rc;
  if (ctx_fail(c, e1, "synchronize") || ctx_fail(c, e2, "synchronize") || ctx_fail(c, e3, "synchronize")) return DEFL_ERR_CUDA;
  return DEFL_OK;
}

}  // extern "C"
