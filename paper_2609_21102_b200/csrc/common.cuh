// Shared declarations of the CUDA library: the product descriptor that both engines consume,
// element-type helpers and the internal kernel-launcher prototypes.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace defl {

enum DType { BF16 = 0, F32 = 1, F16 = 2 };      // F16: IEEE half (operands and iterates of the FP16 projection filter)

__host__ __device__ inline size_t dtype_size(int dt) { return dt == F32 ? 4 : 2; }

// What happens to the fp32 accumulator tile acc[i,j] of C = opA(A) opB(B).
enum Epilogue {
  EPI_STORE = 0,      // C = alpha * acc
  EPI_POLY = 1,       // C = pa * [i==j] + pb * aux[i,j] + pc * acc        (B_t = a I + b A_t + c A_t^2, Eq. 2)
  EPI_AUX_PLUS = 2,   // C = aux_scale * aux[i,j] + alpha * acc            (deflate+normalise, restore, PSD reconstruct)
  EPI_RESID_NORM = 3  // partial sums of (aux[i,j] - acc)^2, nothing stored (||G - U_k S_k V_k^T||_F^2)
};

// One batched product. Element (i,kk) of opA is A[i*sa_i + kk*sa_k]; element (kk,j) of opB is
// B[kk*sb_k + j*sb_j]; C and aux are row-major [M,N] with leading dimension ldc / ld_aux.
// Up to two K segments are summed into the same accumulator: acc = A0 B0 + A1 B1 (used for the
// split-precision panels and for the restore step appended to the last filter product).
struct GemmDesc {
  int batch, M, N;
  int nseg;
  int K[2];
  const void* A[2]; long long sa_i[2], sa_k[2], batch_a[2];
  const void* B[2]; long long sb_k[2], sb_j[2], batch_b[2];
  int in_dtype;                 // type of A (both segments)
  int b_dtype;                  // type of B (both segments); the tensor engine needs b_dtype == in_dtype
  void* C; long long ldc, batch_c; int out_dtype;
  const void* aux; long long ld_aux, batch_aux; int aux_dtype;
  int epilogue;
  float alpha, aux_scale, pa, pb, pc;
  const float* alpha_dev;       // optional per-batch multiplier of alpha (device, [batch])
  const float* aux_scale_dev;   // optional per-batch multiplier of aux_scale (device, [batch])
  double* partials;             // EPI_RESID_NORM: [batch, partials_per_batch] written, one slot per CTA-warp
  int partials_per_batch;
  int b_split;                  // 2: opB = B[0] + B[1] (same shape and strides, nseg must be 1); the A tile is loaded once
  int round_tf32;               // fp32 output rounded to nearest tf32 (it feeds tf32 products, which would truncate)
  int symmetric;                // output is symmetric (M == N): compute upper tiles only and mirror
  int transpose_out;            // element (i, j) of the product is stored at C[j * ldc + i] (tensor engine, EPI_STORE only)
  int seg1_identity;            // tensor engine, nseg = 2: segment 1 adds A[1][i, j] itself to the accumulator, as the product of
                                // A[1] (viewed [M, N], K = the output's column index, K-major) with an identity tile: B[1] points
                                // to a 256 x 256 identity of the operand type (row-major), K[1] is ignored
  int debug_hold_stage;         // test hook, tensor engine, single-CTA form: s > 0 withholds pipeline step s - 1 of each CTA's first tile
};

inline GemmDesc gemm_desc_zero() {
  GemmDesc g;
  memset(&g, 0, sizeof(g));
  g.nseg = 1;
  g.alpha = 1.f;
  g.aux_scale = 1.f;
  return g;
}

// Tuning overrides of the tensor engine, read from the environment ONCE, when a context is created (a value of 0
// keeps the default rule): experiments, and the tests of the tile forms the default rules do not pick.
//   DEFL_TC_BN, DEFL_TC_TILE_M, DEFL_TC_STAGES, DEFL_TC_KSUB, DEFL_TC_PAIR (-1 default, 0 single-CTA form, 1 pair),
//   DEFL_TC_PAIR_MIN_N, DEFL_TC_DYNAMIC (tiles through a counter), DEFL_TC_AUX_PREFETCH (L2 prefetch of `aux`),
//   DEFL_TC_DEBUG, DEFL_TC_WAIT_MS (limit of every device-side wait, default 2000).
struct TcKnobs {
  int bn, tile_m, stages, ksub, pair, pair_min_n, dynamic, aux_prefetch, debug, wait_ms;
};
TcKnobs tc_knobs_from_env();

// Encoded TMA descriptors of recent launches, kept per context: a descriptor depends only on the operand's address,
// shape, strides and box, and the same few operands come back at every step of a filter chain.
struct TmCacheEntry {
  const void* base; long long MN, K, s_mn, s_k, batch, batch_stride; int esize, mn_major; unsigned box_rows;
  alignas(64) unsigned char map[128];
};
struct TmCache {
  static constexpr int SLOTS = 64;
  TmCacheEntry e[SLOTS];
  int used, next;
  long long hits, misses;
};

// Engines (each returns cudaGetLastError() of its launch; they never synchronise).
cudaError_t gemm_simt_launch(const GemmDesc& g, cudaStream_t st, long long* launches);
int gemm_simt_partials_per_batch(const GemmDesc& g);
// Tensor-core engine: returns cudaErrorNotSupported when the descriptor cannot be expressed
// as TMA-tiled tcgen05 products (alignment, type), without launching anything.
cudaError_t gemm_tc_launch(const GemmDesc& g, cudaStream_t st, int* status_word, int num_sms, long long* launches,
                           const TcKnobs* knobs = nullptr, TmCache* cache = nullptr);
bool gemm_tc_supported(const GemmDesc& g);
int gemm_tc_partials_per_batch(const GemmDesc& g, const TcKnobs* knobs = nullptr);

__device__ __forceinline__ float ld_as_float(const void* p, long long idx, int dt) {
  return dt == BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx])
         : dt == F16 ? __half2float(reinterpret_cast<const __half*>(p)[idx])
                     : reinterpret_cast<const float*>(p)[idx];
}
__device__ __forceinline__ float round_to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
__device__ __forceinline__ void st_from_float(void* p, long long idx, int dt, float v) {
  if (dt == BF16) reinterpret_cast<__nv_bfloat16*>(p)[idx] = __float2bfloat16_rn(v);
  else if (dt == F16) reinterpret_cast<__half*>(p)[idx] = __float2half_rn(v);
  else reinterpret_cast<float*>(p)[idx] = v;
}

// two packed 16-bit values (bf16 or, with `f16`, IEEE half) <-> two floats
__device__ __forceinline__ float2 unpack16x2(uint32_t w, bool f16) {
  if (f16) return __half22float2(*reinterpret_cast<const __half2*>(&w));
  return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w));
}
__device__ __forceinline__ uint32_t pack16x2(float a, float b, bool f16) {
  uint32_t w;
  if (f16) { const __half2 h = __floats2half2_rn(a, b); w = *reinterpret_cast<const uint32_t*>(&h); }
  else { const __nv_bfloat162 h = __floats2bfloat162_rn(a, b); w = *reinterpret_cast<const uint32_t*>(&h); }
  return w;
}

}  // namespace defl
