// fp32-FMA product engine: C = epilogue(opA(A) opB(B)) for arbitrary strides and bf16/half/fp32 inputs.
// It is the library's own reference engine (every shape, exact fp32 products) and the engine of
// the fp32 polar path; the large bf16 products normally run on the tensor-core engine instead.
#include "common.cuh"

namespace defl {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

template <typename TIn>
__device__ __forceinline__ float to_f(TIn v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <>
__device__ __forceinline__ float to_f<__half>(__half v) { return __half2float(v); }

template <typename TIn, typename TB>
__global__ void __launch_bounds__(NT) gemm_simt_kernel(const GemmDesc g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  __shared__ double red[NT / 32];

  const int tn = blockIdx.x, tm = blockIdx.y, bz = blockIdx.z;
  if (g.symmetric && tn < tm) return;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  const int row0 = tm * BM, col0 = tn * BN;

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int seg = 0; seg < g.nseg; ++seg) {
    const TIn* A = reinterpret_cast<const TIn*>(g.A[seg]) + (long long)bz * g.batch_a[seg];
    const TB* B = reinterpret_cast<const TB*>(g.B[seg]) + (long long)bz * g.batch_b[seg];
    const long long sai = g.sa_i[seg], sak = g.sa_k[seg], sbk = g.sb_k[seg], sbj = g.sb_j[seg];
    const int K = g.K[seg];
    const bool a_kfast = (sak == 1), b_jfast = (sbj == 1);
    for (int k0 = 0; k0 < K; k0 += BK) {
      // A tile: BM x BK, fastest thread index along the contiguous direction
#pragma unroll
      for (int it = 0; it < (BM * BK) / NT; ++it) {
        const int e = tid + it * NT;
        int i, kk;
        if (a_kfast) { i = e / BK; kk = e % BK; } else { kk = e / BM; i = e % BM; }
        const int gi = row0 + i, gk = k0 + kk;
        float v = 0.f;
        if (gi < g.M && gk < K) v = to_f<TIn>(A[(long long)gi * sai + (long long)gk * sak]);
        As[kk][i] = v;
      }
#pragma unroll
      for (int it = 0; it < (BN * BK) / NT; ++it) {
        const int e = tid + it * NT;
        int j, kk;
        if (b_jfast) { kk = e / BN; j = e % BN; } else { j = e / BK; kk = e % BK; }
        const int gj = col0 + j, gk = k0 + kk;
        float v = 0.f;
        if (gj < g.N && gk < K) {
          v = to_f<TB>(B[(long long)gk * sbk + (long long)gj * sbj]);
          if (g.b_split == 2)
            v += to_f<TB>((reinterpret_cast<const TB*>(g.B[1]) + (long long)bz * g.batch_b[0])[(long long)gk * sbk + (long long)gj * sbj]);
        }
        Bs[kk][j] = v;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        float a[TM], b[TN];
#pragma unroll
        for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
        for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
      __syncthreads();
    }
  }

  float alpha = g.alpha, aux_scale = g.aux_scale;
  if (g.alpha_dev) alpha *= g.alpha_dev[bz];
  if (g.aux_scale_dev) aux_scale *= g.aux_scale_dev[bz];
  const long long coff = (long long)bz * g.batch_c, xoff = (long long)bz * g.batch_aux;
  double sq = 0.0;
  // fp32 rows that a thread can take 16 bytes at a time (the rank-k updates of n x n matrices are pure epilogue)
  const bool vec4 = TN == 4 && !g.symmetric && g.out_dtype == F32 && (g.epilogue == EPI_STORE || g.aux_dtype == F32) &&
                    g.epilogue != EPI_RESID_NORM && col0 + BN <= g.N && (g.ldc & 3) == 0 && (g.batch_c & 3) == 0 &&
                    (reinterpret_cast<uintptr_t>(g.C) & 15) == 0 &&
                    (g.epilogue == EPI_STORE || ((g.ld_aux & 3) == 0 && (g.batch_aux & 3) == 0 &&
                                                 (reinterpret_cast<uintptr_t>(g.aux) & 15) == 0));
  if (vec4) {
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const int gi = row0 + ty * TM + i;
      if (gi >= g.M) continue;
      const int gj = col0 + tx * TN;
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      if (g.epilogue != EPI_STORE) {
        const float4 x4 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g.aux) + xoff + (long long)gi * g.ld_aux + gj);
        x[0] = x4.x; x[1] = x4.y; x[2] = x4.z; x[3] = x4.w;
      }
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a = acc[i][j];
        if (g.epilogue == EPI_STORE) v[j] = alpha * a;
        else if (g.epilogue == EPI_POLY) v[j] = g.pb * x[j] + g.pc * a + ((gi == gj + j) ? g.pa : 0.f);
        else v[j] = aux_scale * x[j] + alpha * a;
        if (g.round_tf32) v[j] = round_to_tf32(v[j]);
      }
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(g.C) + coff + (long long)gi * g.ldc + gj) = make_float4(v[0], v[1], v[2], v[3]);
    }
    return;
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int gi = row0 + ty * TM + i;
    if (gi >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int gj = col0 + tx * TN + j;
      if (gj >= g.N) continue;
      const float a = acc[i][j];
      float v;
      switch (g.epilogue) {
        case EPI_STORE: v = alpha * a; break;
        case EPI_POLY:
          v = g.pb * ld_as_float(g.aux, xoff + (long long)gi * g.ld_aux + gj, g.aux_dtype) + g.pc * a +
              ((gi == gj) ? g.pa : 0.f);
          break;
        case EPI_AUX_PLUS:
          v = aux_scale * ld_as_float(g.aux, xoff + (long long)gi * g.ld_aux + gj, g.aux_dtype) + alpha * a;
          break;
        default: {  // EPI_RESID_NORM
          const float r = ld_as_float(g.aux, xoff + (long long)gi * g.ld_aux + gj, g.aux_dtype) - a;
          sq += (double)r * (double)r;
          continue;
        }
      }
      if (g.round_tf32) v = round_to_tf32(v);
      if (g.symmetric) {
        if (gj >= gi) st_from_float(g.C, coff + (long long)gi * g.ldc + gj, g.out_dtype, v);
        if (gj > gi) st_from_float(g.C, coff + (long long)gj * g.ldc + gi, g.out_dtype, v);
      } else {
        st_from_float(g.C, coff + (long long)gi * g.ldc + gj, g.out_dtype, v);
      }
    }
  }
  if (g.epilogue == EPI_RESID_NORM) {
    // fixed-order block reduction: lanes by shuffle tree, warps summed in index order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_down_sync(0xffffffffu, sq, o);
    if ((tid & 31) == 0) red[tid >> 5] = sq;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int w = 0; w < NT / 32; ++w) t += red[w];
      g.partials[(long long)bz * g.partials_per_batch + (long long)tm * gridDim.x + tn] = t;
    }
  }
}

}  // namespace

int gemm_simt_partials_per_batch(const GemmDesc& g) {
  return ((g.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
}

cudaError_t gemm_simt_launch(const GemmDesc& g, cudaStream_t st, long long* launches) {
  if (g.batch <= 0 || g.M <= 0 || g.N <= 0) return cudaSuccess;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  if (g.in_dtype == F16 || g.b_dtype == F16) {
    // IEEE half operands (iterates of the bf16 path on shapes the tensor engine cannot take): both or neither
    if (g.in_dtype != F16 || g.b_dtype != F16) return cudaErrorNotSupported;
    gemm_simt_kernel<__half, __half><<<grid, NT, 0, st>>>(g);
  } else if (g.in_dtype == BF16 && g.b_dtype == BF16) gemm_simt_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, NT, 0, st>>>(g);
  else if (g.in_dtype == BF16) gemm_simt_kernel<__nv_bfloat16, float><<<grid, NT, 0, st>>>(g);
  else if (g.b_dtype == BF16) gemm_simt_kernel<float, __nv_bfloat16><<<grid, NT, 0, st>>>(g);
  else gemm_simt_kernel<float, float><<<grid, NT, 0, st>>>(g);
  if (launches) ++*launches;
  return cudaGetLastError();
}

}  // namespace defl
