// Deflated PSD projection (Algorithm 2). Placeholder translation unit until the kernels land.
#include "../../include/defl.h"
#include "ctx.cuh"

extern "C" {
size_t defl_psd_workspace_bytes(int n, int K) { (void)n; (void)K; return 0; }
int defl_psd_project(defl_ctx* ctx, const void* X, void* P, int n, int k, float* warm_basis, int K,
                     const float* coeff_schedule, int T, const defl_opts* opts, const defl_info* info) {
  (void)ctx; (void)X; (void)P; (void)n; (void)k; (void)warm_basis; (void)K; (void)coeff_schedule; (void)T; (void)opts; (void)info;
  return DEFL_ERR_UNSUPPORTED;
}
}
