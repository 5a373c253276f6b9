// Launchers of the small-panel kernels (see panel.cu). None of them synchronises.
#pragma once
#include <cuda_runtime.h>

namespace defl {

constexpr int MAX_L = 64;   // widest panel (sketch width / PSD basis width)

int gram_num_chunks(int rows);
// partial Gram blocks of Y^T Y2 (Y2 = nullptr: Y^T Y)
cudaError_t gram_partial_launch(const float* Y, long long batch_stride, int batch, int rows, int l, int ld,
                                double* partial, cudaStream_t st, long long* launches, const float* Y2 = nullptr);
cudaError_t chol_inv_launch(const double* partial, int nchunk, int batch, int l, float* Rinv, int* status,
                            cudaStream_t st, long long* launches);
cudaError_t panel_apply_launch(const float* In, long long in_bs, int ld_in, const float* Mtx, int ldm, int batch,
                               int rows, int l, int kout, float* Out, long long out_bs, int ld_out, cudaStream_t st,
                               long long* launches);
cudaError_t jacobi_eig_launch(const double* partial, int nchunk, int batch, int l, int signed_input, float* s_out,
                              float* E, float* Es, int* status, cudaStream_t st, long long* launches, int max_sweeps = 0);
cudaError_t frob_partial_launch(const void* X, int dtype, int batch, long long count, int nblk, double* partial,
                                cudaStream_t st, long long* launches);
constexpr int FROB_VEC_BLOCKS = 148;    // CTAs (and partial sums) per matrix of the vectorised Frobenius pass
cudaError_t frob_partial_vec_launch(const void* X, int dtype, int batch, long long count, int nblk, double* partial,
                                    cudaStream_t st, long long* launches);
cudaError_t rho_identity_launch(const double* partial, int nper, int batch, const float* s, int ld_s, const int* keff,
                                float* rho, float* inv_rho, float* inv_rho2, int* status, cudaStream_t st,
                                long long* launches);
cudaError_t finite_probe_launch(const void* X, int dtype, int batch, long long count, int* status, cudaStream_t st,
                                long long* launches);
cudaError_t rho_finalize_launch(const double* partial, int nper, int batch, float* rho, float* inv_rho,
                                float* inv_rho2, int* status, cudaStream_t st, long long* launches);
cudaError_t scale_cols_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int k, const float* s,
                              int ld_s, const float* inv_rho, float c0, float c1, float* Out, long long out_bs,
                              int ld_out, cudaStream_t st, long long* launches, const int* keff = nullptr);
cudaError_t scale_launch(const void* In, int in_dt, void* Out, int out_dt, int batch, long long count,
                         const float* scale, cudaStream_t st, long long* launches, int round_tf32 = 0, float mult = 1.f);
cudaError_t fill_gaussian_launch(void* dst, long long count, int dtype, unsigned long long seed, long long per_stream,
                                 unsigned long long seed_stride, cudaStream_t st, long long* launches);
cudaError_t fill_int_launch(int* p, int n, int v, cudaStream_t st, long long* launches);

}  // namespace defl

#include <cuda_bf16.h>
namespace defl {
cudaError_t split_panel_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int l, int lp,
                               __nv_bfloat16* hi, __nv_bfloat16* lo, cudaStream_t st, long long* launches);
cudaError_t split_concat3_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int k, int kp,
                                 const float* s, int ld_s, const float* inv_rho, float c0, float c1, int pattern,
                                 __nv_bfloat16* Out, cudaStream_t st, long long* launches, const int* keff = nullptr,
                                 int f16 = 0, int transposed = 0, float mult = 1.f, const float* rho = nullptr);
cudaError_t zero_residual_entry_launch(const int* status, const float* P, const float* W, const int* keff, int batch, int m,
                                       int n, int k, float scale, void* X0, int dtype, cudaStream_t st, long long* launches);
cudaError_t gate_launch(const float* s, int ld_s, int batch, int window, int kmax, float tau, int* keff, cudaStream_t st,
                        long long* launches);
}  // namespace defl

namespace defl {
int fused_num_chunks(int rows, int batch);
// Out = In * Mtx[:, :kout] (Mtx null: identity), optional fp32 / bf16 hi+lo outputs, optional Gram partials of Out
// ([b, fused_num_chunks(rows, b), w, w] fp64 with w = width of Out)
cudaError_t panel_fused_launch(const float* In, long long in_bs, int ld_in, int batch, int rows, int l, const float* Mtx,
                               int ldm, int kout, float* Out, long long out_bs, int ld_out, __nv_bfloat16* hi,
                               __nv_bfloat16* lo, int lp, double* partial, cudaStream_t st, long long* launches);
// Muon momentum: Mom <- mu Mom + Grad (stored type `dtype`); look (may be null) <- Grad + mu Mom_stored
cudaError_t momentum_launch(void* Mom, const void* Grad, void* look, int dtype, long long count, float mu, cudaStream_t st,
                            long long* launches);

}  // namespace defl
