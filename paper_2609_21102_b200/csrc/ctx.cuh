// The context behind the opaque defl_ctx handle, shared by api.cu and psd.cu.
#pragma once
#include <cuda_runtime.h>
#include "common.cuh"
#include <cuda_bf16.h>

#define DEFL_MAX_MARKS 12
#define DEFL_PROFILE_CALLS 64

#define DEFL_HOST_MAX_CHUNKS 8

struct defl_ctx {
  int device;
  int num_sms;
  cudaStream_t stream;
  void* ws;              // scratch memory owned by the context
  size_t ws_bytes;
  void* stage_in;        // device staging of host inputs/outputs (defl_polar_batched_host)
  void* stage_out;
  size_t stage_bytes;
  cudaStream_t copy_in, copy_out;          // host-buffer entry point: copies overlap the compute stream
  cudaEvent_t chunk_in[DEFL_HOST_MAX_CHUNKS], chunk_done[DEFL_HOST_MAX_CHUNKS];
  int copy_ready;                           // streams and events above exist
  int* wait_status;      // device words: [0] the tensor engine ORs DEFL_ST_DEVICE_WAIT into it (cleared at the start of
                         // every polar / PSD call), [1] its tile counter
  defl::TcKnobs tc_knobs;        // tuning overrides, read from the environment when the context was created
  struct { int transposed_apply; int host_chunks; int jacobi_sweeps; int paired_steps; } knobs;   // DEFL_NO_TRANSPOSED_APPLY, DEFL_HOST_CHUNKS, DEFL_JACOBI_SWEEPS, DEFL_NO_PAIRED_STEPS
  defl::TmCache tm_cache;        // encoded TMA descriptors of recent launches
  void* ident_bf16;              // device, 256 x 256 bf16 identity (operand of the engine's identity segment)
  long long launches;    // kernels launched so far
  bool profiling;
  // stage marks of the last DEFL_PROFILE_CALLS calls (events are created when profiling is first switched on)
  long long call_seq;                                   // calls that recorded marks so far
  int n_marks[DEFL_PROFILE_CALLS];
  cudaEvent_t marks[DEFL_PROFILE_CALLS][DEFL_MAX_MARKS];
  bool marks_ready;
  char err[256];
};

namespace defl {
size_t align_up(size_t x, size_t a);
bool ctx_fail(defl_ctx* c, cudaError_t e, const char* where);
int ctx_reserve(defl_ctx* c, size_t bytes);
void ctx_stage_mark(defl_ctx* c);
void ctx_profile_begin(defl_ctx* c);     // a call starts: its marks go to the next slot of the ring
int run_gemm(defl_ctx* c, const GemmDesc& g, int engine, const char* what);
int partials_per_batch(defl_ctx* c, const GemmDesc& g, int engine);
int orthonormalise(defl_ctx* c, float* P, int b, int rows, int l, double* gram, float* Rinv, int* status,
                   __nv_bfloat16* hi = nullptr, __nv_bfloat16* lo = nullptr, int lp = 0, int passes = 2);
cudaError_t or_status_launch(int* status, int n, const int* word, cudaStream_t st, long long* launches);
}  // namespace defl
