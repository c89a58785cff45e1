// Shared host/device helpers of the sm_100a denoising-step library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ds.h"

namespace ds {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Count of kernels launched through the C ABI (read by ds_launch_count()).
void note_launch(int n = 1);

inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// Number of SMs of the current device (cached per device).
int sm_count();

#define DS_CUDA_OK(expr)                          \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) {                      \
      (void)cudaGetLastError();                   \
      ::ds::note_cuda_error((int)_e);             \
      return DS_ERR_CUDA;                         \
    }                                             \
  } while (0)

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Launchers implemented in the per-kernel translation units.
int launch_confidence(const void *logits, int dtype, int64_t rows, int64_t V, int64_t ld,
                      const int32_t *row_list, int64_t n_listed, const int32_t *n_listed_dev, float *conf,
                      int32_t *tok, void *workspace, size_t workspace_bytes, cudaStream_t stream);
size_t confidence_workspace_bytes(int64_t rows, int64_t V, int dtype);
int launch_confidence_static(const void *logits, int dtype, int64_t rows, int64_t V, int64_t ld,
                             const int32_t *row_list, int64_t n_listed, float *conf, int32_t *tok,
                             cudaStream_t stream);
size_t lmhead_workspace_bytes(int64_t rows, int64_t V);
int launch_lmhead_confidence(const void *hidden, const void *weight, int64_t rows, int64_t hid, int64_t V, int64_t ld_h,
                             int64_t ld_w, float *conf, int32_t *tok, void *workspace, uint32_t *status,
                             cudaStream_t stream);
int launch_block_begin(const ds_block_params &p, cudaStream_t stream);
int launch_select(const ds_select_params &p, cudaStream_t stream);
int launch_rope_gather(const ds_rope_params &p, cudaStream_t stream);
int launch_bounded_wait_selftest(uint32_t poll_limit, uint32_t *status, int32_t *report, cudaStream_t stream);
void note_cuda_error(int code);  // remembered per host thread for ds_last_cuda_error
int launch_attn_simt(const ds_attn_params &p, cudaStream_t stream);
int launch_attn_tc(const ds_attn_params &p, cudaStream_t stream);
int launch_attn_tc2(const ds_attn_params &p, cudaStream_t stream);

// An attention call whose kernel parameters (tensor maps included) have been worked out once: what a
// ds_attn_plan holds and what the one-shot launchers build on the stack.
enum : int { kAttnPathSimt = 0, kAttnPathTc = 1, kAttnPathTc2 = 2 };
struct AttnPrepared {
  int path;
  int grid;          // CTAs to launch; 0 = nothing to do
  ds_attn_params p;  // validated copy of the caller's arguments (the SIMT kernel takes it as it is)
  alignas(64) unsigned char kernel_params[2048];  // the tensor-core kernels' parameter struct
};
int prepare_attn_tc(const ds_attn_params &p, AttnPrepared &out);
int prepare_attn_tc2(const ds_attn_params &p, AttnPrepared &out);
int launch_prepared_tc(const AttnPrepared &a, cudaStream_t stream);
int launch_prepared_tc2(const AttnPrepared &a, cudaStream_t stream);
bool attn_tc_supported(const ds_attn_params &p);
size_t attn_tc_workspace_bytes(const ds_attn_params &p);

}  // namespace ds
