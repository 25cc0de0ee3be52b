// Shared host-side helpers of the NAT library: error reporting and launch checks.
#pragma once

#include <cuda_runtime.h>
#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "nat.h"

namespace nat {

// Thread-local message behind nat_last_error().
char* error_buffer();
int fail(int status, const char* fmt, ...);

inline int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return NAT_OK;
  return fail(NAT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define NAT_CUDA(call)                                   \
  do {                                                   \
    int _s = ::nat::check_cuda((call), #call);           \
    if (_s != NAT_OK) return _s;                         \
  } while (0)

#define NAT_LAUNCH_CHECK(name)                                   \
  do {                                                           \
    int _s = ::nat::check_cuda(cudaGetLastError(), name);        \
    if (_s != NAT_OK) return _s;                                 \
  } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The tensor-core kernels only exist for compute capability 10.x.
int require_sm100();

// ---- entry points of the per-dtype loss implementations -------------------
struct LossArgs {
  nat_loss_params p;
  const void* hidden;
  const void* W;
  const int32_t* targets;
  const float* old_logp;
  const float* adv;
  const float* pi;
  const int32_t* cu_seqlens;
  const int32_t* sel_idx;
  const int32_t* sel_resp;
  const int32_t* n_sel;
  int64_t cap;
  float* loss;
  float* logp;
  float* lse;
  const float* dloss;
  void* dHidden;
  float* dW;
  void* workspace;
  size_t workspace_bytes;
  cudaStream_t stream;
};

size_t loss_f32_workspace_bytes(const nat_loss_params& p, int64_t cap);
int loss_f32_fwd(const LossArgs& a);
int loss_f32_bwd(const LossArgs& a);
int loss_f32_fwd_bwd(const LossArgs& a);

size_t loss_bf16_workspace_bytes(const nat_loss_params& p, int64_t cap);
int loss_bf16_fwd(const LossArgs& a);
int loss_bf16_bwd(const LossArgs& a);
int loss_bf16_fwd_bwd(const LossArgs& a);
int trace_begin();
int trace_end(float* ms_by_kind, int32_t* launches_by_kind);

}  // namespace nat
