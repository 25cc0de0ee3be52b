// Per-token scalar part of the policy loss, shared by the fp32 and bf16 paths:
// importance ratio, clipped surrogate, Horvitz-Thompson weight, the gradient
// coefficient, and the fixed-order reduction of the loss.
#pragma once

#include "nat_common.cuh"

namespace nat {

// Layout of the head of every loss workspace.
struct WorkspaceHead {
  uint32_t status;  // NAT_DEV_* bits, or-ed in by kernels
  uint32_t pad[63];
};
static_assert(sizeof(WorkspaceHead) == 256, "workspace head is one 256-byte block");

struct TokenCtx {
  const int32_t* targets;
  const float* old_logp;
  const float* adv;
  const float* pi;
  const int32_t* cu_seqlens;
  const int32_t* sel_idx;
  const int32_t* sel_resp;
  int B;
  float clip_lo, clip_hi;
  float kl_beta;          // 0: no KL term
  const float* ref_logp;  // read only when kl_beta != 0
  int V;                  // targets outside [0, V) are reported and their tokens left out
  uint32_t* status;       // the workspace's status word
};

// Fills the fields every loss path takes from the call's arguments.
TokenCtx make_token_ctx(const LossArgs& a, uint32_t* status);

// For selected token k with log-probability logp:
//   r = exp(logp - old_logp), S = min(r A, clip(r) A), w = 1 / (pi T B)
//   term = -w (S - kl_beta (logp - ref_logp))      (the token's share of the loss)
//   g    = -dloss w (A r [surrogate not saturated] - kl_beta)
__device__ __forceinline__ bool target_ok(const TokenCtx& c, int k) {
  return (unsigned)c.targets[c.sel_idx[k]] < (unsigned)c.V;
}

__device__ __forceinline__ void token_eval(const TokenCtx& c, int k, float logp, float dloss,
                                           float* term, float* g) {
  const int n = c.sel_idx[k];
  const int i = c.sel_resp[k];
  if ((unsigned)c.targets[n] >= (unsigned)c.V) {  // no such vocabulary entry: leave the token out
    atomicOr(c.status, NAT_DEV_BAD_TARGET);
    *term = 0.f;
    *g = 0.f;
    return;
  }
  const float A = c.adv[i];
  const float T = (float)(c.cu_seqlens[i + 1] - c.cu_seqlens[i]);
  const float w = 1.f / (c.pi[n] * T * (float)c.B);
  const float r = expf(logp - c.old_logp[n]);
  const float hi = 1.f + c.clip_hi, lo = 1.f - c.clip_lo;
  const float rc = fminf(fmaxf(r, lo), hi);
  const float S = fminf(r * A, rc * A);
  const bool live = (A > 0.f && r <= hi) || (A < 0.f && r >= lo);
  float t = -w * S;
  float gk = live ? -dloss * w * A * r : 0.f;
  if (c.kl_beta != 0.f) {
    t += w * c.kl_beta * (logp - c.ref_logp[n]);
    gk += dloss * w * c.kl_beta;
  }
  *term = t;
  *g = gk;
}

// loss = sum_k term[k] in a fixed order: each of 1024 threads adds a strided
// slice in double, then a shared-memory tree combines them.
int launch_loss_reduce(const float* term, const int32_t* n_sel, int64_t cap, float* loss,
                       WorkspaceHead* head, cudaStream_t stream);

// g[k] for every selected token from the forward's logp (backward's first step).
int launch_grad_coeff(const TokenCtx& c, const float* logp, const int32_t* n_sel, int64_t cap,
                      const float* dloss, float* g, cudaStream_t stream);

}  // namespace nat
