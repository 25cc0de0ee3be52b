// Fixed-order loss reduction and gradient-coefficient kernels.
#include "nat_token.cuh"

namespace nat {
namespace {

__global__ void __launch_bounds__(1024)
loss_reduce_kernel(const float* __restrict__ term, const int32_t* __restrict__ n_sel, int64_t cap,
                   float* __restrict__ loss, WorkspaceHead* head) {
  __shared__ double part[1024];
  int64_t n = *n_sel;
  if (n > cap) {
    n = cap;
    if (threadIdx.x == 0) atomicOr(&head->status, NAT_DEV_CAPACITY);
  }
  double s = 0.0;
  for (int64_t k = threadIdx.x; k < n; k += 1024) s += (double)term[k];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *loss = (float)part[0];
}

__global__ void grad_coeff_kernel(TokenCtx c, const float* __restrict__ logp,
                                  const int32_t* __restrict__ n_sel, int64_t cap,
                                  const float* __restrict__ dloss, float* __restrict__ g) {
  const int64_t n = min((int64_t)*n_sel, cap);
  const float dl = dloss ? *dloss : 1.f;
  for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n;
       k += (int64_t)gridDim.x * blockDim.x) {
    float term, gk;
    token_eval(c, (int)k, logp[k], dl, &term, &gk);
    g[k] = gk;
  }
}

}  // namespace

TokenCtx make_token_ctx(const LossArgs& a, uint32_t* status) {
  TokenCtx c;
  c.targets = a.targets;
  c.old_logp = a.old_logp;
  c.adv = a.adv;
  c.pi = a.pi;
  c.cu_seqlens = a.cu_seqlens;
  c.sel_idx = a.sel_idx;
  c.sel_resp = a.sel_resp;
  c.B = a.p.B;
  c.clip_lo = a.p.clip_lo;
  c.clip_hi = a.p.clip_hi;
  c.kl_beta = a.p.kl_beta;
  c.ref_logp = a.p.ref_logp;
  c.V = a.p.V;
  c.status = status;
  return c;
}

int launch_loss_reduce(const float* term, const int32_t* n_sel, int64_t cap, float* loss,
                       WorkspaceHead* head, cudaStream_t stream) {
  loss_reduce_kernel<<<1, 1024, 0, stream>>>(term, n_sel, cap, loss, head);
  NAT_LAUNCH_CHECK("loss_reduce_kernel");
  return NAT_OK;
}

int launch_grad_coeff(const TokenCtx& c, const float* logp, const int32_t* n_sel, int64_t cap,
                      const float* dloss, float* g, cudaStream_t stream) {
  if (cap == 0) return NAT_OK;
  const int grid = (int)min((int64_t)1184, (cap + 255) / 256);
  grad_coeff_kernel<<<grid, 256, 0, stream>>>(c, logp, n_sel, cap, dloss, g);
  NAT_LAUNCH_CHECK("grad_coeff_kernel");
  return NAT_OK;
}

}  // namespace nat
