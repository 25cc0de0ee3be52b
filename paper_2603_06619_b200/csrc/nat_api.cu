// C-ABI entry points of the policy loss: argument validation and dispatch to
// the fp32 (SIMT) or bf16 (tensor-core) implementation.
#include <cstring>

#include "nat_common.cuh"

namespace nat {

char* error_buffer() {
  static thread_local char buf[512] = {0};
  return buf;
}

int fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(error_buffer(), 512, fmt, ap);
  va_end(ap);
  return status;
}

int require_sm100() {
  int dev = 0;
  NAT_CUDA(cudaGetDevice(&dev));
  int major = 0;
  NAT_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10)
    return fail(NAT_ERR_UNSUPPORTED, "the bf16 path needs compute capability 10.x (found %d.x)",
                major);
  return NAT_OK;
}

static int validate(const char* who, const nat_loss_params* p, const LossArgs& a, bool bwd,
                    bool fwd = true) {
  if (!p) return fail(NAT_ERR_INVALID_ARG, "%s: params is null", who);
  if (p->d <= 0 || p->V <= 0 || p->B <= 0)
    return fail(NAT_ERR_INVALID_ARG, "%s: d, V and B must be positive", who);
  if (p->dtype != NAT_F32 && p->dtype != NAT_BF16)
    return fail(NAT_ERR_UNSUPPORTED, "%s: unknown dtype %d", who, p->dtype);
  if (!(p->clip_lo >= 0.f) || !(p->clip_hi >= 0.f))
    return fail(NAT_ERR_INVALID_ARG, "%s: clip bounds must be >= 0", who);
  if (p->kl_beta != 0.f && !p->ref_logp)
    return fail(NAT_ERR_INVALID_ARG, "%s: kl_beta != 0 needs ref_logp", who);
  if (a.cap < 0 || a.cap > 0x7FFFFFFFll)
    return fail(NAT_ERR_INVALID_ARG, "%s: n_sel_cap out of range", who);
  if (!a.hidden || !a.W || !a.targets || !a.old_logp || !a.adv || !a.pi || !a.cu_seqlens ||
      !a.sel_idx || !a.sel_resp || !a.n_sel || !a.logp || !a.lse)
    return fail(NAT_ERR_INVALID_ARG, "%s: null pointer", who);
  if ((!bwd || fwd) && !a.loss) return fail(NAT_ERR_INVALID_ARG, "%s: loss is null", who);
  if (bwd && (!a.dHidden || !a.dW)) return fail(NAT_ERR_INVALID_ARG, "%s: null gradient", who);
  if (p->dtype == NAT_BF16) {
    if (p->d % 64 != 0)
      return fail(NAT_ERR_UNSUPPORTED, "%s: the bf16 path needs d %% 64 == 0 (d = %d)", who, p->d);
    if (((uintptr_t)a.hidden & 15u) || ((uintptr_t)a.W & 15u) ||
        (bwd && (((uintptr_t)a.dHidden & 15u) || ((uintptr_t)a.dW & 15u))))
      return fail(NAT_ERR_INVALID_ARG, "%s: matrices must be 16-byte aligned", who);
  }
  const size_t need = nat_policy_loss_workspace_bytes(p, a.cap);
  if (need == 0)
    return fail(NAT_ERR_UNSUPPORTED, "%s: this dtype does not cover d = %d (float32 needs d <= 1024)",
                who, p->d);
  if (!a.workspace || a.workspace_bytes < need)
    return fail(NAT_ERR_CAPACITY, "%s: workspace too small (%zu < %zu)", who, a.workspace_bytes,
                need);
  if ((uintptr_t)a.workspace & 255u)
    return fail(NAT_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
  return NAT_OK;
}

}  // namespace nat

extern "C" {

const char* nat_status_string(int status) {
  switch (status) {
    case NAT_OK: return "ok";
    case NAT_ERR_INVALID_ARG: return "invalid argument";
    case NAT_ERR_UNSUPPORTED: return "unsupported configuration";
    case NAT_ERR_CAPACITY: return "capacity too small";
    case NAT_ERR_CUDA: return "CUDA error";
    default: return "unknown status";
  }
}

const char* nat_last_error(void) { return nat::error_buffer(); }

int nat_version(void) { return 2; }

int nat_poll_status(const void* workspace, void* stream, uint32_t* host_word) {
  if (!workspace || !host_word)
    return nat::fail(NAT_ERR_INVALID_ARG, "nat_poll_status: null pointer");
  NAT_CUDA(cudaMemcpyAsync(host_word, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost,
                           (cudaStream_t)stream));
  NAT_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  return NAT_OK;
}

size_t nat_policy_loss_workspace_bytes(const nat_loss_params* p, int64_t n_sel_cap) {
  if (!p || n_sel_cap < 0 || p->d <= 0 || p->V <= 0) return 0;
  if (p->dtype == NAT_F32) return nat::loss_f32_workspace_bytes(*p, n_sel_cap);
  if (p->dtype == NAT_BF16) return nat::loss_bf16_workspace_bytes(*p, n_sel_cap);
  return 0;
}

int nat_policy_loss_fwd(const nat_loss_params* params, const void* hidden, const void* W,
                        const int32_t* targets, const float* old_logp, const float* adv,
                        const float* pi, const int32_t* cu_seqlens, const int32_t* sel_idx,
                        const int32_t* sel_resp, const int32_t* n_sel, int64_t n_sel_cap,
                        float* loss, float* logp, float* lse, void* workspace,
                        size_t workspace_bytes, void* stream) {
  nat::LossArgs a{};
  if (params) a.p = *params;
  a.hidden = hidden; a.W = W; a.targets = targets; a.old_logp = old_logp; a.adv = adv; a.pi = pi;
  a.cu_seqlens = cu_seqlens; a.sel_idx = sel_idx; a.sel_resp = sel_resp; a.n_sel = n_sel;
  a.cap = n_sel_cap; a.loss = loss; a.logp = logp; a.lse = lse;
  a.workspace = workspace; a.workspace_bytes = workspace_bytes; a.stream = (cudaStream_t)stream;
  int s = nat::validate("nat_policy_loss_fwd", params, a, false);
  if (s != NAT_OK) return s;
  return params->dtype == NAT_F32 ? nat::loss_f32_fwd(a) : nat::loss_bf16_fwd(a);
}

int nat_policy_loss_bwd(const nat_loss_params* params, const void* hidden, const void* W,
                        const int32_t* targets, const float* old_logp, const float* adv,
                        const float* pi, const int32_t* cu_seqlens, const int32_t* sel_idx,
                        const int32_t* sel_resp, const int32_t* n_sel, int64_t n_sel_cap,
                        const float* logp, const float* lse, const float* dloss, void* dHidden,
                        float* dW, void* workspace, size_t workspace_bytes, void* stream) {
  nat::LossArgs a{};
  if (params) a.p = *params;
  a.hidden = hidden; a.W = W; a.targets = targets; a.old_logp = old_logp; a.adv = adv; a.pi = pi;
  a.cu_seqlens = cu_seqlens; a.sel_idx = sel_idx; a.sel_resp = sel_resp; a.n_sel = n_sel;
  a.cap = n_sel_cap; a.logp = const_cast<float*>(logp); a.lse = const_cast<float*>(lse);
  a.dloss = dloss; a.dHidden = dHidden; a.dW = dW;
  a.workspace = workspace; a.workspace_bytes = workspace_bytes; a.stream = (cudaStream_t)stream;
  int s = nat::validate("nat_policy_loss_bwd", params, a, true, false);
  if (s != NAT_OK) return s;
  return params->dtype == NAT_F32 ? nat::loss_f32_bwd(a) : nat::loss_bf16_bwd(a);
}

int nat_policy_loss_fwd_bwd(const nat_loss_params* params, const void* hidden, const void* W,
                            const int32_t* targets, const float* old_logp, const float* adv,
                            const float* pi, const int32_t* cu_seqlens, const int32_t* sel_idx,
                            const int32_t* sel_resp, const int32_t* n_sel, int64_t n_sel_cap,
                            const float* dloss, float* loss, float* logp, float* lse,
                            void* dHidden, float* dW, void* workspace, size_t workspace_bytes,
                            void* stream) {
  nat::LossArgs a{};
  if (params) a.p = *params;
  a.hidden = hidden; a.W = W; a.targets = targets; a.old_logp = old_logp; a.adv = adv; a.pi = pi;
  a.cu_seqlens = cu_seqlens; a.sel_idx = sel_idx; a.sel_resp = sel_resp; a.n_sel = n_sel;
  a.cap = n_sel_cap; a.loss = loss; a.logp = logp; a.lse = lse; a.dloss = dloss;
  a.dHidden = dHidden; a.dW = dW;
  a.workspace = workspace; a.workspace_bytes = workspace_bytes; a.stream = (cudaStream_t)stream;
  int s = nat::validate("nat_policy_loss_fwd_bwd", params, a, true, true);
  if (s != NAT_OK) return s;
  return params->dtype == NAT_F32 ? nat::loss_f32_fwd_bwd(a) : nat::loss_bf16_fwd_bwd(a);
}

int nat_trace_begin(void) { return nat::trace_begin(); }

int nat_trace_end(float* ms_by_kind, int32_t* launches_by_kind) {
  return nat::trace_end(ms_by_kind, launches_by_kind);
}

}  // extern "C"
