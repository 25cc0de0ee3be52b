// fp32 policy loss: plain SIMT kernels for small heads (the Tiny workload).
//
// The contraction here is a few MFLOP, far below what fills a tensor-core
// tile, so these kernels favour a fixed summation order over throughput:
// every output element is produced by one thread or one warp, so results are
// reproducible run to run.
#include "nat_token.cuh"

namespace nat {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxD = 1024;           // registers hold d/32 values per lane
constexpr int kRegs = kMaxD / 32;

struct F32Ws {
  WorkspaceHead* head;
  float* term;  // [cap]
  float* g;     // [cap]
};

F32Ws carve(void* ws, int64_t cap) {
  char* p = reinterpret_cast<char*>(ws);
  F32Ws w;
  w.head = reinterpret_cast<WorkspaceHead*>(p);
  p += sizeof(WorkspaceHead);
  w.term = reinterpret_cast<float*>(p);
  p += align_up(sizeof(float) * (size_t)cap, 256);
  w.g = reinterpret_cast<float*>(p);
  return w;
}

__device__ __forceinline__ const float* hidden_row(const float* hidden, const int32_t* sel_idx,
                                                   int compact, int k, int d) {
  const int64_t row = compact ? (int64_t)k : (int64_t)sel_idx[k];
  return hidden + row * d;
}

__device__ __forceinline__ float warp_dot(const float* __restrict__ a, const float* __restrict__ b,
                                          int d, int lane) {
  float s = 0.f;
  for (int j = lane; j < d; j += 32) s = fmaf(a[j], b[j], s);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  return s;
}

// One block per selected row: every warp sweeps a strided set of vocabulary
// rows with an online max / sum-of-exponentials, then the warps are combined.
__global__ void __launch_bounds__(kThreads)
f32_fwd_kernel(TokenCtx c, const float* __restrict__ hidden, const float* __restrict__ W, int d,
               int V, int compact, const int32_t* __restrict__ n_sel, int64_t cap,
               float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ term) {
  extern __shared__ float h_s[];
  __shared__ float m_s[kWarps], s_s[kWarps], zt_s[kWarps];
  const int n = (int)min((int64_t)*n_sel, cap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int k = blockIdx.x; k < n; k += gridDim.x) {
    const float* h = hidden_row(hidden, c.sel_idx, compact, k, d);
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += kThreads) h_s[j] = h[j];
    __syncthreads();
    const int y = c.targets[c.sel_idx[k]];
    float m = -INFINITY, s = 0.f, zt = 0.f;
    for (int v = warp; v < V; v += kWarps) {
      const float z = warp_dot(W + (int64_t)v * d, h_s, d, lane);
      if (v == y) zt = z;
      const float mn = fmaxf(m, z);
      s = s * expf(m - mn) + expf(z - mn);
      m = mn;
    }
    if (lane == 0) {
      m_s[warp] = m;
      s_s[warp] = s;
      zt_s[warp] = zt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float M = -INFINITY;
      for (int w = 0; w < kWarps; ++w) M = fmaxf(M, m_s[w]);
      float S = 0.f;
      for (int w = 0; w < kWarps; ++w)
        if (s_s[w] > 0.f) S += s_s[w] * expf(m_s[w] - M);
      const float l = M + logf(S);
      const bool y_ok = (unsigned)y < (unsigned)V;
      const float lp = y_ok ? zt_s[y % kWarps] - l : __int_as_float(0x7FC00000);
      lse[k] = l;
      logp[k] = lp;
      float t, g;
      token_eval(c, k, lp, 1.f, &t, &g);
      term[k] = t;
    }
  }
}

// dHidden: one block per selected row.  The vocabulary is swept in tiles of
// 256: the warps fill the tile's dz values, then each thread accumulates its
// columns over the tile in index order.
__global__ void __launch_bounds__(kThreads)
f32_dh_kernel(TokenCtx c, const float* __restrict__ hidden, const float* __restrict__ W, int d,
              int V, int compact, const int32_t* __restrict__ n_sel, int64_t cap,
              const float* __restrict__ lse, const float* __restrict__ g,
              float* __restrict__ dH) {
  extern __shared__ float h_s[];
  __shared__ float dz_s[kThreads];
  const int n = (int)min((int64_t)*n_sel, cap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int k = blockIdx.x; k < n; k += gridDim.x) {
    const float* h = hidden_row(hidden, c.sel_idx, compact, k, d);
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += kThreads) h_s[j] = h[j];
    __syncthreads();
    const int y = c.targets[c.sel_idx[k]];
    const float gk = g[k], l = lse[k];
    float acc[kMaxD / kThreads];
#pragma unroll
    for (int q = 0; q < kMaxD / kThreads; ++q) acc[q] = 0.f;
    for (int v0 = 0; v0 < V; v0 += kThreads) {
      const int vend = min(kThreads, V - v0);
      for (int vv = warp; vv < vend; vv += kWarps) {
        const int v = v0 + vv;
        const float z = warp_dot(W + (int64_t)v * d, h_s, d, lane);
        if (lane == 0) dz_s[vv] = gk * ((v == y ? 1.f : 0.f) - expf(z - l));
      }
      __syncthreads();
#pragma unroll
      for (int q = 0; q < kMaxD / kThreads; ++q) {
        const int j = threadIdx.x + q * kThreads;
        if (j < d) {
          float a = acc[q];
          for (int vv = 0; vv < vend; ++vv) a = fmaf(dz_s[vv], W[(int64_t)(v0 + vv) * d + j], a);
          acc[q] = a;
        }
      }
      __syncthreads();
    }
#pragma unroll
    for (int q = 0; q < kMaxD / kThreads; ++q) {
      const int j = threadIdx.x + q * kThreads;
      if (j < d) dH[(int64_t)k * d + j] = acc[q];
    }
  }
}

// dW: one warp per vocabulary row, selected tokens visited in order.
__global__ void __launch_bounds__(kThreads)
f32_dw_kernel(TokenCtx c, const float* __restrict__ hidden, const float* __restrict__ W, int d,
              int V, int compact, const int32_t* __restrict__ n_sel, int64_t cap,
              const float* __restrict__ lse, const float* __restrict__ g, int accumulate,
              float* __restrict__ dW) {
  const int n = (int)min((int64_t)*n_sel, cap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int v = blockIdx.x * kWarps + warp; v < V; v += gridDim.x * kWarps) {
    float w[kRegs], acc[kRegs];
#pragma unroll
    for (int q = 0; q < kRegs; ++q) {
      const int j = lane + 32 * q;
      w[q] = j < d ? W[(int64_t)v * d + j] : 0.f;
      acc[q] = 0.f;
    }
    for (int k = 0; k < n; ++k) {
      const float gk = g[k];
      if (gk == 0.f) continue;  // contributes exactly zero
      const float* h = hidden_row(hidden, c.sel_idx, compact, k, d);
      float hv[kRegs];
      float s = 0.f;
#pragma unroll
      for (int q = 0; q < kRegs; ++q) {
        const int j = lane + 32 * q;
        hv[q] = j < d ? h[j] : 0.f;
        s = fmaf(w[q], hv[q], s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
      const int y = c.targets[c.sel_idx[k]];
      const float dz = gk * ((v == y ? 1.f : 0.f) - expf(s - lse[k]));
#pragma unroll
      for (int q = 0; q < kRegs; ++q) acc[q] = fmaf(dz, hv[q], acc[q]);
    }
#pragma unroll
    for (int q = 0; q < kRegs; ++q) {
      const int j = lane + 32 * q;
      if (j < d) {
        float* o = dW + (int64_t)v * d + j;
        *o = accumulate ? *o + acc[q] : acc[q];
      }
    }
  }
}

int check_shape(const LossArgs& a) {
  if (a.p.d > kMaxD)
    return fail(NAT_ERR_UNSUPPORTED, "the fp32 path supports d <= %d (d = %d)", kMaxD, a.p.d);
  return NAT_OK;
}

}  // namespace

size_t loss_f32_workspace_bytes(const nat_loss_params& p, int64_t cap) {
  if (p.d > kMaxD) return 0;  // not supported: see check_shape
  return sizeof(WorkspaceHead) + 2 * align_up(sizeof(float) * (size_t)cap, 256);
}

int loss_f32_fwd(const LossArgs& a) {
  int s = check_shape(a);
  if (s != NAT_OK) return s;
  F32Ws w = carve(a.workspace, a.cap);
  NAT_CUDA(cudaMemsetAsync(w.head, 0, sizeof(WorkspaceHead), a.stream));
  const TokenCtx c = make_token_ctx(a, &w.head->status);
  if (a.cap > 0) {
    const int grid = (int)min((int64_t)4096, a.cap);
    f32_fwd_kernel<<<grid, kThreads, sizeof(float) * a.p.d, a.stream>>>(
        c, (const float*)a.hidden, (const float*)a.W, a.p.d, a.p.V, a.p.hidden_is_compact, a.n_sel,
        a.cap, a.logp, a.lse, w.term);
    NAT_LAUNCH_CHECK("f32_fwd_kernel");
  }
  return launch_loss_reduce(w.term, a.n_sel, a.cap, a.loss, w.head, a.stream);
}

int loss_f32_bwd(const LossArgs& a) {
  int s = check_shape(a);
  if (s != NAT_OK) return s;
  F32Ws w = carve(a.workspace, a.cap);
  NAT_CUDA(cudaMemsetAsync(w.head, 0, sizeof(WorkspaceHead), a.stream));
  const TokenCtx c = make_token_ctx(a, &w.head->status);
  s = launch_grad_coeff(c, a.logp, a.n_sel, a.cap, a.dloss, w.g, a.stream);
  if (s != NAT_OK) return s;
  if (a.cap > 0) {
    const int grid = (int)min((int64_t)4096, a.cap);
    f32_dh_kernel<<<grid, kThreads, sizeof(float) * a.p.d, a.stream>>>(
        c, (const float*)a.hidden, (const float*)a.W, a.p.d, a.p.V, a.p.hidden_is_compact, a.n_sel,
        a.cap, a.lse, w.g, (float*)a.dHidden);
    NAT_LAUNCH_CHECK("f32_dh_kernel");
  }
  const int grid = min(4096, (a.p.V + kWarps - 1) / kWarps);
  f32_dw_kernel<<<grid, kThreads, 0, a.stream>>>(c, (const float*)a.hidden, (const float*)a.W,
                                                 a.p.d, a.p.V, a.p.hidden_is_compact, a.n_sel,
                                                 a.cap, a.lse, w.g, a.p.accumulate_dW, a.dW);
  NAT_LAUNCH_CHECK("f32_dw_kernel");
  return NAT_OK;
}

// The fp32 path has no single-pass variant: forward, then backward.
int loss_f32_fwd_bwd(const LossArgs& a) {
  int s = loss_f32_fwd(a);
  if (s != NAT_OK) return s;
  return loss_f32_bwd(a);
}

}  // namespace nat
