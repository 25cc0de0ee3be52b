// Test probe: the bounded mbarrier wait of the tensor-core kernels, exercised on a barrier
// that nobody ever arrives at.  No TMA copy and no MMA is in flight; the kernel must come
// back by itself with the block's abort flag raised.
//   warp 0 waits with a 2 ms limit          -> gives up, raises the flag
//   warp 1 waits with a 2 s limit           -> returns early because it sees the flag
//   warp 2 waits on a barrier that IS signalled -> succeeds (the wait itself works)
#include <cstdint>
#include <cuda_runtime.h>

#include "nat_tc.cuh"

namespace tc = nat::tc;

__global__ void bounded_wait_kernel(uint32_t* out) {
  __shared__ uint64_t never_bar, done_bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&never_bar, 1);
    tc::mbar_init(&done_bar, 1);
    abort_flag = 0u;
    tc::fence_barrier_init();
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t t0 = tc::global_timer_ns();
  if (lane == 0) {
    if (warp == 0) {
      const bool ok = tc::mbar_wait(&never_bar, 0u, &abort_flag, 2000000ull);
      out[0] = ok ? 1u : 0u;
      out[1] = (uint32_t)((tc::global_timer_ns() - t0) / 1000ull);  // microseconds waited
    } else if (warp == 1) {
      const bool ok = tc::mbar_wait(&never_bar, 0u, &abort_flag, 2000000000ull);
      out[2] = ok ? 1u : 0u;
      out[3] = (uint32_t)((tc::global_timer_ns() - t0) / 1000ull);
    } else if (warp == 2) {
      tc::mbar_arrive(&done_bar);
      const bool ok = tc::mbar_wait(&done_bar, 0u, &abort_flag, 2000000ull);
      out[4] = ok ? 1u : 0u;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) out[5] = abort_flag;
}

extern "C" int bounded_wait_probe(uint32_t* host_out /* [6] */) {
  uint32_t* dev = nullptr;
  if (cudaMalloc(&dev, 6 * sizeof(uint32_t)) != cudaSuccess) return -1;
  cudaMemset(dev, 0xFF, 6 * sizeof(uint32_t));
  bounded_wait_kernel<<<1, 96>>>(dev);
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(host_out, dev, 6 * sizeof(uint32_t), cudaMemcpyDeviceToHost);
  cudaFree(dev);
  return e == cudaSuccess ? 0 : -2;
}
