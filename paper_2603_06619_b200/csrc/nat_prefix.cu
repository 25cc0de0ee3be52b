// Prefix-structured selection: compaction straight from the cut lengths (no mask read),
// and Random Prefix Cutting under a caller-given cut law, whose survival function is the
// suffix sum of the law (a scan over the packed stream).
//
// Both are bound by HBM traffic.  nat_compact_prefix writes 8 bytes per selected token and
// reads only the B cut lengths.  nat_select_cutlaw reads the law twice (4 bytes per token
// each: chunk sums with the local prefixes at the response starts, final pass) and writes
// mask and pi (5 bytes per token); all sums are exact 64-bit integers of fixed-point
// masses, so the result does not depend on how the scan is split over chunks and threads.
#include <cstdint>

#include "nat_common.cuh"
#include "nat_stream.cuh"

namespace nat {
namespace {

// ------------------------------------------------ compaction of prefix masks
// sel_offsets = exclusive scan of min(max(cut_len, 0), T_i) over the responses (one block).
__global__ void __launch_bounds__(1024)
prefix_scan_kernel(int B, const int32_t* __restrict__ cu, const int32_t* __restrict__ cut_len,
                   int32_t* __restrict__ sel_offsets, int32_t* __restrict__ n_sel) {
  __shared__ int warp_tot[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int carry = 0;
  for (int base = 0, tile = 0; base < B; base += 1024, ++tile) {
    const int i = base + (int)threadIdx.x;
    int v = 0;
    if (i < B) {
      const int T = cu[i + 1] - cu[i];
      v = min(max(cut_len[i], 0), T);
    }
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    int* tot = warp_tot[tile & 1];
    if (lane == 31) tot[warp] = incl;
    __syncthreads();
    const int wt = tot[lane];
    int wincl = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, wincl, o);
      if (lane >= o) wincl += up;
    }
    const int tile_total = __shfl_sync(0xFFFFFFFFu, wincl, 31);
    const int warp_excl = __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
    if (i < B) sel_offsets[i] = carry + warp_excl + incl - v;
    carry += tile_total;
  }
  if (threadIdx.x == 0) {
    sel_offsets[B] = carry;
    *n_sel = carry;
  }
}

// One block per 4096 consecutive output slots; a thread writes four groups of four slots so
// that every warp store covers 512 contiguous bytes of each list.
__global__ void __launch_bounds__(kSelThreads)
prefix_write_kernel(int B, const int32_t* __restrict__ cu, const int32_t* __restrict__ so,
                    const int32_t* __restrict__ n_sel, int64_t cap, int32_t* __restrict__ sel_idx,
                    int32_t* __restrict__ sel_resp) {
  __shared__ int range_s[2];
  const int64_t n = min((int64_t)*n_sel, cap);
  const int64_t k0 = (int64_t)blockIdx.x * kSelBlockTokens;
  if (k0 >= n) return;
  const int64_t k_last = min(k0 + (int64_t)kSelBlockTokens, n) - 1;
  if (threadIdx.x < 32) {  // responses that own the block's first and last slot
    const int ub0 = warp_upper_bound(so, B, k0, 0);
    const int ub1 = warp_upper_bound(so, B, k_last, ub0);
    if (threadIdx.x == 0) {
      range_s[0] = ub0 - 1;
      range_s[1] = ub1 - 1;
    }
  }
  __syncthreads();
  const int r0 = range_s[0], r1 = range_s[1];
  const bool one_owner = (r0 == r1);
  const int base0 = one_owner ? cu[r0] - so[r0] : 0;  // idx = k + base0 when one response owns all
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(sel_idx) |
                        reinterpret_cast<uintptr_t>(sel_resp)) & 15u) == 0;
#pragma unroll
  for (int j = 0; j < kTokPerThread / 4; ++j) {
    const int64_t k = k0 + 4 * (int64_t)(j * kSelThreads + (int)threadIdx.x);
    if (k > k_last) continue;
    int idx[4], rsp[4];
    if (one_owner) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        idx[e] = (int)(k + e) + base0;
        rsp[e] = r0;
      }
    } else {
      int i = owner_between(so, r0, r1, k);
      int next = so[i + 1];
      int shift = cu[i] - so[i];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (k + e <= k_last) {
          while (k + e >= next) {  // skips responses with nothing selected
            ++i;
            next = so[i + 1];
            shift = cu[i] - so[i];
          }
        }
        idx[e] = (int)(k + e) + shift;
        rsp[e] = i;
      }
    }
    if (vec_ok && k + 3 <= k_last) {
      *reinterpret_cast<int4*>(sel_idx + k) = make_int4(idx[0], idx[1], idx[2], idx[3]);
      *reinterpret_cast<int4*>(sel_resp + k) = make_int4(rsp[0], rsp[1], rsp[2], rsp[3]);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (k + e <= k_last) {
          sel_idx[k + e] = idx[e];
          sel_resp[k + e] = rsp[e];
        }
    }
  }
}

// ------------------------------------------------------------- cut laws
// Fixed-point mass of one token: min(floor(q 2^32), 2^32 - 1) for q > 0, else 0 (NaN and
// negative masses count as 0).  Taken from the float's bits with integer operations only
// (a float-to-integer conversion instruction runs at a sixteenth of their rate): for
// 0 < q < 1, q = m 2^(e - 150) with the 24-bit significand m, so floor(q 2^32) is
// (m 2^8) >> (126 - e), a 32-bit value shifted right; the shift instruction yields 0 for
// amounts of 32 and more, which covers the tiny masses (subnormals included, whose missing
// hidden bit no longer matters there).
__device__ __forceinline__ uint32_t cutlaw_count(float q) {
  const uint32_t bits = __float_as_uint(q);
  const uint32_t e = bits >> 23;                   // biased exponent where q > 0
  const uint32_t m8 = (bits << 8) | 0x80000000u;   // significand with its hidden bit, times 2^8
  uint32_t r;
  asm("shr.u32 %0, %1, %2;" : "=r"(r) : "r"(m8), "r"(126u - e));  // amounts >= 32 give 0
  if (e >= 127u) r = 0xFFFFFFFFu;                  // q >= 1 (infinity included)
  return q > 0.f ? r : 0u;                         // zero, negative, NaN
}

__device__ __forceinline__ void load_counts(const float* __restrict__ q, int64_t n0, int64_t n_tot,
                                            uint32_t* k) {
  if (n0 + kTokPerThread <= n_tot) {
#pragma unroll
    for (int v = 0; v < kTokPerThread / 4; ++v) {
      const float4 f = __ldg(reinterpret_cast<const float4*>(q + n0) + v);
      k[4 * v] = cutlaw_count(f.x);
      k[4 * v + 1] = cutlaw_count(f.y);
      k[4 * v + 2] = cutlaw_count(f.z);
      k[4 * v + 3] = cutlaw_count(f.w);
    }
  } else {
#pragma unroll
    for (int j = 0; j < kTokPerThread; ++j) k[j] = (n0 + j < n_tot) ? cutlaw_count(q[n0 + j]) : 0u;
  }
}

// Sum over the block's threads of `v`; every thread gets the exclusive prefix of its own
// value and (through *total) the block's sum.
__device__ __forceinline__ unsigned long long block_excl_scan(unsigned long long v,
                                                              unsigned long long* warp_tot,
                                                              unsigned long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  unsigned long long before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kSelThreads / 32; ++w) {
    const unsigned long long t = warp_tot[w];
    if (w < warp) before += t;
    all += t;
  }
  *total = all;
  return before + incl - v;
}

// Pass 1: the sum of the counts of each 4096-token chunk and, for every response that starts
// strictly inside the chunk, the sum of the chunk's counts before its first token (the
// chunk's counts are kept in shared memory so that a start in the middle of a thread's 16
// tokens can be resolved).  A start on a chunk boundary needs no such local part.
__global__ void __launch_bounds__(kSelThreads)
cutlaw_sum_kernel(int B, const int32_t* __restrict__ cu, const float* __restrict__ q,
                  int64_t n_tot, unsigned long long* __restrict__ chunk_sum,
                  unsigned long long* __restrict__ rlocal) {
  __shared__ unsigned long long warp_tot[kSelThreads / 32];
  __shared__ unsigned long long thread_excl[kSelThreads];
  __shared__ uint32_t k_s[kSelThreads * kPiPad];  // 17 slots per thread: no bank conflicts
  __shared__ int first_s;
  const int64_t chunk0 = (int64_t)blockIdx.x * kSelBlockTokens;
  const int64_t chunk_lim = chunk0 + (int64_t)kSelBlockTokens;  // starts inside: (chunk0, chunk_lim)
  if (threadIdx.x < 32) {  // first response whose start is > chunk0
    int w0, first_in = 0;
    const int64_t v = cu_window(cu, B, chunk0, n_tot, &w0);
    if (!window_first(__ballot_sync(0xFFFFFFFFu, v > chunk0), w0, &first_in))
      first_in = warp_upper_bound(cu, B, chunk0, 0);
    if (threadIdx.x == 0) first_s = first_in;
  }
  const int64_t n0 = chunk0 + (int64_t)threadIdx.x * kTokPerThread;
  uint32_t k[kTokPerThread];
  unsigned long long s = 0;
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) k[j] = 0;
  if (n0 < n_tot) load_counts(q, n0, n_tot, k);
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) s += k[j];
  unsigned long long total;
  const unsigned long long excl = block_excl_scan(s, warp_tot, &total);  // has a __syncthreads
  if (threadIdx.x == 0) chunk_sum[blockIdx.x] = total;
  const int first_in = first_s;
  // block-uniform: no response starts strictly inside this chunk
  if (first_in > B || (int64_t)cu[first_in] >= chunk_lim) return;
  thread_excl[threadIdx.x] = excl;
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) k_s[threadIdx.x * kPiPad + j] = k[j];
  __syncthreads();
  for (int i = first_in + (int)threadIdx.x; i <= B; i += kSelThreads) {
    const int64_t n = cu[i];
    if (n >= chunk_lim) break;
    const int rel = (int)(n - chunk0);  // 1 .. 4095; counts past the stream's end are zero
    const int t = rel / kTokPerThread, j = rel % kTokPerThread;
    unsigned long long g = thread_excl[t];
    for (int e = 0; e < j; ++e) g += k_s[t * kPiPad + e];
    rlocal[i] = g;
  }
}

// Pass 2: exclusive scan of the chunk sums in place by one block; total to chunk_sum[n_chunks].
__global__ void __launch_bounds__(1024)
cutlaw_scan_kernel(unsigned long long* __restrict__ chunk_sum, int n_chunks) {
  __shared__ unsigned long long warp_tot[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long carry = 0;
  for (int base = 0, tile = 0; base < n_chunks; base += 1024, ++tile) {
    const int c = base + (int)threadIdx.x;
    const unsigned long long v = c < n_chunks ? chunk_sum[c] : 0ull;
    unsigned long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    unsigned long long* tot = warp_tot[tile & 1];
    if (lane == 31) tot[warp] = incl;
    __syncthreads();
    const unsigned long long wt = tot[lane];
    unsigned long long wincl = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, wincl, o);
      if (lane >= o) wincl += up;
    }
    const unsigned long long tile_total = __shfl_sync(0xFFFFFFFFu, wincl, 31);
    const unsigned long long warp_excl = __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
    if (c < n_chunks) chunk_sum[c] = carry + warp_excl + incl - v;
    carry += tile_total;
  }
  if (threadIdx.x == 0) chunk_sum[n_chunks] = carry;
}

struct CutConst {
  uint32_t k0, k1, off_lo, resp_base;
};

// Pass 3: G[cu_i], the sum of all counts before the first token of response i: the scanned
// sum of the chunks before the one that holds cu_i plus the local part of pass 1 (none when
// cu_i sits on a chunk boundary; chunk_off has one entry past the last chunk, the grand
// total, for starts at the stream's end), and the response's 64-bit draw.  One thread per
// response.
__global__ void __launch_bounds__(256)
cutlaw_starts_kernel(CutConst c, int B, const int32_t* __restrict__ cu,
                     const unsigned long long* __restrict__ chunk_off,
                     unsigned long long* __restrict__ rstart,
                     unsigned long long* __restrict__ udraw) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i > B) return;
  const int64_t n = cu[i];
  const unsigned long long local = (n % kSelBlockTokens) != 0 ? rstart[i] : 0ull;
  rstart[i] = chunk_off[n / kSelBlockTokens] + local;
  if (i < B) {
    const Philox4 x = philox4x32_10(0u, c.resp_base + (uint32_t)i, 3u, c.off_lo, c.k0, c.k1);
    udraw[i] = ((unsigned long long)x.y << 32) | (unsigned long long)x.x;
  }
}

// double(x), correctly rounded.  Below 2^52 the value is exact and comes from one integer
// OR and one addition (2^52 + x has x in its low significand bits); the conversion
// instruction, which is slow, is left to the counts that large.
__device__ __forceinline__ double below_2p52_to_double(unsigned long long x) {
  return __dadd_rn(__longlong_as_double((long long)(0x4330000000000000ull | x)),
                   -4503599627370496.0);
}

__device__ __forceinline__ double u64_to_double(unsigned long long x) {
  if (x < (1ull << 52)) return below_2p52_to_double(x);
  return __ull2double_rn(x);
}

// Pass 4: survival counts S_t = S_1 - (G[n] - G[cu_i]), the draw of each response, mask, pi
// and the cut lengths.  One thread per 16 consecutive tokens.
__global__ void __launch_bounds__(kSelThreads, 4)
cutlaw_final_kernel(int B, const int32_t* __restrict__ cu, int64_t n_tot,
                    const float* __restrict__ q, const unsigned long long* __restrict__ chunk_off,
                    const unsigned long long* __restrict__ rstart,
                    const unsigned long long* __restrict__ udraw, uint8_t* __restrict__ mask,
                    float* __restrict__ pi, int32_t* __restrict__ cut_len) {
  __shared__ unsigned long long warp_tot[kSelThreads / 32];
  __shared__ float pi_s[kSelThreads * kPiPad];
  __shared__ int range_s[2];
  const int64_t nb0 = (int64_t)blockIdx.x * kSelBlockTokens;
  const int cnt_block = (int)min((int64_t)kSelBlockTokens, n_tot - nb0);
  if (threadIdx.x < 32) {  // responses that own the block's first and last token
    const int64_t last = nb0 + cnt_block - 1;
    int w0, ub0 = 0, ub1 = 0;
    const int64_t v = cu_window(cu, B, nb0, n_tot, &w0);
    const bool hit = window_first(__ballot_sync(0xFFFFFFFFu, v > nb0), w0, &ub0) &&
                     window_first(__ballot_sync(0xFFFFFFFFu, v > last), w0, &ub1);
    if (!hit) {
      ub0 = warp_upper_bound(cu, B, nb0, 0);
      ub1 = warp_upper_bound(cu, B, last, ub0);
    }
    if (threadIdx.x == 0) {
      range_s[0] = ub0 - 1;
      range_s[1] = ub1 - 1;
    }
  }
  const int64_t n0 = nb0 + (int64_t)threadIdx.x * kTokPerThread;
  const bool active = n0 < n_tot;
  const int cnt = active ? (int)min((int64_t)kTokPerThread, n_tot - n0) : 0;
  uint32_t k[kTokPerThread];
  unsigned long long s = 0;
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) k[j] = 0;
  if (active) load_counts(q, n0, n_tot, k);
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) s += k[j];
  unsigned long long total;
  const unsigned long long excl = block_excl_scan(s, warp_tot, &total);  // has a __syncthreads
  if (active) {
    unsigned long long G = chunk_off[blockIdx.x] + excl;  // sum of all counts before token n0
    int i = owner_between(cu, range_s[0], range_s[1], n0);
    int64_t start = cu[i], end = cu[i + 1];
    // St: the survival count of the current token, stepped down by its own count afterwards
    unsigned long long S1 = 0, r = 0, St = 0;
    double inv_total = 1.0;
    auto enter_response = [&](unsigned long long before) {  // `before`: counts preceding the token
      const unsigned long long g0 = rstart[i];
      S1 = rstart[i + 1] - g0;
      St = S1 - (before - g0);
      r = __umul64hi(udraw[i], S1);
      inv_total = __drcp_rn(u64_to_double(S1));
    };
    enter_response(G);
    uint32_t bits = 0;
    float* pr = pi_s + threadIdx.x * kPiPad;
    if (cnt == kTokPerThread && n0 + kTokPerThread <= end && S1 != 0ull) {
      // the usual case: the thread's 16 tokens lie inside one response whose law has mass;
      // every survival count is at most S1, so one test picks the conversion for all of them
      if (S1 < (1ull << 52)) {
#pragma unroll
        for (int j = 0; j < kTokPerThread; ++j) {
          bits |= (St > r ? 1u : 0u) << j;
          pr[j] = __double2float_rn(__dmul_rn(below_2p52_to_double(St), inv_total));
          St -= k[j];
        }
      } else {
#pragma unroll
        for (int j = 0; j < kTokPerThread; ++j) {
          bits |= (St > r ? 1u : 0u) << j;
          pr[j] = __double2float_rn(__dmul_rn(u64_to_double(St), inv_total));
          St -= k[j];
        }
      }
      // the kept tokens are a prefix of the response; this thread holds its last one when
      // some but not all of its tokens are kept, or all are and the next token (St is its
      // survival count by now) is past the end or not kept
      if (bits != 0u && (bits != 0xFFFFu || n0 + kTokPerThread == end || !(St > r)))
        cut_len[i] = (int32_t)(n0 - start) + __popc(bits);
    } else {
#pragma unroll
      for (int j = 0; j < kTokPerThread; ++j) {
        float pv = 0.f;
        if (j < cnt) {
          const int64_t n = n0 + j;
          if (n >= end) {
            while (n >= end) {  // skips empty responses too
              ++i;
              start = end;
              end = cu[i + 1];
            }
            enter_response(G);
          }
          if (S1 == 0ull) {  // a law without mass: the response is kept whole
            bits |= 1u << j;
            pv = 1.f;
            if (n + 1 == end) cut_len[i] = (int32_t)(end - start);
          } else {
            const bool keep = St > r;
            const unsigned long long next = St - k[j];  // survival count of the following token
            bits |= (keep ? 1u : 0u) << j;
            pv = __double2float_rn(__dmul_rn(u64_to_double(St), inv_total));
            // last kept token of the response: the next one is past the end or not kept
            if (keep && (n + 1 == end || !(next > r))) cut_len[i] = (int32_t)(n - start) + 1;
            St = next;
          }
        }
        pr[j] = pv;
        G += k[j];
      }
    }
    if (cnt == kTokPerThread) {
      *reinterpret_cast<uint4*>(mask + n0) = bits_to_bytes(bits);
    } else {
      for (int j = 0; j < cnt; ++j) mask[n0 + j] = (uint8_t)((bits >> j) & 1u);
    }
  }
  __syncthreads();
  // pi: element e of the block sits at pi_s[(e / 16) * 17 + e % 16]
  if (cnt_block == kSelBlockTokens) {
#pragma unroll
    for (int v = 0; v < kTokPerThread / 4; ++v) {
      const int e = (v * kSelThreads + threadIdx.x) * 4;
      const float* src = pi_s + (e / kTokPerThread) * kPiPad + (e % kTokPerThread);
      *reinterpret_cast<float4*>(pi + nb0 + e) = make_float4(src[0], src[1], src[2], src[3]);
    }
  } else {
    for (int e = threadIdx.x; e < cnt_block; e += kSelThreads)
      pi[nb0 + e] = pi_s[(e / kTokPerThread) * kPiPad + (e % kTokPerThread)];
  }
}

}  // namespace
}  // namespace nat

extern "C" {

int nat_compact_prefix(int32_t B, const int32_t* cu_seqlens, int64_t n_tot,
                       const int32_t* cut_len, int32_t* sel_idx, int32_t* sel_resp,
                       int32_t* sel_offsets, int32_t* n_sel, int64_t cap, void* stream_) {
  using namespace nat;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0 || cap < 0)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_prefix: negative size");
  if (n_tot > 0x7FFFFFFFll)
    return fail(NAT_ERR_UNSUPPORTED, "nat_compact_prefix: n_tot exceeds int32");
  if (!cu_seqlens || !sel_offsets || !n_sel || (B > 0 && !cut_len))
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_prefix: null pointer");
  if (cap > 0 && (!sel_idx || !sel_resp))
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_prefix: null list");
  prefix_scan_kernel<<<1, 1024, 0, stream>>>(B, cu_seqlens, cut_len, sel_offsets, n_sel);
  NAT_LAUNCH_CHECK("prefix_scan_kernel");
  const int64_t slots = n_tot < cap ? n_tot : cap;  // at most this many tokens are listed
  if (slots > 0) {
    const unsigned grid = (unsigned)((slots + kSelBlockTokens - 1) / kSelBlockTokens);
    prefix_write_kernel<<<grid, kSelThreads, 0, stream>>>(B, cu_seqlens, sel_offsets, n_sel, cap,
                                                          sel_idx, sel_resp);
    NAT_LAUNCH_CHECK("prefix_write_kernel");
  }
  return NAT_OK;
}

size_t nat_select_cutlaw_workspace_bytes(int32_t B, int64_t n_tot) {
  if (B < 0 || n_tot < 0) return 0;
  const int64_t chunks = (n_tot + nat::kSelBlockTokens - 1) / nat::kSelBlockTokens;
  return nat::align_up((size_t)(chunks + 1) * 8, 256) + 2 * nat::align_up((size_t)(B + 1) * 8, 256);
}

int nat_select_cutlaw(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const float* q,
                      uint64_t seed, uint64_t offset, int32_t resp_base, uint8_t* mask, float* pi,
                      int32_t* cut_len, void* workspace, size_t workspace_bytes, void* stream_) {
  using namespace nat;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select_cutlaw: negative size");
  if (n_tot > 0x7FFFFFFFll)
    return fail(NAT_ERR_UNSUPPORTED, "nat_select_cutlaw: n_tot exceeds int32");
  if (resp_base < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select_cutlaw: resp_base < 0");
  if (!cu_seqlens || (B > 0 && !cut_len) || (n_tot > 0 && (!q || !mask || !pi)))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_cutlaw: null pointer");
  if (((uintptr_t)q & 15u) || ((uintptr_t)mask & 15u) || ((uintptr_t)pi & 15u))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_cutlaw: q, mask and pi must be 16-byte aligned");
  const size_t need = nat_select_cutlaw_workspace_bytes(B, n_tot);
  if (!workspace || workspace_bytes < need)
    return fail(NAT_ERR_CAPACITY, "nat_select_cutlaw: workspace too small (%zu < %zu)",
                workspace_bytes, need);
  if ((uintptr_t)workspace & 255u)
    return fail(NAT_ERR_INVALID_ARG, "nat_select_cutlaw: workspace must be 256-byte aligned");
  if (B == 0) return NAT_OK;
  const int n_chunks = (int)((n_tot + kSelBlockTokens - 1) / kSelBlockTokens);
  unsigned long long* chunk_off = reinterpret_cast<unsigned long long*>(workspace);
  unsigned long long* rstart = reinterpret_cast<unsigned long long*>(
      reinterpret_cast<char*>(workspace) + align_up((size_t)(n_chunks + 1) * 8, 256));
  unsigned long long* udraw = rstart + align_up((size_t)(B + 1) * 8, 256) / 8;
  NAT_CUDA(cudaMemsetAsync(cut_len, 0, sizeof(int32_t) * (size_t)B, stream));
  if (n_chunks == 0) return NAT_OK;  // every response is empty
  CutConst c;
  c.k0 = (uint32_t)(seed & 0xFFFFFFFFull);
  c.k1 = (uint32_t)((seed >> 32) ^ (offset >> 32));
  c.off_lo = (uint32_t)(offset & 0xFFFFFFFFull);
  c.resp_base = (uint32_t)resp_base;
  cutlaw_sum_kernel<<<n_chunks, kSelThreads, 0, stream>>>(B, cu_seqlens, q, n_tot, chunk_off,
                                                          rstart);
  NAT_LAUNCH_CHECK("cutlaw_sum_kernel");
  cutlaw_scan_kernel<<<1, 1024, 0, stream>>>(chunk_off, n_chunks);
  NAT_LAUNCH_CHECK("cutlaw_scan_kernel");
  cutlaw_starts_kernel<<<(B + 256) / 256, 256, 0, stream>>>(c, B, cu_seqlens, chunk_off, rstart,
                                                            udraw);
  NAT_LAUNCH_CHECK("cutlaw_starts_kernel");
  cutlaw_final_kernel<<<n_chunks, kSelThreads, 0, stream>>>(B, cu_seqlens, n_tot, q, chunk_off,
                                                            rstart, udraw, mask, pi, cut_len);
  NAT_LAUNCH_CHECK("cutlaw_final_kernel");
  return NAT_OK;
}

}  // extern "C"
