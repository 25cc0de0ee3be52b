// Group-relative advantages, token selection (URS / RPC / deterministic
// truncation) and stream compaction of the selected indices.
//
// These kernels are bound by HBM traffic (select writes 5 bytes per token and
// reads nothing; compact reads the mask twice and writes 8 bytes per selected
// token), so they use 16-byte accesses: one thread owns 16 consecutive tokens.
// Floating-point steps that must agree bit for bit with a plain IEEE
// evaluation use the explicit round-to-nearest intrinsics, which the compiler
// never contracts into fused multiply-adds.
#include <climits>
#include <cstdint>
#include <mutex>

#include "nat_common.cuh"
#include "nat_stream.cuh"

namespace nat {
namespace {

// ------------------------------------------------------------ advantages
__global__ void grpo_adv_kernel(int P, int G, const float* __restrict__ rewards, float eps,
                                float* __restrict__ adv) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= P) return;
  const float* R = rewards + (size_t)g * G;
  double s = 0.0;
  for (int j = 0; j < G; ++j) s = __dadd_rn(s, (double)R[j]);
  const double mu = __ddiv_rn(s, (double)G);
  double v = 0.0;
  for (int j = 0; j < G; ++j) {
    const double dlt = __dsub_rn((double)R[j], mu);
    v = __dadd_rn(v, __dmul_rn(dlt, dlt));
  }
  const double sigma = __dsqrt_rn(__ddiv_rn(v, (double)G));
  const double den = __dadd_rn(sigma, (double)eps);
  for (int j = 0; j < G; ++j)
    adv[(size_t)g * G + j] = (float)__ddiv_rn(__dsub_rn((double)R[j], mu), den);
}

// -------------------------------------------------------------- selection

struct SelConst {
  int mode;
  int min_cut;
  double beta;
  uint64_t thr;    // URS threshold, 1..2^32
  float pi_urs;    // thr / 2^32
  uint32_t k0, k1, off_lo;
  uint32_t resp_base;  // global index of the first response of cu (draws are keyed by it)
};

// One thread per response: the RPC cut L_i (or the truncation length K_i).
__global__ void cut_kernel(SelConst c, int B, const int32_t* __restrict__ cu,
                           int32_t* __restrict__ cut_len) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B) return;
  const int T = cu[i + 1] - cu[i];
  int L = 0;
  if (T > 0) {
    if (c.mode == NAT_SEL_RPC) {
      const int C = min(max(c.min_cut, 1), T);
      const uint64_t n = (uint64_t)(T - C + 1);
      const Philox4 r = philox4x32_10(0u, c.resp_base + (uint32_t)i, 1u, c.off_lo, c.k0, c.k1);
      const uint64_t u = ((uint64_t)r.y << 32) | (uint64_t)r.x;
      L = C + (int)__umul64hi(u, n);
    } else {
      L = max(1, (int)floor(__dmul_rn(c.beta, (double)T)));
    }
  }
  cut_len[i] = L;
}

// One block per 4096 consecutive packed tokens, one thread per 16 of them.  The mask
// leaves as one 16-byte store per thread and pi as 16-byte stores that cover 512
// contiguous bytes per warp.
//
// URS.  Token t of response i uses word (t-1) % 4 of Philox block (t-1) / 4, so 16
// consecutive tokens of one response need four blocks when they start on a block
// boundary and a fifth otherwise.  A thread evaluates the four blocks that start at or
// before its first token; the up to three draws it still lacks are the first block of the
// thread after it (same response, same alignment) and arrive by a warp shuffle, or through
// shared memory from the next warp.  Only a thread whose successor cannot help (end of the
// block, or a response boundary) evaluates a fifth block.  pi is a constant.
//
// RPC / truncation.  No draws per token; pi = (T-t+1)/(T-C+1) must be the correctly
// rounded float32 quotient.  With y = RN(1/b) computed once per response, q0 = RN(a y),
// r = a - q0 b (exact in an FMA) and q = RN(q0 + r y) is the correctly rounded a/b
// (Markstein's theorem on FMA division); three operations per token instead of a division.

__device__ __forceinline__ float div_rn_by(float a, float b, float rcp_b) {
  const float q0 = __fmul_rn(a, rcp_b);
  const float r = __fmaf_rn(-q0, b, a);
  return __fmaf_rn(r, rcp_b, q0);
}

// Bit w set iff word w of the block lies below the threshold (1 .. 2^32; at 2^32 every
// word does: the test is the same for all threads, and below it the compares are 32-bit).
__device__ __forceinline__ uint32_t philox_below(const Philox4& r, uint64_t thr) {
  if ((thr >> 32) != 0ull) return 0xFu;
  const uint32_t t = (uint32_t)thr;
  return (r.x < t ? 1u : 0u) | (r.y < t ? 2u : 0u) | (r.z < t ? 4u : 0u) | (r.w < t ? 8u : 0u);
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(SelConst c, int B, const int32_t* __restrict__ cu, int64_t n_tot,
              const int32_t* __restrict__ cut_len, uint8_t* __restrict__ mask,
              float* __restrict__ pi) {
  __shared__ float pi_s[kSelThreads * kPiPad];
  __shared__ int range_s[2];
  __shared__ int edge_tag_s[kSelThreads / 32 + 1];
  __shared__ uint32_t edge_nib_s[kSelThreads / 32 + 1];
  const int64_t nb0 = (int64_t)blockIdx.x * kSelBlockTokens;
  const int cnt_block = (int)min((int64_t)kSelBlockTokens, n_tot - nb0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) {  // responses that own the block's first and last token
    const int64_t last = nb0 + cnt_block - 1;
    int w0, ub0 = 0, ub1 = 0;
    const int64_t v = cu_window(cu, B, nb0, n_tot, &w0);
    const bool hit = window_first(__ballot_sync(0xFFFFFFFFu, v > nb0), w0, &ub0) &&
                     window_first(__ballot_sync(0xFFFFFFFFu, v > last), w0, &ub1);
    if (!hit) {
      ub0 = warp_upper_bound(cu, B, nb0, 0);
      ub1 = warp_upper_bound(cu, B, last, ub0);
    }
    const int r0 = ub0 - 1, r1 = ub1 - 1;
    if (lane == 0) {
      range_s[0] = r0;
      range_s[1] = r1;
      edge_tag_s[kSelThreads / 32] = -1;  // nobody follows the last warp
    }
  }
  __syncthreads();
  const int64_t n0 = nb0 + (int64_t)threadIdx.x * kTokPerThread;
  const bool active = n0 < n_tot;
  const int cnt = active ? (int)min((int64_t)kTokPerThread, n_tot - n0) : 0;
  int i = 0;
  int64_t start = 0, end = 0;
  if (active) {
    i = owner_between(cu, range_s[0], range_s[1], n0);
    start = cu[i];
    end = cu[i + 1];
  }
  // the whole 16-token span lies inside response i
  const bool inside = active && cnt == kTokPerThread && n0 + kTokPerThread <= end;
  uint32_t bits = 0;

  if (c.mode == NAT_SEL_URS) {
    const uint32_t t0 = (uint32_t)(n0 - start);  // (position - 1) of the first token
    const uint32_t sh = t0 & 3u;
    uint32_t low = 0;                            // draws of blocks blk0 .. blk0+3, bit 4q+word
    if (inside) {
      const uint32_t blk0 = t0 >> 2;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        low |= philox_below(philox4x32_10(blk0 + q, c.resp_base + (uint32_t)i, 0u, c.off_lo, c.k0, c.k1), c.thr)
               << (4 * q);
    }
    const int tag = inside ? i : -1;
    if (lane == 0) {
      edge_tag_s[warp] = tag;
      edge_nib_s[warp] = low & 0xFu;
    }
    int next_tag = __shfl_down_sync(0xFFFFFFFFu, tag, 1);
    uint32_t next_nib = __shfl_down_sync(0xFFFFFFFFu, low, 1) & 0xFu;
    __syncthreads();
    if (lane == 31) {
      next_tag = edge_tag_s[warp + 1];
      next_nib = edge_nib_s[warp + 1];
    }
    if (inside) {
      if (sh != 0u && next_tag != i)
        next_nib = philox_below(
            philox4x32_10((t0 >> 2) + 4u, c.resp_base + (uint32_t)i, 0u, c.off_lo, c.k0, c.k1), c.thr);
      bits = ((low | (next_nib << 16)) >> sh) & 0xFFFFu;
      *reinterpret_cast<uint4*>(mask + n0) = bits_to_bytes(bits);
    } else if (active) {
      // a span that crosses a response boundary or the end of the stream: token by token
      uint32_t cached_blk = 0xFFFFFFFFu;
      int cached_resp = -1;
      Philox4 rnd = {0, 0, 0, 0};
      alignas(16) uint8_t m[kTokPerThread];
#pragma unroll
      for (int j = 0; j < kTokPerThread; ++j) {
        m[j] = 0;
        if (j < cnt) {
          const int64_t n = n0 + j;
          while (n >= end) {  // skips empty responses too
            ++i;
            start = end;
            end = cu[i + 1];
          }
          const uint32_t tj = (uint32_t)(n - start);
          const uint32_t blk = tj >> 2;
          if (blk != cached_blk || i != cached_resp) {
            rnd = philox4x32_10(blk, c.resp_base + (uint32_t)i, 0u, c.off_lo, c.k0, c.k1);
            cached_blk = blk;
            cached_resp = i;
          }
          const uint32_t word = tj & 3u;
          const uint32_t x = word == 0 ? rnd.x : word == 1 ? rnd.y : word == 2 ? rnd.z : rnd.w;
          m[j] = ((uint64_t)x < c.thr) ? 1 : 0;
        }
      }
      if (cnt == kTokPerThread) {
        *reinterpret_cast<uint4*>(mask + n0) = *reinterpret_cast<const uint4*>(m);
      } else {
        for (int j = 0; j < cnt; ++j) mask[n0 + j] = m[j];
      }
    }
    // pi is the same for every token
    if (cnt_block == kSelBlockTokens) {
      const float4 v = make_float4(c.pi_urs, c.pi_urs, c.pi_urs, c.pi_urs);
#pragma unroll
      for (int k = 0; k < kTokPerThread / 4; ++k)
        *reinterpret_cast<float4*>(pi + nb0 + (int64_t)(k * kSelThreads + threadIdx.x) * 4) = v;
    } else {
      for (int e = threadIdx.x; e < cnt_block; e += kSelThreads) pi[nb0 + e] = c.pi_urs;
    }
    return;
  }

  // ---- RPC / deterministic truncation
  if (active) {
    int L = 0, C = 0;
    float den = 1.f, rden = 1.f;
    auto enter_response = [&]() {
      L = cut_len[i];
      const int T = (int)(end - start);
      C = (c.mode == NAT_SEL_RPC) ? min(max(c.min_cut, 1), T) : T;
      den = (float)(T - C + 1);
      rden = __frcp_rn(den);
    };
    enter_response();
    float* pr = pi_s + threadIdx.x * kPiPad;
    if (inside) {
      const int T = (int)(end - start);
      const int t_first = (int)(n0 - start) + 1;
      // the kept tokens are the first L - t_first + 1 of the thread's 16 (clamped)
      const int keep = min(max(L - t_first + 1, 0), kTokPerThread);
      bits = (1u << keep) - 1u;
      // numerators T - t + 1 by exact float subtraction (integers below 2^24): one
      // int-to-float conversion per thread instead of one per token
      const float a0 = (float)(T - t_first + 1);
      const int ones = C - t_first + 1;  // tokens of the thread with t <= C
#pragma unroll
      for (int j = 0; j < kTokPerThread; ++j)
        pr[j] = (j < ones) ? 1.f : div_rn_by(a0 - (float)j, den, rden);
      *reinterpret_cast<uint4*>(mask + n0) = bits_to_bytes(bits);
    } else {
      alignas(16) uint8_t m[kTokPerThread];
#pragma unroll
      for (int j = 0; j < kTokPerThread; ++j) {
        m[j] = 0;
        float pv = 0.f;
        if (j < cnt) {
          const int64_t n = n0 + j;
          while (n >= end) {  // skips empty responses too
            ++i;
            start = end;
            end = cu[i + 1];
            if (n < end) enter_response();
          }
          const int t = (int)(n - start) + 1;
          const int T = (int)(end - start);
          m[j] = (t <= L) ? 1 : 0;
          pv = (t <= C) ? 1.f : div_rn_by((float)(T - t + 1), den, rden);
        }
        pr[j] = pv;
      }
      if (cnt == kTokPerThread) {
        *reinterpret_cast<uint4*>(mask + n0) = *reinterpret_cast<const uint4*>(m);
      } else {
        for (int j = 0; j < cnt; ++j) mask[n0 + j] = m[j];
      }
    }
  }
  __syncthreads();
  // pi: element e of the block sits at pi_s[(e / 16) * 17 + e % 16]
  if (cnt_block == kSelBlockTokens) {
#pragma unroll
    for (int k = 0; k < kTokPerThread / 4; ++k) {
      const int e = (k * kSelThreads + threadIdx.x) * 4;
      const float* src = pi_s + (e / kTokPerThread) * kPiPad + (e % kTokPerThread);
      *reinterpret_cast<float4*>(pi + nb0 + e) = make_float4(src[0], src[1], src[2], src[3]);
    }
  } else {
    for (int e = threadIdx.x; e < cnt_block; e += kSelThreads)
      pi[nb0 + e] = pi_s[(e / kTokPerThread) * kPiPad + (e % kTokPerThread)];
  }
}

// Random prefix cutting under a caller-given survival schedule: response i draws one
// uniform u = (x0 >> 8) 2^-24 (Philox counter (0, i, 2, offset_lo)); token t is kept iff
// u < surv.  One thread per 16 consecutive tokens, 16-byte loads and stores; the thread
// that sees the last kept token of a response writes its cut length.
__global__ void __launch_bounds__(kSelThreads)
select_survival_kernel(SelConst c, int B, const int32_t* __restrict__ cu, int64_t n_tot,
                       const float* __restrict__ surv, uint8_t* __restrict__ mask,
                       int32_t* __restrict__ cut_len) {
  __shared__ int range_s[2];
  const int64_t nb0 = (int64_t)blockIdx.x * kSelBlockTokens;
  if (threadIdx.x < 32) {  // responses that own the block's first and last token
    const int64_t last = min(nb0 + (int64_t)kSelBlockTokens, n_tot) - 1;
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
  __syncthreads();
  const int64_t n0 = nb0 + (int64_t)threadIdx.x * kTokPerThread;
  if (n0 >= n_tot) return;
  const int cnt = (int)min((int64_t)kTokPerThread, n_tot - n0);
  int i = owner_between(cu, range_s[0], range_s[1], n0);
  int64_t start = cu[i], end = cu[i + 1];
  auto draw = [&]() {
    const Philox4 r = philox4x32_10(0u, c.resp_base + (uint32_t)i, 2u, c.off_lo, c.k0, c.k1);
    return __fmul_rn((float)(r.x >> 8), 5.9604644775390625e-08f);  // 2^-24, exact
  };
  float u = draw();
  alignas(16) float p[kTokPerThread];
  if (cnt == kTokPerThread) {
#pragma unroll
    for (int q = 0; q < 4; ++q)
      *reinterpret_cast<float4*>(p + 4 * q) = __ldg(reinterpret_cast<const float4*>(surv + n0) + q);
  } else {
    for (int j = 0; j < kTokPerThread; ++j) p[j] = j < cnt ? surv[n0 + j] : 0.f;
  }
  alignas(16) uint8_t m[kTokPerThread];
#pragma unroll
  for (int j = 0; j < kTokPerThread; ++j) {
    m[j] = 0;
    if (j < cnt) {
      const int64_t n = n0 + j;
      while (n >= end) {
        ++i;
        start = end;
        end = cu[i + 1];
        if (n < end) u = draw();
      }
      const bool keep = u < p[j];
      m[j] = keep ? 1 : 0;
      if (keep) {
        // last kept token of the response: the next one is past the end or not kept
        const bool last = (n + 1 == end) ||
                          !(u < (j + 1 < cnt ? p[j + 1] : __ldg(surv + n + 1)));
        if (last) cut_len[i] = (int32_t)(n - start) + 1;
      }
    }
  }
  if (cnt == kTokPerThread) {
    *reinterpret_cast<uint4*>(mask + n0) = *reinterpret_cast<const uint4*>(m);
  } else {
    for (int j = 0; j < cnt; ++j) mask[n0 + j] = m[j];
  }
}

// ------------------------------------------------ packing selected rows
// dst[k, :] = src[sel_idx[k], :] (gather) or dst[sel_idx[k], :] = src[k, :] (scatter) for
// k < n_sel; rows are row_vec 16-byte vectors.  One warp per row keeps each row's
// traffic in whole 512-byte warp transactions; the kernels are bound by HBM bandwidth
// (row_bytes read + row_bytes written per selected row).
__global__ void __launch_bounds__(256)
move_rows_kernel(const uint4* __restrict__ src, int64_t row_vec,
                 const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ n_sel,
                 int64_t cap, int scatter, uint4* __restrict__ dst) {
  const int64_t n = min((int64_t)*n_sel, cap);
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t k = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); k < n;
       k += warps) {
    const int64_t row = sel_idx[k];
    const uint4* s = src + (scatter ? k : row) * row_vec;
    uint4* d = dst + (scatter ? row : k) * row_vec;
    for (int64_t j = lane; j < row_vec; j += 32) d[j] = __ldg(s + j);
  }
}

// ------------------------------------------------------------- compaction
// Pass 1: selected count of each 4096-token chunk.  Pass 2: one block scans
// the chunk counts.  Pass 3: each chunk scans its own mask and writes the
// indices, the owning responses and the per-response offsets whose boundary
// falls inside the chunk.
constexpr int kCmpThreads = 256;
constexpr int kChunk = kCmpThreads * kTokPerThread;  // 4096 tokens
constexpr int kCountChunks = 8;                      // chunks per block of the counting pass

__device__ __forceinline__ uint32_t load_mask_bits(const uint8_t* __restrict__ mask, int64_t n0,
                                                   int64_t n_tot) {
  uint32_t bits = 0;
  if (n0 + kTokPerThread <= n_tot) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask + n0));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      // byte != 0 -> its bit 7 set -> gathered into bits 0..3 (a multiply collects them)
      const uint32_t nz = ((w[q] & 0x7F7F7F7Fu) + 0x7F7F7F7Fu | w[q]) & 0x80808080u;
      bits |= (((nz >> 7) * 0x01020408u) >> 24 & 0xFu) << (4 * q);
    }
  } else {
    for (int j = 0; j < kTokPerThread; ++j)
      if (n0 + j < n_tot && mask[n0 + j] != 0) bits |= 1u << j;
  }
  return bits;
}

// Each block counts kCountChunks consecutive chunks: that many independent 16-byte loads
// per thread are in flight at once.
__global__ void __launch_bounds__(kCmpThreads)
compact_count_kernel(const uint8_t* __restrict__ mask, int64_t n_tot, int n_chunks,
                     int32_t* __restrict__ chunk_count) {
  __shared__ int warp_sum[kCountChunks][kCmpThreads / 32];
  const int chunk_first = blockIdx.x * kCountChunks;
  int c[kCountChunks];
#pragma unroll
  for (int q = 0; q < kCountChunks; ++q) {
    const int64_t n0 = (int64_t)(chunk_first + q) * kChunk + (int64_t)threadIdx.x * kTokPerThread;
    c[q] = (n0 < n_tot) ? __popc(load_mask_bits(mask, n0, n_tot)) : 0;
  }
#pragma unroll
  for (int q = 0; q < kCountChunks; ++q) {
    const int r = __reduce_add_sync(0xFFFFFFFFu, c[q]);
    if ((threadIdx.x & 31) == 0) warp_sum[q][threadIdx.x >> 5] = r;
  }
  __syncthreads();
  if (threadIdx.x < kCountChunks && chunk_first + (int)threadIdx.x < n_chunks) {
    int t = 0;
    for (int w = 0; w < kCmpThreads / 32; ++w) t += warp_sum[threadIdx.x][w];
    chunk_count[chunk_first + threadIdx.x] = t;
  }
}

// Exclusive scan of the chunk counts by a single block (in place), total to
// chunk_count[n_chunks], n_sel and sel_offsets[B].  Tiles of 4096 counts: every thread
// takes four consecutive counts with one 16-byte load (the next tile's load is issued
// before this tile's barrier), the warps scan by shuffles and meet once per tile.
__global__ void __launch_bounds__(1024)
compact_scan_kernel(int32_t* __restrict__ chunk_count, int n_chunks, int32_t* __restrict__ n_sel,
                    int32_t* __restrict__ sel_offsets, int B) {
  __shared__ int warp_tot[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_tiles = (n_chunks + 4095) / 4096;
  auto load4 = [&](int tile) {
    const int k = tile * 4096 + (int)threadIdx.x * 4;
    int4 v = make_int4(0, 0, 0, 0);
    if (k < n_chunks) v = *reinterpret_cast<const int4*>(chunk_count + k);  // padded allocation
    if (k + 1 >= n_chunks) v.y = 0;
    if (k + 2 >= n_chunks) v.z = 0;
    if (k + 3 >= n_chunks) v.w = 0;
    return v;
  };
  int carry = 0;
  int4 cur = n_tiles > 0 ? load4(0) : make_int4(0, 0, 0, 0);
  for (int tile = 0; tile < n_tiles; ++tile) {
    const int4 nxt = tile + 1 < n_tiles ? load4(tile + 1) : make_int4(0, 0, 0, 0);
    const int sum = cur.x + cur.y + cur.z + cur.w;
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += up;
    }
    int* tot = warp_tot[tile & 1];
    if (lane == 31) tot[warp] = incl;
    __syncthreads();
    // every warp scans the 32 warp totals itself
    const int wt = tot[lane];
    int wincl = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, wincl, o);
      if (lane >= o) wincl += up;
    }
    const int tile_total = __shfl_sync(0xFFFFFFFFu, wincl, 31);
    const int warp_excl = __shfl_sync(0xFFFFFFFFu, wincl - wt, warp);
    const int e0 = carry + warp_excl + incl - sum;
    const int k = tile * 4096 + (int)threadIdx.x * 4;
    if (k + 3 < n_chunks) {
      *reinterpret_cast<int4*>(chunk_count + k) =
          make_int4(e0, e0 + cur.x, e0 + cur.x + cur.y, e0 + cur.x + cur.y + cur.z);
    } else {
      if (k < n_chunks) chunk_count[k] = e0;
      if (k + 1 < n_chunks) chunk_count[k + 1] = e0 + cur.x;
      if (k + 2 < n_chunks) chunk_count[k + 2] = e0 + cur.x + cur.y;
    }
    carry += tile_total;
    cur = nxt;
  }
  if (threadIdx.x == 0) {
    chunk_count[n_chunks] = carry;
    *n_sel = carry;
    sel_offsets[B] = carry;
  }
}

// Staging index of output slot k: one spare slot after every 32 keeps both the writes
// (threads 8 or 16 slots apart) and the reads (consecutive slots) free of bank conflicts.
__device__ __forceinline__ int skew(int k) { return k + (k >> 5); }

__global__ void __launch_bounds__(kCmpThreads)
compact_write_kernel(int B, const int32_t* __restrict__ cu, int64_t n_tot,
                     const uint8_t* __restrict__ mask, const int32_t* __restrict__ chunk_offset,
                     int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_resp,
                     int32_t* __restrict__ sel_offsets, int64_t cap) {
  __shared__ int warp_tot[kCmpThreads / 32];
  __shared__ int thread_excl[kCmpThreads];
  __shared__ uint32_t thread_bits[kCmpThreads];
  __shared__ int32_t idx_s[kChunk + kChunk / 32];
  __shared__ int32_t resp_s[kChunk + kChunk / 32];
  __shared__ int range_s[3];
  const int64_t chunk0 = (int64_t)blockIdx.x * kChunk;
  const int64_t chunk_end = min(chunk0 + (int64_t)kChunk, n_tot);
  const int64_t n0 = chunk0 + (int64_t)threadIdx.x * kTokPerThread;
  const uint32_t bits = (n0 < n_tot) ? load_mask_bits(mask, n0, n_tot) : 0u;
  const int base = chunk_offset[blockIdx.x];
  if (threadIdx.x < 32) {
    // first response whose start lies in this chunk, and the responses that own the
    // chunk's first and last token
    int w0, first_in = 0, ub0 = 0, ub1 = 0;
    const int64_t v = cu_window(cu, B, chunk0, n_tot, &w0);
    const bool hit = window_first(__ballot_sync(0xFFFFFFFFu, v >= chunk0), w0, &first_in) &&
                     window_first(__ballot_sync(0xFFFFFFFFu, v > chunk0), w0, &ub0) &&
                     window_first(__ballot_sync(0xFFFFFFFFu, v > chunk_end - 1), w0, &ub1);
    if (!hit) {
      first_in = warp_upper_bound(cu, B, chunk0 - 1, 0);
      ub0 = warp_upper_bound(cu, B, chunk0, first_in);
      ub1 = warp_upper_bound(cu, B, chunk_end - 1, ub0);
    }
    if (threadIdx.x == 0) {
      range_s[0] = ub0 - 1;
      range_s[1] = ub1 - 1;
      range_s[2] = first_in;
    }
  }
  const int c = __popc(bits);
  int incl = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if ((threadIdx.x & 31) >= o) incl += up;
  }
  if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = incl;
  __syncthreads();
  int warp_excl = 0;
  for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) warp_excl += warp_tot[w];
  const int excl = base + warp_excl + incl - c;  // selected tokens before n0
  thread_excl[threadIdx.x] = excl;
  thread_bits[threadIdx.x] = bits;

  // The chunk's selected tokens are consecutive in the output lists: stage them in
  // shared memory, then write them out with coalesced 16-byte stores.  A chunk that lies
  // inside one response (the usual case for long responses) has a constant owner and
  // stages the indices only.
  const int r_first = range_s[0];
  const bool one_owner = (r_first == range_s[1]);
  if (bits != 0u) {
    int k = excl - base;
    int i = r_first;
    int64_t end = INT64_MAX;
    if (!one_owner) {
      i = owner_between(cu, r_first, range_s[1], n0);
      end = cu[i + 1];
    }
    if (n0 + kTokPerThread <= end) {  // the thread's 16 tokens have one owner
#pragma unroll
      for (int j = 0; j < kTokPerThread; ++j) {
        if ((bits >> j) & 1u) {
          idx_s[skew(k)] = (int32_t)(n0 + j);
          if (!one_owner) resp_s[skew(k)] = i;
          ++k;
        }
      }
    } else {
      uint32_t rest = bits;
      while (rest != 0u) {
        const int j = __ffs(rest) - 1;
        rest &= rest - 1u;
        const int64_t n = n0 + j;
        while (n >= end) end = cu[++i + 1];
        idx_s[skew(k)] = (int32_t)n;
        resp_s[skew(k)] = i;
        ++k;
      }
    }
  }
  __syncthreads();
  {
    int total = 0;
    for (int w = 0; w < kCmpThreads / 32; ++w) total += warp_tot[w];
    const bool vec_ok = (int64_t)base + total <= cap &&
                        ((reinterpret_cast<uintptr_t>(sel_idx) |
                          reinterpret_cast<uintptr_t>(sel_resp)) & 15u) == 0;
    if (vec_ok) {
      // slots [head, head + 4 * groups) start on a 16-byte boundary of the output lists
      const int head = min(total, (4 - (base & 3)) & 3);
      const int groups = (total - head) / 4;
      for (int g = threadIdx.x; g < groups; g += kCmpThreads) {
        const int e = head + 4 * g;
        const int4 v = make_int4(idx_s[skew(e)], idx_s[skew(e + 1)], idx_s[skew(e + 2)],
                                 idx_s[skew(e + 3)]);
        const int4 r = one_owner ? make_int4(r_first, r_first, r_first, r_first)
                                 : make_int4(resp_s[skew(e)], resp_s[skew(e + 1)],
                                             resp_s[skew(e + 2)], resp_s[skew(e + 3)]);
        *reinterpret_cast<int4*>(sel_idx + base + e) = v;
        *reinterpret_cast<int4*>(sel_resp + base + e) = r;
      }
      const int done = head + 4 * groups;
      const int rest_n = head + (total - done);  // slots before the first and after the last group
      if ((int)threadIdx.x < rest_n) {
        const int e = (int)threadIdx.x < head ? (int)threadIdx.x : done + ((int)threadIdx.x - head);
        sel_idx[base + e] = idx_s[skew(e)];
        sel_resp[base + e] = one_owner ? r_first : resp_s[skew(e)];
      }
    } else {
      for (int e = threadIdx.x; e < total; e += kCmpThreads) {
        const int64_t k = (int64_t)base + e;
        if (k < cap) {
          sel_idx[k] = idx_s[skew(e)];
          sel_resp[k] = one_owner ? r_first : resp_s[skew(e)];
        }
      }
    }
  }

  // Per-response offsets: every i with cu[i] inside this chunk (the last chunk
  // also takes the boundaries equal to n_tot).  sel_offsets[B] is the scan's.
  const bool last = (chunk_end == n_tot);
  for (int i = range_s[2] + threadIdx.x; i < B; i += kCmpThreads) {
    const int64_t n = cu[i];
    if (n > chunk_end || (n == chunk_end && !last)) break;
    if (n == n_tot) {
      // nothing after the stream's end: all selected tokens precede it
      const int t = kCmpThreads - 1;
      sel_offsets[i] = thread_excl[t] + __popc(thread_bits[t]);
    } else {
      const int rel = (int)(n - chunk0);
      const int t = rel / kTokPerThread, j = rel % kTokPerThread;
      sel_offsets[i] = thread_excl[t] + __popc(thread_bits[t] & ((1u << j) - 1u));
    }
  }
}

}  // namespace

static int select_impl(const nat_select_params* sp, int32_t B, const int32_t* cu_seqlens,
                       int64_t n_tot, uint8_t* mask, float* pi, int32_t* cut_len,
                       cudaStream_t stream) {
  if (!sp) return fail(NAT_ERR_INVALID_ARG, "nat_select: params is null");
  if (B < 0 || n_tot < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select: negative size");
  if (n_tot > 0x7FFFFFFFll) return fail(NAT_ERR_UNSUPPORTED, "nat_select: n_tot exceeds int32");
  if (!cu_seqlens) return fail(NAT_ERR_INVALID_ARG, "nat_select: cu_seqlens is null");
  if (n_tot > 0 && (!mask || !pi)) return fail(NAT_ERR_INVALID_ARG, "nat_select: null output");
  if (((uintptr_t)mask & 15u) || ((uintptr_t)pi & 15u))
    return fail(NAT_ERR_INVALID_ARG, "nat_select: mask and pi must be 16-byte aligned");
  if (sp->resp_base < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select: resp_base < 0");
  SelConst c{};
  c.resp_base = (uint32_t)sp->resp_base;
  c.mode = sp->mode;
  c.min_cut = sp->min_cut;
  c.beta = sp->beta;
  c.k0 = (uint32_t)(sp->seed & 0xFFFFFFFFull);
  c.k1 = (uint32_t)((sp->seed >> 32) ^ (sp->offset >> 32));
  c.off_lo = (uint32_t)(sp->offset & 0xFFFFFFFFull);
  c.thr = 0;
  c.pi_urs = 0.f;
  switch (sp->mode) {
    case NAT_SEL_URS: {
      if (!(sp->p > 0.0 && sp->p <= 1.0))
        return fail(NAT_ERR_INVALID_ARG, "nat_select: URS needs 0 < p <= 1 (got %g)", sp->p);
      double t = __builtin_floor(sp->p * 4294967296.0);
      uint64_t thr = (uint64_t)t;
      if (thr < 1) thr = 1;
      if (thr > (1ull << 32)) thr = 1ull << 32;
      c.thr = thr;
      c.pi_urs = (float)((double)thr / 4294967296.0);
      break;
    }
    case NAT_SEL_RPC:
      if (sp->min_cut < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select: min_cut < 0");
      if (!cut_len && B > 0) return fail(NAT_ERR_INVALID_ARG, "nat_select: RPC needs cut_len");
      break;
    case NAT_SEL_DET:
      if (!(sp->beta > 0.0 && sp->beta <= 1.0))
        return fail(NAT_ERR_INVALID_ARG, "nat_select: DET needs 0 < beta <= 1 (got %g)", sp->beta);
      if (!cut_len && B > 0) return fail(NAT_ERR_INVALID_ARG, "nat_select: DET needs cut_len");
      break;
    default:
      return fail(NAT_ERR_INVALID_ARG, "nat_select: unknown mode %d", sp->mode);
  }
  if (B == 0) return NAT_OK;
  if (sp->mode != NAT_SEL_URS) {
    cut_kernel<<<(B + 127) / 128, 128, 0, stream>>>(c, B, cu_seqlens, cut_len);
    NAT_LAUNCH_CHECK("cut_kernel");
  }
  if (n_tot > 0) {
    const unsigned grid = (unsigned)((n_tot + kSelBlockTokens - 1) / kSelBlockTokens);
    select_kernel<<<grid, kSelThreads, 0, stream>>>(c, B, cu_seqlens, n_tot, cut_len, mask, pi);
    NAT_LAUNCH_CHECK("select_kernel");
  }
  return NAT_OK;
}

// Argument checks and the launch sequence shared by nat_compact and nat_compact_static
// (they differ only in where the chunk-count scratch lives).
static int compact_check(const char* who, int32_t B, const int32_t* cu_seqlens, int64_t n_tot,
                         const uint8_t* mask, const int32_t* sel_idx, const int32_t* sel_resp,
                         const int32_t* sel_offsets, const int32_t* n_sel, int64_t cap) {
  if (B < 0 || n_tot < 0 || cap < 0) return fail(NAT_ERR_INVALID_ARG, "%s: negative size", who);
  if (n_tot > 0x7FFFFFFFll) return fail(NAT_ERR_UNSUPPORTED, "%s: n_tot exceeds int32", who);
  if (!cu_seqlens || !sel_offsets || !n_sel) return fail(NAT_ERR_INVALID_ARG, "%s: null pointer", who);
  if (n_tot > 0 && !mask) return fail(NAT_ERR_INVALID_ARG, "%s: mask is null", who);
  if ((uintptr_t)mask & 15u)
    return fail(NAT_ERR_INVALID_ARG, "%s: mask must be 16-byte aligned", who);
  if (cap > 0 && (!sel_idx || !sel_resp)) return fail(NAT_ERR_INVALID_ARG, "%s: null list", who);
  return NAT_OK;
}

static int compact_launch(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const uint8_t* mask,
                          int32_t* sel_idx, int32_t* sel_resp, int32_t* sel_offsets,
                          int32_t* n_sel, int64_t cap, int32_t* chunk_count, cudaStream_t stream) {
  // Every scratch entry read here is written earlier in the same sequence (counts by the
  // first kernel, offsets and total by the scan), so the scratch needs no clearing.
  const int n_chunks = (int)((n_tot + kChunk - 1) / kChunk);
  if (n_chunks > 0) {
    compact_count_kernel<<<(n_chunks + kCountChunks - 1) / kCountChunks, kCmpThreads, 0, stream>>>(
        mask, n_tot, n_chunks, chunk_count);
    NAT_LAUNCH_CHECK("compact_count_kernel");
  }
  compact_scan_kernel<<<1, 1024, 0, stream>>>(chunk_count, n_chunks, n_sel, sel_offsets, B);
  NAT_LAUNCH_CHECK("compact_scan_kernel");
  if (n_chunks > 0) {
    compact_write_kernel<<<n_chunks, kCmpThreads, 0, stream>>>(B, cu_seqlens, n_tot, mask,
                                                               chunk_count, sel_idx, sel_resp,
                                                               sel_offsets, cap);
    NAT_LAUNCH_CHECK("compact_write_kernel");
  } else if (B > 0) {
    NAT_CUDA(cudaMemsetAsync(sel_offsets, 0, sizeof(int32_t) * (size_t)B, stream));
  }
  return NAT_OK;
}

}  // namespace nat

extern "C" {

int nat_grpo_adv(int32_t P, int32_t G, const float* rewards, float eps, float* adv,
                 void* stream) {
  if (P < 0 || G <= 0) return nat::fail(NAT_ERR_INVALID_ARG, "nat_grpo_adv: need P >= 0, G > 0");
  if (!(eps >= 0.f)) return nat::fail(NAT_ERR_INVALID_ARG, "nat_grpo_adv: eps must be >= 0");
  if (P == 0) return NAT_OK;
  if (!rewards || !adv) return nat::fail(NAT_ERR_INVALID_ARG, "nat_grpo_adv: null pointer");
  nat::grpo_adv_kernel<<<(P + 127) / 128, 128, 0, (cudaStream_t)stream>>>(P, G, rewards, eps, adv);
  NAT_LAUNCH_CHECK("grpo_adv_kernel");
  return NAT_OK;
}

int nat_select(const nat_select_params* params, int32_t B, const int32_t* cu_seqlens,
               int64_t n_tot, uint8_t* mask, float* pi, int32_t* cut_len, void* stream) {
  return nat::select_impl(params, B, cu_seqlens, n_tot, mask, pi, cut_len, (cudaStream_t)stream);
}

int nat_select_survival(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const float* surv,
                        uint64_t seed, uint64_t offset, int32_t resp_base, uint8_t* mask,
                        int32_t* cut_len, void* stream_) {
  using namespace nat;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: negative size");
  if (n_tot > 0x7FFFFFFFll)
    return fail(NAT_ERR_UNSUPPORTED, "nat_select_survival: n_tot exceeds int32");
  if (!cu_seqlens || (B > 0 && !cut_len) || (n_tot > 0 && (!surv || !mask)))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: null pointer");
  if (((uintptr_t)surv & 15u) || ((uintptr_t)mask & 15u))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: surv and mask must be 16-byte aligned");
  if (resp_base < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: resp_base < 0");
  if (B == 0) return NAT_OK;
  SelConst c{};
  c.resp_base = (uint32_t)resp_base;
  c.k0 = (uint32_t)(seed & 0xFFFFFFFFull);
  c.k1 = (uint32_t)((seed >> 32) ^ (offset >> 32));
  c.off_lo = (uint32_t)(offset & 0xFFFFFFFFull);
  NAT_CUDA(cudaMemsetAsync(cut_len, 0, sizeof(int32_t) * (size_t)B, stream));
  if (n_tot > 0) {
    const int64_t per_block = (int64_t)kSelThreads * kTokPerThread;
    const unsigned grid = (unsigned)((n_tot + per_block - 1) / per_block);
    select_survival_kernel<<<grid, kSelThreads, 0, stream>>>(c, B, cu_seqlens, n_tot, surv, mask,
                                                             cut_len);
    NAT_LAUNCH_CHECK("select_survival_kernel");
  }
  return NAT_OK;
}

static int move_rows(const char* who, const void* src, int64_t row_bytes, const int32_t* sel_idx,
                     const int32_t* n_sel, int64_t cap, int scatter, void* dst,
                     cudaStream_t stream) {
  using namespace nat;
  if (row_bytes <= 0 || (row_bytes & 15) != 0)
    return fail(NAT_ERR_INVALID_ARG, "%s: row_bytes must be a positive multiple of 16", who);
  if (cap < 0) return fail(NAT_ERR_INVALID_ARG, "%s: negative capacity", who);
  if (!n_sel || (cap > 0 && (!src || !dst || !sel_idx)))
    return fail(NAT_ERR_INVALID_ARG, "%s: null pointer", who);
  if (((uintptr_t)src & 15u) || ((uintptr_t)dst & 15u))
    return fail(NAT_ERR_INVALID_ARG, "%s: src and dst must be 16-byte aligned", who);
  if (cap == 0) return NAT_OK;
  const int64_t blocks = (cap + 7) / 8;
  const unsigned grid = (unsigned)(blocks < 148 * 8 ? blocks : 148 * 8);
  move_rows_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const uint4*>(src), row_bytes / 16,
                                             sel_idx, n_sel, cap, scatter,
                                             reinterpret_cast<uint4*>(dst));
  NAT_LAUNCH_CHECK("move_rows_kernel");
  return NAT_OK;
}

int nat_gather_rows(const void* src, int64_t row_bytes, const int32_t* sel_idx,
                    const int32_t* n_sel, int64_t cap, void* dst, void* stream) {
  return move_rows("nat_gather_rows", src, row_bytes, sel_idx, n_sel, cap, 0, dst,
                   (cudaStream_t)stream);
}

int nat_scatter_rows(const void* src, int64_t row_bytes, const int32_t* sel_idx,
                     const int32_t* n_sel, int64_t cap, int64_t n_tot, void* dst, void* stream) {
  if (n_tot < 0) return nat::fail(NAT_ERR_INVALID_ARG, "nat_scatter_rows: negative n_tot");
  if (n_tot > 0 && row_bytes > 0 && dst) {
    int s = nat::check_cuda(cudaMemsetAsync(dst, 0, (size_t)n_tot * (size_t)row_bytes,
                                            (cudaStream_t)stream), "cudaMemsetAsync");
    if (s != NAT_OK) return s;
  }
  return move_rows("nat_scatter_rows", src, row_bytes, sel_idx, n_sel, cap, 1, dst,
                   (cudaStream_t)stream);
}

size_t nat_compact_workspace_bytes(int64_t n_tot) {
  if (n_tot < 0) return 0;
  const int64_t chunks = (n_tot + nat::kChunk - 1) / nat::kChunk;
  return nat::align_up((size_t)(chunks + 1) * sizeof(int32_t), 256);
}

int nat_compact(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const uint8_t* mask,
                int32_t* sel_idx, int32_t* sel_resp, int32_t* sel_offsets, int32_t* n_sel,
                int64_t cap, void* workspace, size_t workspace_bytes, void* stream_) {
  using namespace nat;
  int s = compact_check("nat_compact", B, cu_seqlens, n_tot, mask, sel_idx, sel_resp, sel_offsets,
                        n_sel, cap);
  if (s != NAT_OK) return s;
  if (workspace_bytes < nat_compact_workspace_bytes(n_tot) || !workspace)
    return fail(NAT_ERR_CAPACITY, "nat_compact: workspace too small (%zu < %zu)", workspace_bytes,
                nat_compact_workspace_bytes(n_tot));
  if (((uintptr_t)workspace & 255u) != 0)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact: workspace must be 256-byte aligned");
  return compact_launch(B, cu_seqlens, n_tot, mask, sel_idx, sel_resp, sel_offsets, n_sel, cap,
                        reinterpret_cast<int32_t*>(workspace), (cudaStream_t)stream_);
}

}  // extern "C"

// ---------------------------------------------------------------------------
// nat_compact_static: the same compaction with its scan scratch held inside the
// library instead of passed in.
// ---------------------------------------------------------------------------
namespace nat {
namespace {

// Chunk counts / offsets for up to kStaticMaxChunks chunks of 4096 tokens.
// Lives in every CUDA context that loads this library, until the process ends.
constexpr int kStaticMaxChunks = 16384;
static __device__ __align__(256) int32_t g_compact_scratch[kStaticMaxChunks + 1];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
int32_t* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of g_compact_scratch on the current device.  In host code the
// array's name is only a handle for the runtime, never a pointer a kernel could
// use, so the address is asked for once per device and remembered.
int static_scratch(int32_t** out) {
  int dev = 0;
  NAT_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices)
    return fail(NAT_ERR_UNSUPPORTED, "nat_compact_static: device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    NAT_CUDA(cudaGetSymbolAddress(&ptr, g_compact_scratch));
    if (!ptr) return fail(NAT_ERR_CUDA, "nat_compact_static: scratch symbol has no address");
    g_scratch_addr[dev] = static_cast<int32_t*>(ptr);
  }
  *out = g_scratch_addr[dev];
  return NAT_OK;
}

}  // namespace
}  // namespace nat

extern "C" {

int64_t nat_compact_static_max_tokens(void) {
  return (int64_t)nat::kStaticMaxChunks * nat::kChunk;
}

int nat_compact_static(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const uint8_t* mask,
                       int32_t* sel_idx, int32_t* sel_resp, int32_t* sel_offsets, int32_t* n_sel,
                       int64_t cap, void* stream_) {
  using namespace nat;
  int s = compact_check("nat_compact_static", B, cu_seqlens, n_tot, mask, sel_idx, sel_resp,
                        sel_offsets, n_sel, cap);
  if (s != NAT_OK) return s;
  if (n_tot > nat_compact_static_max_tokens())
    return fail(NAT_ERR_CAPACITY,
                "nat_compact_static: n_tot = %lld exceeds the built-in scratch (at most %lld "
                "tokens); use nat_compact with a caller-provided workspace",
                (long long)n_tot, (long long)nat_compact_static_max_tokens());
  int32_t* chunk_count = nullptr;
  s = static_scratch(&chunk_count);
  if (s != NAT_OK) return s;
  return compact_launch(B, cu_seqlens, n_tot, mask, sel_idx, sel_resp, sel_offsets, n_sel, cap,
                        chunk_count, (cudaStream_t)stream_);
}

}  // extern "C"
