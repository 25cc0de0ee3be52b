// Group-relative advantages, token selection (URS / RPC / deterministic
// truncation) and stream compaction of the selected indices.
//
// These kernels are bound by HBM traffic (select writes 5 bytes per token and
// reads nothing; compact reads the mask twice and writes 8 bytes per selected
// token), so they use 16-byte accesses: one thread owns 16 consecutive tokens.
// Floating-point steps that must agree bit for bit with a plain IEEE
// evaluation use the explicit round-to-nearest intrinsics, which the compiler
// never contracts into fused multiply-adds.
#include <mutex>

#include "nat_common.cuh"

namespace nat {
namespace {

// ---------------------------------------------------------------- Philox
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplies
// with the key advanced by Weyl constants between rounds.
struct Philox4 {
  uint32_t x, y, z, w;
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                                 uint32_t c3, uint32_t k0, uint32_t k1) {
  constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
  constexpr uint32_t kWeylA = 0x9E3779B9u, kWeylB = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hiA = __umulhi(kMulA, c0), loA = kMulA * c0;
    const uint32_t hiB = __umulhi(kMulB, c2), loB = kMulB * c2;
    c0 = hiB ^ c1 ^ k0;
    c1 = loB;
    c2 = hiA ^ c3 ^ k1;
    c3 = loA;
    k0 += kWeylA;
    k1 += kWeylB;
  }
  return {c0, c1, c2, c3};
}

// Largest i with cu[i] <= n among responses that are not empty at n, i.e. the
// response that owns packed token n (cu is non-decreasing, cu[B] > n).
__device__ __forceinline__ int owner_of(const int32_t* __restrict__ cu, int B, int64_t n) {
  int lo = 0, hi = B;  // invariant: cu[lo] <= n < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(cu + mid) <= n) lo = mid; else hi = mid;
  }
  return lo;
}

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
constexpr int kTokPerThread = 16;
constexpr int kSelThreads = 256;

struct SelConst {
  int mode;
  int min_cut;
  double beta;
  uint64_t thr;    // URS threshold, 1..2^32
  float pi_urs;    // thr / 2^32
  uint32_t k0, k1, off_lo;
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
      const Philox4 r = philox4x32_10(0u, (uint32_t)i, 1u, c.off_lo, c.k0, c.k1);
      const uint64_t u = ((uint64_t)r.y << 32) | (uint64_t)r.x;
      L = C + (int)__umul64hi(u, n);
    } else {
      L = max(1, (int)floor(__dmul_rn(c.beta, (double)T)));
    }
  }
  cut_len[i] = L;
}

// Owner search restricted to responses lo..hi (cu[lo] <= n < cu[hi + 1]).
__device__ __forceinline__ int owner_between(const int32_t* __restrict__ cu, int lo, int hi,
                                             int64_t n) {
  ++hi;  // invariant: cu[lo] <= n < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(cu + mid) <= n) lo = mid; else hi = mid;
  }
  return lo;
}

// One block per 4096 consecutive packed tokens, one thread per 16 of them (so a thread
// reuses each Philox block for up to four tokens).  The mask leaves as one 16-byte store
// per thread; pi is transposed through shared memory so that every warp store covers 512
// contiguous bytes.
constexpr int kSelBlockTokens = kSelThreads * kTokPerThread;  // 4096
constexpr int kPiPad = kTokPerThread + 1;                     // 17: conflict-free rows

__global__ void __launch_bounds__(kSelThreads)
select_kernel(SelConst c, int B, const int32_t* __restrict__ cu, int64_t n_tot,
              const int32_t* __restrict__ cut_len, uint8_t* __restrict__ mask,
              float* __restrict__ pi) {
  __shared__ float pi_s[kSelThreads * kPiPad];
  __shared__ int range_s[2];
  const int64_t nb0 = (int64_t)blockIdx.x * kSelBlockTokens;
  const int cnt_block = (int)min((int64_t)kSelBlockTokens, n_tot - nb0);
  if (threadIdx.x == 0) {
    range_s[0] = owner_of(cu, B, nb0);
    range_s[1] = owner_of(cu, B, nb0 + cnt_block - 1);
  }
  __syncthreads();
  const int64_t n0 = nb0 + (int64_t)threadIdx.x * kTokPerThread;
  if (n0 < n_tot) {
    const int cnt = (int)min((int64_t)kTokPerThread, n_tot - n0);
    int i = owner_between(cu, range_s[0], range_s[1], n0);
    int64_t start = cu[i], end = cu[i + 1];
    int L = 0, C = 0;
    float den = 1.f;
    auto enter_response = [&]() {
      if (c.mode != NAT_SEL_URS) {
        L = cut_len[i];
        const int T = (int)(end - start);
        C = (c.mode == NAT_SEL_RPC) ? min(max(c.min_cut, 1), T) : T;
        den = (float)(T - C + 1);
      }
    };
    enter_response();
    uint32_t cached_blk = 0xFFFFFFFFu;
    int cached_resp = -1;
    Philox4 rnd = {0, 0, 0, 0};

    alignas(16) uint8_t m[kTokPerThread];
    float* pr = pi_s + threadIdx.x * kPiPad;
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
        const uint32_t t0 = (uint32_t)(n - start);  // t - 1
        if (c.mode == NAT_SEL_URS) {
          const uint32_t blk = t0 >> 2;
          if (blk != cached_blk || i != cached_resp) {
            rnd = philox4x32_10(blk, (uint32_t)i, 0u, c.off_lo, c.k0, c.k1);
            cached_blk = blk;
            cached_resp = i;
          }
          const uint32_t lane = t0 & 3u;
          const uint32_t x = lane == 0 ? rnd.x : lane == 1 ? rnd.y : lane == 2 ? rnd.z : rnd.w;
          m[j] = ((uint64_t)x < c.thr) ? 1 : 0;
          pv = c.pi_urs;
        } else {
          const int t = (int)t0 + 1;
          m[j] = (t <= L) ? 1 : 0;
          const int T = (int)(end - start);
          pv = (t <= C) ? 1.f : __fdiv_rn((float)(T - t + 1), den);
        }
      }
      pr[j] = pv;
    }
    if (cnt == kTokPerThread) {
      *reinterpret_cast<uint4*>(mask + n0) = *reinterpret_cast<const uint4*>(m);
    } else {
      for (int j = 0; j < cnt; ++j) mask[n0 + j] = m[j];
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
  const int64_t n0 = ((int64_t)blockIdx.x * kSelThreads + threadIdx.x) * kTokPerThread;
  if (n0 >= n_tot) return;
  const int cnt = (int)min((int64_t)kTokPerThread, n_tot - n0);
  int i = owner_of(cu, B, n0);
  int64_t start = cu[i], end = cu[i + 1];
  auto draw = [&]() {
    const Philox4 r = philox4x32_10(0u, (uint32_t)i, 2u, c.off_lo, c.k0, c.k1);
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

__device__ __forceinline__ uint32_t load_mask_bits(const uint8_t* __restrict__ mask, int64_t n0,
                                                   int64_t n_tot) {
  uint32_t bits = 0;
  if (n0 + kTokPerThread <= n_tot) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask + n0));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if ((w[q] >> (8 * b)) & 0xFFu) bits |= 1u << (4 * q + b);
  } else {
    for (int j = 0; j < kTokPerThread; ++j)
      if (n0 + j < n_tot && mask[n0 + j] != 0) bits |= 1u << j;
  }
  return bits;
}

__global__ void __launch_bounds__(kCmpThreads)
compact_count_kernel(const uint8_t* __restrict__ mask, int64_t n_tot,
                     int32_t* __restrict__ chunk_count) {
  __shared__ int warp_sum[kCmpThreads / 32];
  const int64_t n0 = (int64_t)blockIdx.x * kChunk + (int64_t)threadIdx.x * kTokPerThread;
  int c = (n0 < n_tot) ? __popc(load_mask_bits(mask, n0, n_tot)) : 0;
  c = __reduce_add_sync(0xFFFFFFFFu, c);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int w = 0; w < kCmpThreads / 32; ++w) s += warp_sum[w];
    chunk_count[blockIdx.x] = s;
  }
}

// Exclusive scan of the chunk counts by a single block (in place), total to
// chunk_count[n_chunks], n_sel and sel_offsets[B].
__global__ void __launch_bounds__(1024)
compact_scan_kernel(int32_t* __restrict__ chunk_count, int n_chunks, int32_t* __restrict__ n_sel,
                    int32_t* __restrict__ sel_offsets, int B) {
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n_chunks; base += 1024) {
    const int idx = base + threadIdx.x;
    const int v = idx < n_chunks ? chunk_count[idx] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if ((threadIdx.x & 31) >= o) incl += up;
    }
    if ((threadIdx.x & 31) == 31) warp_tot[threadIdx.x >> 5] = incl;
    __syncthreads();
    if (threadIdx.x < 32) {
      int w = warp_tot[threadIdx.x];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, w, o);
        if (threadIdx.x >= o) w += up;
      }
      warp_tot[threadIdx.x] = w;  // inclusive over warps
    }
    __syncthreads();
    const int carry = carry_s;
    const int warp_excl = (threadIdx.x >> 5) ? warp_tot[(threadIdx.x >> 5) - 1] : 0;
    if (idx < n_chunks) chunk_count[idx] = carry + warp_excl + incl - v;
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + warp_tot[31];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    chunk_count[n_chunks] = carry_s;
    *n_sel = carry_s;
    sel_offsets[B] = carry_s;
  }
}

__global__ void __launch_bounds__(kCmpThreads)
compact_write_kernel(int B, const int32_t* __restrict__ cu, int64_t n_tot,
                     const uint8_t* __restrict__ mask, const int32_t* __restrict__ chunk_offset,
                     int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_resp,
                     int32_t* __restrict__ sel_offsets, int64_t cap) {
  __shared__ int warp_tot[kCmpThreads / 32];
  __shared__ int thread_excl[kCmpThreads];
  __shared__ uint32_t thread_bits[kCmpThreads];
  __shared__ int32_t idx_s[kChunk];
  __shared__ int32_t resp_s[kChunk];
  __shared__ int range_s[2];
  const int64_t chunk0 = (int64_t)blockIdx.x * kChunk;
  if (threadIdx.x == 0) {  // responses that own the chunk's first and last token
    const int64_t last = min(chunk0 + (int64_t)kChunk, n_tot) - 1;
    range_s[0] = owner_of(cu, B, chunk0);
    range_s[1] = owner_of(cu, B, last);
  }
  const int64_t n0 = chunk0 + (int64_t)threadIdx.x * kTokPerThread;
  const uint32_t bits = (n0 < n_tot) ? load_mask_bits(mask, n0, n_tot) : 0u;
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
  const int base = chunk_offset[blockIdx.x];
  const int excl = base + warp_excl + incl - c;  // selected tokens before n0
  thread_excl[threadIdx.x] = excl;
  thread_bits[threadIdx.x] = bits;
  __syncthreads();

  // The chunk's selected tokens are consecutive in the output lists: stage them in
  // shared memory, then write them out with fully coalesced stores.
  if (bits != 0u) {
    int i = owner_between(cu, range_s[0], range_s[1], n0);
    int64_t end = cu[i + 1];
    int k = excl - base;
    for (int j = 0; j < kTokPerThread; ++j) {
      if ((bits >> j) & 1u) {
        const int64_t n = n0 + j;
        while (n >= end) end = cu[++i + 1];
        idx_s[k] = (int32_t)n;
        resp_s[k] = i;
        ++k;
      }
    }
  }
  __syncthreads();
  {
    int total = 0;
    for (int w = 0; w < kCmpThreads / 32; ++w) total += warp_tot[w];
    for (int e = threadIdx.x; e < total; e += kCmpThreads) {
      const int64_t k = (int64_t)base + e;
      if (k < cap) {
        sel_idx[k] = idx_s[e];
        sel_resp[k] = resp_s[e];
      }
    }
  }

  // Per-response offsets: every i with cu[i] inside this chunk (the last chunk
  // also takes the boundaries equal to n_tot).  sel_offsets[B] is the scan's.
  const int64_t chunk_end = min(chunk0 + (int64_t)kChunk, n_tot);
  const bool last = (chunk_end == n_tot);
  // first i with cu[i] >= chunk0
  int lo = 0, hi = B;  // search in [0, B]
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if ((int64_t)cu[mid] < chunk0) lo = mid + 1; else hi = mid;
  }
  for (int i = lo + threadIdx.x; i < B; i += kCmpThreads) {
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
  SelConst c{};
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
                        uint64_t seed, uint64_t offset, uint8_t* mask, int32_t* cut_len,
                        void* stream_) {
  using namespace nat;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0) return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: negative size");
  if (n_tot > 0x7FFFFFFFll)
    return fail(NAT_ERR_UNSUPPORTED, "nat_select_survival: n_tot exceeds int32");
  if (!cu_seqlens || (B > 0 && !cut_len) || (n_tot > 0 && (!surv || !mask)))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: null pointer");
  if (((uintptr_t)surv & 15u) || ((uintptr_t)mask & 15u))
    return fail(NAT_ERR_INVALID_ARG, "nat_select_survival: surv and mask must be 16-byte aligned");
  if (B == 0) return NAT_OK;
  SelConst c{};
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
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0 || cap < 0) return fail(NAT_ERR_INVALID_ARG, "nat_compact: negative size");
  if (n_tot > 0x7FFFFFFFll) return fail(NAT_ERR_UNSUPPORTED, "nat_compact: n_tot exceeds int32");
  if (!cu_seqlens || !sel_offsets || !n_sel)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact: null pointer");
  if (n_tot > 0 && !mask) return fail(NAT_ERR_INVALID_ARG, "nat_compact: mask is null");
  if (cap > 0 && (!sel_idx || !sel_resp)) return fail(NAT_ERR_INVALID_ARG, "nat_compact: null list");
  if (workspace_bytes < nat_compact_workspace_bytes(n_tot) || !workspace)
    return fail(NAT_ERR_CAPACITY, "nat_compact: workspace too small (%zu < %zu)", workspace_bytes,
                nat_compact_workspace_bytes(n_tot));
  if (((uintptr_t)workspace & 255u) != 0)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact: workspace must be 256-byte aligned");
  int32_t* chunk_count = reinterpret_cast<int32_t*>(workspace);
  const int n_chunks = (int)((n_tot + kChunk - 1) / kChunk);
  if (n_chunks > 0) {
    compact_count_kernel<<<n_chunks, kCmpThreads, 0, stream>>>(mask, n_tot, chunk_count);
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
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || n_tot < 0 || cap < 0)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_static: negative size");
  if (n_tot > nat_compact_static_max_tokens())
    return fail(NAT_ERR_CAPACITY,
                "nat_compact_static: n_tot = %lld exceeds the built-in scratch (at most %lld "
                "tokens); use nat_compact with a caller-provided workspace",
                (long long)n_tot, (long long)nat_compact_static_max_tokens());
  if (!cu_seqlens || !sel_offsets || !n_sel)
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_static: null pointer");
  if (n_tot > 0 && !mask) return fail(NAT_ERR_INVALID_ARG, "nat_compact_static: mask is null");
  if (cap > 0 && (!sel_idx || !sel_resp))
    return fail(NAT_ERR_INVALID_ARG, "nat_compact_static: null list");
  int32_t* chunk_count = nullptr;
  int s = static_scratch(&chunk_count);
  if (s != NAT_OK) return s;
  // Every scratch entry this call reads is written earlier in the same call
  // (counts by the first kernel, offsets and total by the scan), so nothing left
  // by a previous call needs clearing.
  const int n_chunks = (int)((n_tot + kChunk - 1) / kChunk);
  if (n_chunks > 0) {
    compact_count_kernel<<<n_chunks, kCmpThreads, 0, stream>>>(mask, n_tot, chunk_count);
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

}  // extern "C"
