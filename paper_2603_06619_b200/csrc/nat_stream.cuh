// Device helpers shared by the kernels that walk the packed token stream (selection,
// compaction, cut laws): the Philox4x32-10 generator, searches in cu_seqlens, and the
// token-to-thread layout (one thread per 16 consecutive tokens, 4096 tokens per block).
#pragma once

#include <climits>
#include <cstdint>

namespace nat {

constexpr int kTokPerThread = 16;
constexpr int kSelThreads = 256;
constexpr int kSelBlockTokens = kSelThreads * kTokPerThread;  // 4096
constexpr int kPiPad = kTokPerThread + 1;                     // 17: conflict-free rows

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
    // each 32x32->64 product as one wide multiply (its halves are the round's hi and lo)
    const unsigned long long pA = (unsigned long long)kMulA * c0;
    const unsigned long long pB = (unsigned long long)kMulB * c2;
    c0 = (uint32_t)(pB >> 32) ^ c1 ^ k0;
    c1 = (uint32_t)pB;
    c2 = (uint32_t)(pA >> 32) ^ c3 ^ k1;
    c3 = (uint32_t)pA;
    k0 += kWeylA;
    k1 += kWeylB;
  }
  return {c0, c1, c2, c3};
}

// First index i >= lo with cu[i] > x among cu[0..B] (B + 1 if there is none), found by a
// whole warp: every step probes 32 positions at once, so a stream of 2^15 responses takes
// four dependent loads instead of fifteen.  The first step probes 32 consecutive entries
// because the answer is usually next to the hint.  All 32 lanes call it with the same
// arguments; cu[i] <= x must hold for every i < lo.
__device__ __forceinline__ int warp_upper_bound(const int32_t* __restrict__ cu, int B, int64_t x,
                                                int lo) {
  const int lane = threadIdx.x & 31;
  int hi = B + 1;
  int step = 1;
  while (lo < hi) {
    const int idx = lo + lane * step;
    const bool gt = idx >= hi || (int64_t)__ldg(cu + idx) > x;
    const unsigned b = __ballot_sync(0xFFFFFFFFu, gt);
    if (b == 0u) {
      lo += 31 * step + 1;
    } else {
      const int f = __ffs(b) - 1;
      hi = min(hi, lo + f * step);
      if (f > 0) lo += (f - 1) * step + 1;
    }
    step = max(1, (hi - lo + 31) / 32);
  }
  return lo;
}

// The searches a block makes for the responses around its token range usually end inside
// one window of 32 consecutive cu entries placed by proportion (position / n_tot * B), so
// one load serves them all.  cu_window loads the window (one entry per lane, +infinity
// past cu[B]); window_first turns the ballot of a monotone predicate over it into the first
// index where it holds, or reports a miss when that index may lie outside the window.
__device__ __forceinline__ int64_t cu_window(const int32_t* __restrict__ cu, int B, int64_t x,
                                             int64_t n_tot, int* w0) {
  const int guess = (int)((x * (int64_t)B) / (n_tot > 0 ? n_tot : 1));
  *w0 = max(0, min(guess - 8, B - 30));
  const int idx = *w0 + (int)(threadIdx.x & 31);
  return idx <= B ? (int64_t)__ldg(cu + idx) : INT64_MAX;
}

__device__ __forceinline__ bool window_first(unsigned ballot, int w0, int* out) {
  if (ballot == 0u || ((ballot & 1u) != 0u && w0 > 0)) return false;
  *out = w0 + __ffs(ballot) - 1;
  return true;
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

// 16 mask bits -> 16 bytes of 0/1 (bit j -> byte j).
__device__ __forceinline__ uint4 bits_to_bytes(uint32_t bits) {
  constexpr uint32_t kSpread = 0x00204081u;  // 1 + 2^7 + 2^14 + 2^21
  uint4 v;
  v.x = ((bits & 0xFu) * kSpread) & 0x01010101u;
  v.y = (((bits >> 4) & 0xFu) * kSpread) & 0x01010101u;
  v.z = (((bits >> 8) & 0xFu) * kSpread) & 0x01010101u;
  v.w = (((bits >> 12) & 0xFu) * kSpread) & 0x01010101u;
  return v;
}

}  // namespace nat
