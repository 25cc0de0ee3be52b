// bf16 policy loss on the Blackwell tensor cores (tcgen05 + TMEM + TMA).
//
// One warp-specialised persistent kernel template serves the four dense
// contractions of the path; they differ in operand layout and epilogue:
//
//   kFwd  S = Hc W^T  (rows x V, K = d)  epilogue: online max / sum-exp and
//                                        target-logit pick per row; the logits
//                                        stay in tensor memory and registers.
//   kDz   S = Hc W^T  recomputed         epilogue: -g exp(S - lse) -> bf16 into
//                                        the bounded scratch dZ[chunk, V].
//   kDh   dH = dZ W   (rows x d, K = V)  epilogue: + g W[y] (one-hot term) -> bf16; or, with
//                                        the K range cut into parts so that the work units
//                                        fill the device, each part's fp32 partial tile
//                                        stored into its slice of a scratch whose slices a
//                                        small pass adds in part order to form dH.
//   kDw   dW += dZ^T Hc (V x d, K = rows) epilogue: fp32 reduction into dW (TMA reduce-add).
//   kE    S = Hc W^T  single-pass variant  epilogue: E = exp(S - mref) -> bf16 into the
//                                        same scratch, row sums of E, target pick.
//
// Two ways through the backward.  The two-pass route recomputes S (kDz) from the
// forward's lse.  The single-pass route (nat_policy_loss_fwd_bwd) computes S once per
// row chunk: kE stores the softmax numerators relative to a per-row reference mref (the
// row maximum over the first vocabulary tile, from a one-tile kFwd launch), the row
// scalars lse, g and c = -g / sum(E) follow, and because they are per-row they move out
// of the contractions: dH = c (E W) + g W[y] (scaled in kDh's epilogue) and
// dW += E^T (c h) (rows of Hc scaled into Hs).  A chunk in which some logit exceeds its
// row's reference by more than 60 (E would leave the fp32/bf16 range) is redone by the
// two-pass kernels, which are launched predicated on the chunk's flag.
//
// Roles per CTA: warp 0 issues TMA loads into a shared-memory ring, warp 1 issues
// tcgen05.mma into fp32 accumulators in tensor memory, four epilogue warps per A sub-tile
// drain them.  kFwd / kDz: one sub-tile, two 128x256 accumulators, so one tile's epilogue
// overlaps the next tile's MMAs.  kE / kDh / kDw: two sub-tiles per CTA (512x256 per CTA
// pair, a quarter less operand traffic); their accumulators fill tensor memory, the
// epilogue is exposed and therefore leaves through a shared-memory staging block by TMA
// store (kE, kDh in K parts) or TMA reduction (kDw) instead of scattered 16-byte accesses.
// Work units are taken round-robin by the CTA pairs; kE's units are single vocabulary
// tiles ordered so that the pairs sweep the vocabulary together (see decode_unit).
// Every mbarrier wait is bounded; a wait that runs out raises the block's
// abort flag and NAT_DEV_TIMEOUT in the workspace's status word.
#include <cuda_bf16.h>

#include <atomic>
#include <mutex>
#include <vector>
#include <cstdlib>

#include "nat_tc.cuh"
#include "nat_token.cuh"

namespace nat {
namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int kABytes = BM * BK * 2;               // 16 KB
constexpr int kBoxBytes = 64 * 64 * 2;             // one 64x64 box of an MN-major operand
// Threads per CTA: a TMA warp, an MMA warp and four epilogue warps per A sub-tile.
constexpr int threads_for(int subs) { return 64 + 128 * subs; }
constexpr int kTmemCols = 512;                     // two 256-column accumulators
constexpr int kGroupRows = 32;                     // row blocks that share a vocabulary sweep
constexpr int kTilesPerSplit = 16;                 // vocabulary tiles per work unit
constexpr int kChunkRows = 8192;                   // rows of the dZ scratch
constexpr int kMaxPairs = 512;                     // progress marks (one per CTA or CTA pair)
constexpr int kRowPad = 512;                       // compact rows are padded to the largest M extent of a work unit

enum Mode { kFwd = 0, kDz = 1, kDh = 2, kDw = 3, kE = 4 };

// The single-pass route accepts S - mref up to 60 (numerators and their sums stay finite):
constexpr float kWindowSum = 1.1420073898156842e26f;  // e^60

struct TcParams {
  const int32_t* n_sel;
  int cap;
  int row0;        // first compact row handled by this launch
  int chunk_rows;  // rows this launch may cover (multiple of 128)
  int d, V;
  int n_splits;    // vocabulary splits (kFwd, kDz)
  int cap_pad;     // stride of the per-split partials
  const int32_t* targets;
  const int32_t* sel_idx;
  float* part_m;
  float* part_s;
  float* zt;
  const float* g;
  const float* lse;
  __nv_bfloat16* dZ;
  int ldz;         // elements per dZ row
  const __nv_bfloat16* W;
  __nv_bfloat16* dH;
  float* dW;
  uint32_t* status;
  const float* mref;       // kE: per-row reference
  const float* row_scale;  // kDh: per-row factor on the accumulator (null = 1)
  int b_row0;              // kDw: first row of the B operand's tensor map for this launch
  int k_splits;            // kDh: the K range (the vocabulary) is cut into this many units per
                           //   output tile; above 1 the partial tiles are added into a float32
                           //   scratch (mapC) and dh_finalize_kernel forms dHidden from it
  const int32_t* flag;     // predicate: the launch does nothing unless
  int run_if;              //   (*flag != 0) == run_if   (flag == null: always runs)
  int32_t* ovf;            // kE: set to 1 when the window is exceeded
  unsigned long long* progress;  // per-pair progress marks of the vocabulary sweeps
  unsigned long long epoch;      // distinguishes this launch's marks from earlier ones
};

struct Unit {
  int mb;      // block along the accumulator's M dimension
  int nt_lo;   // first and one-past-last block along N
  int nt_hi;
  int sp;      // vocabulary split (kFwd, kDz, kE) or K part (kDh)
  int kb_lo;   // k-blocks of this unit: the whole K range, or one of k_splits parts of it (kDh)
  int kb_hi;
};

struct Shape {
  int rows;     // valid rows of this launch
  int n_units;
  int kb;       // k-blocks per tile
  int mblocks;
  int nblocks;  // N blocks (kDh, kDw) or vocabulary tiles (kFwd, kDz)
};

template <int MODE, int CTAS, int SUBS>
__device__ __forceinline__ Shape make_shape(const TcParams& p) {
  constexpr int BMU = BM * CTAS * SUBS;  // rows of the M dimension per work unit
  Shape s;
  int n = *p.n_sel;
  n = n < p.cap ? n : p.cap;
  int rows = n - p.row0;
  rows = rows < 0 ? 0 : (rows > p.chunk_rows ? p.chunk_rows : rows);
  if (p.flag != nullptr && ((*p.flag != 0) ? 1 : 0) != p.run_if) rows = 0;
  s.rows = rows;
  if (MODE == kFwd || MODE == kDz || MODE == kE) {
    s.mblocks = (rows + BMU - 1) / BMU;
    s.nblocks = (p.V + BN - 1) / BN;
    s.n_units = s.mblocks * p.n_splits;
    s.kb = p.d / BK;
  } else if (MODE == kDh) {
    s.mblocks = (rows + BMU - 1) / BMU;
    s.nblocks = (p.d + BN - 1) / BN;
    s.n_units = s.mblocks * s.nblocks * p.k_splits;
    s.kb = (p.V + BK - 1) / BK;
  } else {
    s.mblocks = (p.V + BMU - 1) / BMU;
    s.nblocks = (p.d + BN - 1) / BN;
    s.kb = (rows + BK - 1) / BK;
    s.n_units = rows > 0 ? s.mblocks * s.nblocks : 0;
  }
  return s;
}

// Units are ordered so that CTAs running side by side share operands in L2:
// kFwd/kDz/kE take groups of row blocks (kGroupRows x 128 rows) and, inside a
// group, walk the vocabulary splits with the row block varying fastest.
template <int MODE, int CTAS, int SUBS>
__device__ __forceinline__ Unit decode_unit(const TcParams& p, const Shape& s, int u) {
  constexpr int kGroup = kGroupRows / (CTAS * SUBS);
  Unit w;
  w.kb_lo = 0;
  w.kb_hi = s.kb;
  if (MODE == kFwd || MODE == kDz || MODE == kE) {
    // kE: one vocabulary tile per split, so a unit is one tile and the CTA pairs, which take
    // units round-robin, work on the same few vocabulary tiles at any time (a W tile is
    // fetched from DRAM once and found in L2 by the other row blocks of the group) without
    // any pair waiting for another.  The group (4096 rows) keeps the rows' operand blocks
    // (32 MB at d = 4096) resident in L2 next to the W tiles and the streaming stores.
    const int per_group = kGroup * p.n_splits;
    const int grp = u / per_group;
    const int rem = u - grp * per_group;
    int rows_in_group = s.mblocks - grp * kGroup;
    rows_in_group = rows_in_group < kGroup ? rows_in_group : kGroup;
    w.sp = rem / rows_in_group;
    w.mb = grp * kGroup + (rem - w.sp * rows_in_group);
    w.nt_lo = (int)(((long long)w.sp * s.nblocks) / p.n_splits);
    w.nt_hi = (int)(((long long)(w.sp + 1) * s.nblocks) / p.n_splits);
  } else if (MODE == kDh) {
    // (K part, row block, column block), the column block varying fastest: the pairs in
    // flight work on one K part, i.e. on the same half of W and the same few slabs of the
    // numerators (measured 2 % faster per step than taking the parts of a tile in turn)
    const int per_ks = s.mblocks * s.nblocks;
    const int ks = u / per_ks;
    const int rem = u - ks * per_ks;
    w.sp = ks;  // the K part: its partial tile has a slice of the scratch to itself
    w.mb = rem / s.nblocks;
    w.nt_lo = rem - w.mb * s.nblocks;
    w.nt_hi = w.nt_lo + 1;
    const int per = (s.kb + p.k_splits - 1) / p.k_splits;
    w.kb_lo = ks * per;
    w.kb_hi = w.kb_lo + per < s.kb ? w.kb_lo + per : s.kb;
  } else {
    w.sp = 0;
    w.mb = u / s.nblocks;
    w.nt_lo = u - w.mb * s.nblocks;
    w.nt_hi = w.nt_lo + 1;
  }
  return w;
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr float kLog2e = 1.4426950408889634f;

// Shared-memory ring (192 KB): CTAS = 1: stages of (A 128x64 + B 256x64) = 48 KB;
// CTAS = 2: each CTA of the pair holds its 128 rows of A and its 128-row half
// of B, 32 KB per stage, 6 stages.
// SUBS = 2: each CTA holds two 128-row sub-tiles of A per stage (one B tile serves both,
// which cuts the operand bytes per FLOP by a quarter) and both accumulators belong to the
// same output tile.
template <int CTAS, int SUBS>
struct Ring {
  static constexpr int kBRows = BN / CTAS;
  static constexpr int kBBytes = kBRows * BK * 2;
  static constexpr int kABytesS = kABytes * SUBS;
  static constexpr int kStage = kABytesS + kBBytes;
  static constexpr int kNum = (192 * 1024) / kStage;
  // CTA pairs: 4 KB per epilogue warp (32 rows of 128 bytes) from which finished pieces of
  // the tile leave by TMA store (kE) or TMA reduction (kDw)
  static constexpr int kStaging = CTAS == 2 ? 4 * SUBS * 4096 : 0;
  static constexpr size_t kSmem =
      (size_t)kNum * kStage + kStaging + 1024 /*alignment*/ + 256 /*barriers*/;
};

template <int MODE, int CTAS, int SUBS>
__global__ void __launch_bounds__(threads_for(SUBS), 1)
nat_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
              const __grid_constant__ CUtensorMap mapC, const TcParams p) {
  static_assert(SUBS == 1 || CTAS == 2, "two A sub-tiles per CTA are only used by CTA pairs");
  using R = Ring<CTAS, SUBS>;
  constexpr int kNS = R::kNum;
  constexpr int BMU = BM * CTAS * SUBS;
  constexpr uint32_t kNAcc = 2 / SUBS;  // accumulator buffers: two tiles in flight, or one
  constexpr bool kAmn = (MODE == kDw);
  constexpr bool kBmn = (MODE == kDh || MODE == kDw);
  constexpr uint32_t kIdesc = tc::instr_desc_bf16(BM * CTAS, BN, kAmn ? 1 : 0, kBmn ? 1 : 0);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = smem + (size_t)kNS * R::kStage;  // 1024-byte aligned like the ring
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + R::kStaging);
  uint64_t* full_bar = bars;                   // [kNS]   (CTAS = 2: the even CTA's are used)
  uint64_t* empty_bar = bars + kNS;            // [kNS]
  uint64_t* tfull_bar = bars + 2 * kNS;        // [2]
  uint64_t* tempty_bar = bars + 2 * kNS + 2;   // [2]     (CTAS = 2: the even CTA's are used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kNS + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = CTAS == 2 ? (int)(tc::cluster_ctarank() & 1u) : 0;
  const int unit0 = blockIdx.x / CTAS;
  const int unit_stride = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNS; ++s) {
      tc::mbar_init(&full_bar[s], 1);
      tc::mbar_init(&empty_bar[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      tc::mbar_init(&tfull_bar[a], 1);
      tc::mbar_init(&tempty_bar[a], 4 * SUBS * CTAS);
    }
    *abort_flag = 0u;
    tc::fence_barrier_init();
    tc::fence_proxy_async();
    tc::prefetch_tensormap(&mapA);
    tc::prefetch_tensormap(&mapB);
    tc::prefetch_tensormap(&mapC);
  }
  if (warp == 1) {
    if (CTAS == 2) {
      tc::tmem_alloc_pair(tmem_slot, kTmemCols);
      tc::tmem_relinquish_pair();
    } else {
      tc::tmem_alloc(tmem_slot, kTmemCols);
      tc::tmem_relinquish();
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (CTAS == 2) tc::cluster_sync_all();  // the peer's barriers exist before anyone signals them
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const Shape shape = make_shape<MODE, CTAS, SUBS>(p);

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = unit0; ok && u < shape.n_units; u += unit_stride) {
        const Unit w = decode_unit<MODE, CTAS, SUBS>(p, shape, u);
        for (int nt = w.nt_lo; ok && nt < w.nt_hi; ++nt) {
          if ((MODE == kFwd || MODE == kDz) && rank == 0 && p.progress != nullptr) {
            // Pacing.  The CTAs that sweep the same vocabulary split for different row
            // blocks share every W tile through L2 only while they stay within a few
            // tiles of each other; left alone they drift apart (nothing slows the one in
            // front) and each W tile is then read from DRAM several times, which costs
            // more power than the tensor cores can spare.  So each CTA publishes the tile
            // it is starting and briefly holds back while a mate is more than a tile
            // behind.  Purely advisory: the wait is short and bounded, and results do not
            // depend on it.
            constexpr int kGroup = kGroupRows / (CTAS * SUBS);
            volatile unsigned long long* marks = p.progress;
            const int j = nt - w.nt_lo;
            const unsigned long long iter = (unsigned long long)((u - unit0) / unit_stride);
            marks[unit0] = (p.epoch << 40) | (iter << 10) | (unsigned long long)j;
            if (j > 0) {
              const int per_group = kGroup * p.n_splits;
              const int grp = u / per_group;
              int mates = shape.mblocks - grp * kGroup;
              mates = mates < kGroup ? mates : kGroup;
              const int first = grp * per_group + w.sp * mates;
              // All mates' marks are read together (independent loads, one round trip to
              // L2), so a pair that is in step with its mates loses well under the time
              // its shared-memory ring covers.
              for (int spin = 0; spin < 16; ++spin) {
                bool behind = false;
#pragma unroll
                for (int r = 0; r < kGroup; ++r) {
                  const int um = first + (r < mates ? r : 0);
                  const unsigned long long want = (p.epoch << 40) |
                                                  ((unsigned long long)(um / unit_stride) << 10) |
                                                  (unsigned long long)(j - 1);
                  behind |= marks[um % unit_stride] < want;
                }
                if (!behind) break;
                __nanosleep(200);
              }
            }
          }
          for (int kb = w.kb_lo; kb < w.kb_hi; ++kb, ++it) {
            const int s = it % kNS;
            const uint32_t ph = (it / kNS) & 1u;
            if (!tc::mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag)) { ok = false; break; }
            uint8_t* a_dst = smem + (size_t)s * R::kStage;
            uint8_t* b_dst = a_dst + R::kABytesS;
            // CTAS = 2: both CTAs' loads count on the even CTA's barrier, which its
            // own producer arms with the bytes of the whole pair.
            const uint32_t bar = CTAS == 2 ? tc::map_to_cta(tc::smem_u32(&full_bar[s]), 0)
                                           : tc::smem_u32(&full_bar[s]);
            if (rank == 0) tc::mbar_arrive_expect_tx(&full_bar[s], R::kStage * CTAS);
            auto load = [&](void* dst, const CUtensorMap* map, int x, int y) {
              if (CTAS == 2) tc::tma_load_2d_pair(dst, map, bar, x, y);
              else tc::tma_load_2d(dst, map, &full_bar[s], x, y);
            };
            const int m0 = w.mb * BMU + rank * (BM * SUBS);   // this CTA's rows of A / D
            const int n0 = nt * BN + rank * R::kBRows;        // this CTA's rows of B
            if (MODE == kFwd || MODE == kDz || MODE == kE) {
#pragma unroll
              for (int sub = 0; sub < SUBS; ++sub)
                load(a_dst + sub * kABytes, &mapA, kb * BK, p.row0 + m0 + sub * BM);
              load(b_dst, &mapB, kb * BK, n0);
            } else if (MODE == kDh) {
#pragma unroll
              for (int sub = 0; sub < SUBS; ++sub)
                load(a_dst + sub * kABytes, &mapA, kb * BK, m0 + sub * BM);
#pragma unroll
              for (int j = 0; j < R::kBRows / 64; ++j)
                load(b_dst + j * kBoxBytes, &mapB, n0 + j * 64, kb * BK);
            } else {
#pragma unroll
              for (int j = 0; j < (BM * SUBS) / 64; ++j)
                load(a_dst + j * kBoxBytes, &mapA, m0 + j * 64, kb * BK);
#pragma unroll
              for (int j = 0; j < R::kBRows / 64; ++j)
                load(b_dst + j * kBoxBytes, &mapB, n0 + j * 64, p.b_row0 + kb * BK);
            }
          }
        }
      }
      // Tail: wait until every stage this thread filled has been released, so that no
      // arrival (from this CTA's MMA or the peer's) targets this CTA after it has left,
      // and no load is still writing its shared memory.  Bounded like every wait.
      const uint32_t pending = it < (uint32_t)kNS ? it : (uint32_t)kNS;
      for (uint32_t j = 0; j < pending; ++j) {
        const uint32_t jt = it - 1 - j;
        if (ok) {
          if (!tc::mbar_wait(&empty_bar[jt % kNS], (jt / kNS) & 1u, abort_flag)) ok = false;
        }
        if (!ok && CTAS == 1) {
          const uint64_t t0 = tc::global_timer_ns();
          while (!tc::mbar_try_wait(&full_bar[jt % kNS], (jt / kNS) & 1u)) {
            if (tc::global_timer_ns() - t0 > 100000000ull) break;
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (even CTA of a pair)
    if (lane == 0 && rank == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int u = unit0; ok && u < shape.n_units; u += unit_stride) {
        const Unit w = decode_unit<MODE, CTAS, SUBS>(p, shape, u);
        for (int nt = w.nt_lo; ok && nt < w.nt_hi; ++nt, ++tcount) {
          const uint32_t acc = tcount % kNAcc;
          const uint32_t aph = (tcount / kNAcc) & 1u;
          if (!tc::mbar_wait(&tempty_bar[acc], aph ^ 1u, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t d_tmem = tmem_base + acc * SUBS * BN;
          for (int kb = w.kb_lo; kb < w.kb_hi; ++kb, ++it) {
            const int s = it % kNS;
            const uint32_t ph = (it / kNS) & 1u;
            if (!tc::mbar_wait(&full_bar[s], ph, abort_flag)) { ok = false; break; }
            tc::fence_after_sync();
            const uint32_t a_base = tc::smem_u32(smem + (size_t)s * R::kStage);
            const uint32_t b_base = a_base + R::kABytesS;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
              for (int sub = 0; sub < SUBS; ++sub) {
              const uint32_t a_sub = a_base + sub * kABytes;
              // K-major: 16 elements of K are 32 bytes inside the swizzled
              // 128-byte row; 8-row groups are 1024 bytes apart.
              // MN-major: 16 rows of K are two 8-row groups 1024 bytes apart
              // (stride offset); 64-element groups along M/N are whole boxes
              // apart (leading offset).
              const uint64_t adesc =
                  kAmn ? tc::smem_desc_sw128(a_sub + kk * 2048, kBoxBytes, 1024)
                       : tc::smem_desc_sw128(a_sub + kk * 32, 16, 1024);
              const uint64_t bdesc =
                  kBmn ? tc::smem_desc_sw128(b_base + kk * 2048, kBoxBytes, 1024)
                       : tc::smem_desc_sw128(b_base + kk * 32, 16, 1024);
              if (CTAS == 2)
                tc::umma_bf16_pair(d_tmem + sub * BN, adesc, bdesc, kIdesc, (kb > w.kb_lo || kk > 0) ? 1u : 0u);
              else
                tc::umma_bf16(d_tmem + sub * BN, adesc, bdesc, kIdesc, (kb > w.kb_lo || kk > 0) ? 1u : 0u);
              }
            }
            if (CTAS == 2) tc::umma_commit_pair(&empty_bar[s], 3);
            else tc::umma_commit(&empty_bar[s]);
          }
          if (ok) {
            if (CTAS == 2) tc::umma_commit_pair(&tfull_bar[acc], 3);
            else tc::umma_commit(&tfull_bar[acc]);
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ epilogue (4 warps per A sub-tile)
    const int q = warp & 3;          // tensor-memory lane quadrant this warp may read
    const int sub = (warp - 2) >> 2;  // the A sub-tile whose rows this warp owns
    const int n_valid = p.row0 + shape.rows;  // compact rows below this are real tokens
    uint32_t tcount = 0;
    bool ok = true;
    for (int u = unit0; ok && u < shape.n_units; u += unit_stride) {
      const Unit w = decode_unit<MODE, CTAS, SUBS>(p, shape, u);
      int lrow = 0;  // row inside this launch's M range
      // per-unit row state
      float m_run = -INFINITY, s_run = 0.f, zt_val = 0.f;
      bool zt_found = false;
      int y = -1;
      float gk = 0.f, lk = 0.f, scale = 1.f;
      bool row_ok = false, over = false;
      {  // this thread's row and its scalars
        lrow = w.mb * BMU + rank * (BM * SUBS) + sub * BM + q * 32 + lane;
        y = -1;
        gk = 0.f;
        lk = 0.f;
        scale = 1.f;
        if (MODE != kDw) {
          const int k = p.row0 + lrow;
          row_ok = k < n_valid;
          if (row_ok) {
            if (MODE == kFwd || MODE == kDh || MODE == kE) y = p.targets[p.sel_idx[k]];
            // a target outside the vocabulary has g = 0 (its token is left out); keep the
            // one-hot row read in bounds
            if (MODE == kDh && (unsigned)y >= (unsigned)p.V) y = 0;
            if (MODE == kDz || MODE == kDh) gk = p.g[k];
            if (MODE == kDz) lk = p.lse[k];
            if (MODE == kE) lk = p.mref[k];
            if (MODE == kDh && p.row_scale != nullptr) scale = p.row_scale[k];
          }
        } else {
          row_ok = lrow < p.V;
        }
      }
      for (int nt = w.nt_lo; ok && nt < w.nt_hi; ++nt, ++tcount) {
        const uint32_t acc = tcount % kNAcc;
        const uint32_t aph = (tcount / kNAcc) & 1u;
        // every lane waits (each needs the accumulator's writes visible), then the
        // warp agrees on the outcome so the aligned tensor-memory loads stay converged
        ok = __all_sync(0xFFFFFFFFu, tc::mbar_wait(&tfull_bar[acc], aph, abort_flag) ? 1 : 0) != 0;
        if (!ok) break;
        tc::fence_after_sync();
        const int ncols = (MODE == kFwd || MODE == kDz || MODE == kE) ? p.V : p.d;
        const uint32_t taddr =
            tmem_base + ((uint32_t)(q * 32) << 16) + (acc * SUBS + (uint32_t)sub) * BN;
        if (MODE == kE && CTAS == 2) {
          // 64 columns at a time: two tensor-memory loads in flight, the numerators of the
          // warp's 32 rows x 64 columns go to its staging block (128-byte rows in the
          // 128-byte swizzle) and leave with one TMA store, which writes whole lines.
          uint8_t* stage = staging + (warp - 2) * 4096;
          const int row_base = w.mb * BMU + rank * (BM * SUBS) + sub * BM + q * 32;
          const float nm2 = lk * kLog2e;
#pragma unroll 1
          for (int c2 = 0; c2 < BN / 64; ++c2) {
            const int col0 = nt * BN + c2 * 64;
            if (col0 >= ncols) break;  // warp-uniform
            uint32_t ra[32], rb[32];
            tc::tmem_ld32_issue(taddr + c2 * 64, ra);
            tc::tmem_ld32_issue(taddr + c2 * 64 + 32, rb);
            tc::tmem_ld_wait(ra);
            tc::tmem_ld_pin(rb);
            const int nv = ncols - col0;  // valid columns from col0 on (may exceed 64)
            float part = 0.f;
            uint32_t packed[32];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float e0 = fast_exp2(fmaf(__uint_as_float(ra[2 * j]), kLog2e, -nm2));
              const float e1 = fast_exp2(fmaf(__uint_as_float(ra[2 * j + 1]), kLog2e, -nm2));
              if (2 * j < nv) part += e0;
              if (2 * j + 1 < nv) part += e1;
              packed[j] = pack_bf16(e0, e1);
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float e0 = fast_exp2(fmaf(__uint_as_float(rb[2 * j]), kLog2e, -nm2));
              const float e1 = fast_exp2(fmaf(__uint_as_float(rb[2 * j + 1]), kLog2e, -nm2));
              if (32 + 2 * j < nv) part += e0;
              if (33 + 2 * j < nv) part += e1;
              packed[16 + j] = pack_bf16(e0, e1);
            }
            if (!row_ok) {  // rows past the last token stay zero
              part = 0.f;
#pragma unroll
              for (int j = 0; j < 32; ++j) packed[j] = 0u;
            }
            s_run += part;
            // Any numerator above e^60 makes the sum exceed it too, so one compare per
            // piece catches every row that leaves the window.
            if (part > kWindowSum) over = true;
            if (y >= col0 && y < col0 + 64) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (col0 + j == y) zt_val = __uint_as_float(ra[j]);
                if (col0 + 32 + j == y) zt_val = __uint_as_float(rb[j]);
              }
              zt_found = true;
            }
            // the previous store of this warp has read its staging block
            if (lane == 0) tc::bulk_wait_read_all();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<uint4*>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                  make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tc::tma_store_2d(&mapC, stage, col0, row_base);
              tc::bulk_commit();
            }
          }
        } else
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          const int col0 = nt * BN + c * 32;
          if (col0 >= ncols) break;  // warp-uniform
          float v[32];
          tc::tmem_ld32(taddr + c * 32, v);
          if (MODE == kFwd) {
            const int nv = ncols - col0 < 32 ? ncols - col0 : 32;
            float cmax = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (j < nv) cmax = fmaxf(cmax, v[j]);
            const float m_new = fmaxf(m_run, cmax);
            const float mb2 = m_new * kLog2e;
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (j < nv) part += fast_exp2(fmaf(v[j], kLog2e, -mb2));
            s_run = s_run * fast_exp2((m_run - m_new) * kLog2e) + part;
            m_run = m_new;
            if (y >= col0 && y < col0 + 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j == y) zt_val = v[j];
              zt_found = true;
            }
          } else if (MODE == kE) {
            const int nv = ncols - col0 < 32 ? ncols - col0 : 32;
            const float nm2 = lk * kLog2e;
            float part = 0.f;
            uint32_t packed[16];
            if (row_ok) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const float e0 = fast_exp2(fmaf(v[2 * j], kLog2e, -nm2));
                const float e1 = fast_exp2(fmaf(v[2 * j + 1], kLog2e, -nm2));
                if (2 * j < nv) part += e0;
                if (2 * j + 1 < nv) part += e1;
                packed[j] = pack_bf16(e0, e1);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) packed[j] = 0u;  // rows past the last token stay zero
            }
            s_run += part;
            // Any numerator above e^60 makes the chunk's sum exceed it too, so one
            // compare per chunk catches every row that leaves the window (and at worst flags a
            // few rows that were still inside it, which only costs the redo).
            if (part > kWindowSum) over = true;
            if (y >= col0 && y < col0 + 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j == y) zt_val = v[j];
              zt_found = true;
            }
            __nv_bfloat16* dst = p.dZ + (size_t)lrow * p.ldz + col0;
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8)
              if (col0 + 8 * g8 < ncols)
                *reinterpret_cast<uint4*>(dst + 8 * g8) = make_uint4(
                    packed[4 * g8], packed[4 * g8 + 1], packed[4 * g8 + 2], packed[4 * g8 + 3]);
          } else if (MODE == kDz) {
            const float nl2 = lk * kLog2e;
            const float ng = -gk;
            uint32_t packed[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float p0 = ng * fast_exp2(fmaf(v[2 * j], kLog2e, -nl2));
              const float p1 = ng * fast_exp2(fmaf(v[2 * j + 1], kLog2e, -nl2));
              packed[j] = pack_bf16(p0, p1);
            }
            __nv_bfloat16* dst = p.dZ + (size_t)lrow * p.ldz + col0;
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8)
              if (col0 + 8 * g8 < ncols)
                *reinterpret_cast<uint4*>(dst + 8 * g8) = make_uint4(
                    packed[4 * g8], packed[4 * g8 + 1], packed[4 * g8 + 2], packed[4 * g8 + 3]);
          } else if (MODE == kDh && SUBS == 2 && p.k_splits > 1) {
            // partial tile of a K part: stored into the part's own slice of the float32
            // scratch through the warp's staging block (a TMA store of whole lines); the
            // slices are added in part order by dh_finalize_kernel, so the sum's order is fixed
            uint8_t* stage = staging + (warp - 2) * 4096;
            if (lane == 0) tc::bulk_wait_read_all();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<float4*>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                  make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tc::tma_store_2d(&mapC, stage, col0, w.sp * p.chunk_rows + lrow);
              tc::bulk_commit();
            }
          } else if (MODE == kDh) {
            if (row_ok) {
              const int k = p.row0 + lrow;
              const uint4* wsrc = reinterpret_cast<const uint4*>(p.W + (size_t)y * p.d + col0);
              uint4* dst = reinterpret_cast<uint4*>(p.dH + (size_t)k * p.d + col0);
#pragma unroll
              for (int g8 = 0; g8 < 4; ++g8) {
                const uint4 wv = __ldg(wsrc + g8);
                const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
                uint32_t o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const __nv_bfloat162 w2 = *reinterpret_cast<const __nv_bfloat162*>(&ww[e]);
                  const float lo = fmaf(gk, __low2float(w2), scale * v[8 * g8 + 2 * e]);
                  const float hi = fmaf(gk, __high2float(w2), scale * v[8 * g8 + 2 * e + 1]);
                  o[e] = pack_bf16(lo, hi);
                }
                dst[g8] = make_uint4(o[0], o[1], o[2], o[3]);
              }
            }
          } else if (SUBS == 2) {
            // dW += tile: the warp's 32 rows x 32 columns go to its staging block (128-byte
            // rows in the 128-byte swizzle) and leave as one TMA reduction, which the L2
            // applies to whole lines; rows past V are clipped by the tensor map.  Every
            // element is touched once per launch and launches are stream-ordered, so the
            // sum's order is fixed.
            uint8_t* stage = staging + (warp - 2) * 4096;
            if (lane == 0) tc::bulk_wait_read_all();  // the previous reduction has read the block
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<float4*>(stage + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                  make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            tc::fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tc::tma_reduce_add_2d(&mapC, stage, col0, lrow);
              tc::bulk_commit();
            }
          } else {
            if (row_ok) {
              // dW += tile: 16-byte reductions performed by the L2 (nothing comes back to
              // the SM, so the epilogue does not wait on DRAM).  Every element is touched by
              // one thread per launch and launches are stream-ordered: the sum's order is fixed.
              float* dst = p.dW + (size_t)lrow * p.d + col0;
#pragma unroll
              for (int g4 = 0; g4 < 8; ++g4)
                tc::red_add_f32x4(dst + 4 * g4, v[4 * g4], v[4 * g4 + 1], v[4 * g4 + 2],
                                  v[4 * g4 + 3]);
            }
          }
        }
        tc::fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          if (CTAS == 2) tc::mbar_arrive_cluster(tc::map_to_cta(tc::smem_u32(&tempty_bar[acc]), 0));
          else tc::mbar_arrive(&tempty_bar[acc]);
        }
      }
      if (MODE == kFwd && ok && row_ok) {
        const int k = p.row0 + lrow;
        p.part_m[(size_t)w.sp * p.cap_pad + k] = m_run;
        p.part_s[(size_t)w.sp * p.cap_pad + k] = s_run;
        if (zt_found) p.zt[k] = zt_val;
      }
      if (MODE == kE && ok && row_ok) {
        // one partial row sum per vocabulary tile, local to the chunk: [tile][row in chunk]
        p.part_s[(size_t)w.sp * p.cap_pad + lrow] = s_run;
        if (zt_found) p.zt[p.row0 + lrow] = zt_val;
        if (over) *p.ovf = 1;
      }
    }
  }

  if (CTAS == 2 && warp >= 2 && lane == 0) tc::bulk_wait_all();  // this warp's stores are done
  tc::fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag != 0u) atomicOr(p.status, NAT_DEV_TIMEOUT);
  if (CTAS == 2) tc::cluster_sync_all();  // the pair leaves together
  if (warp == 1) {
    tc::fence_after_sync();
    if (CTAS == 2) tc::tmem_dealloc_pair(tmem_base, kTmemCols);
    else tc::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------- small kernels
__device__ __forceinline__ bool predicate_off(const int32_t* flag, int run_if) {
  return flag != nullptr && ((*flag != 0) ? 1 : 0) != run_if;
}

// Hc[k, :] = hidden[row(k), :] for k < n_sel, zero up to rows_pad, so that
// every tile the tensor-core kernels touch holds finite values.
__global__ void gather_rows_kernel(const __nv_bfloat16* __restrict__ hidden,
                                   const int32_t* __restrict__ sel_idx, int compact,
                                   const int32_t* __restrict__ n_sel, int cap, int rows_pad, int d,
                                   __nv_bfloat16* __restrict__ Hc) {
  int n = *n_sel;
  n = n < cap ? n : cap;
  const int vec = d / 8;
  for (int k = blockIdx.x; k < rows_pad; k += gridDim.x) {
    uint4* dst = reinterpret_cast<uint4*>(Hc + (size_t)k * d);
    if (k < n) {
      const int64_t row = compact ? (int64_t)k : (int64_t)sel_idx[k];
      const uint4* src = reinterpret_cast<const uint4*>(hidden + row * d);
      for (int j = threadIdx.x; j < vec; j += blockDim.x) dst[j] = __ldg(src + j);
    } else {
      for (int j = threadIdx.x; j < vec; j += blockDim.x) dst[j] = make_uint4(0, 0, 0, 0);
    }
  }
}

// Rows [row0, row0 + rows_max): combine the per-split (max, sum-exp) pairs of each row,
// then the token's log-probability, its share of the loss and (when g_out is given) its
// gradient coefficient.
__global__ void fwd_finalize_kernel(TokenCtx c, const int32_t* __restrict__ n_sel, int cap,
                                    int row0, int rows_max, int n_splits, int cap_pad,
                                    const float* __restrict__ part_m,
                                    const float* __restrict__ part_s, const float* __restrict__ zt,
                                    float* __restrict__ logp, float* __restrict__ lse,
                                    float* __restrict__ term, float* __restrict__ g_out,
                                    const float* __restrict__ dloss,
                                    const int32_t* __restrict__ flag, int run_if) {
  if (predicate_off(flag, run_if)) return;
  int n = *n_sel;
  n = n < cap ? n : cap;
  const int end = n < row0 + rows_max ? n : row0 + rows_max;
  const float dl = dloss ? *dloss : 1.f;
  for (int k = row0 + blockIdx.x * blockDim.x + threadIdx.x; k < end;
       k += gridDim.x * blockDim.x) {
    float M = -INFINITY;
    for (int sp = 0; sp < n_splits; ++sp) M = fmaxf(M, part_m[(size_t)sp * cap_pad + k]);
    float S = 0.f;
    for (int sp = 0; sp < n_splits; ++sp)
      S += part_s[(size_t)sp * cap_pad + k] * expf(part_m[(size_t)sp * cap_pad + k] - M);
    const float l = M + logf(S);
    const float lp = target_ok(c, k) ? zt[k] - l : __int_as_float(0x7FC00000);
    lse[k] = l;
    logp[k] = lp;
    float t, g;
    token_eval(c, k, lp, dl, &t, &g);
    term[k] = t;
    if (g_out) g_out[k] = g;
  }
}

// Single-pass route, rows [row0, row0 + chunk_rows) (one block per row): from the row
// sums of E = exp(z - mref): lse = mref + log sum, logp, loss term, g, the row factor
// c = -g / sum, and Hs[row - row0, :] = c * Hc[row, :].  Rows past the last selected
// token are zero-filled in Hs.
__global__ void __launch_bounds__(128)
fused_finalize_kernel(TokenCtx c, const int32_t* __restrict__ n_sel, int cap, int row0,
                      int chunk_rows, int n_parts, const float* __restrict__ mref,
                      const float* __restrict__ part_s, const float* __restrict__ zt,
                      const float* __restrict__ dloss, float* __restrict__ logp,
                      float* __restrict__ lse, float* __restrict__ term, float* __restrict__ g_out,
                      float* __restrict__ cs, const __nv_bfloat16* __restrict__ Hc,
                      __nv_bfloat16* __restrict__ Hs, int d, const int32_t* __restrict__ flag) {
  if (predicate_off(flag, 0)) return;
  __shared__ float c_s;
  __shared__ float warp_sum[4];
  int n = *n_sel;
  n = n < cap ? n : cap;
  const float dl = dloss ? *dloss : 1.f;
  const int vec = d / 8;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = blockIdx.x; r < chunk_rows; r += gridDim.x) {
    const int k = row0 + r;
    if (k >= n && r >= ((n - row0 + kRowPad - 1) / kRowPad) * kRowPad) break;  // beyond the tiles in use
    __syncthreads();
    if (k < n) {
      // the row's sum of numerators: one partial per vocabulary tile, [tile][row in chunk];
      // every thread adds a strided share, then a fixed tree combines them
      float part = 0.f;
      for (int sp = threadIdx.x; sp < n_parts; sp += 128)
        part += part_s[(size_t)sp * chunk_rows + r];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
      if (lane == 0) warp_sum[warp] = part;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      float cv = 0.f;
      if (k < n) {
        const float S = (warp_sum[0] + warp_sum[1]) + (warp_sum[2] + warp_sum[3]);
        const float l = mref[k] + logf(S);
        const float lp = target_ok(c, k) ? zt[k] - l : __int_as_float(0x7FC00000);
        lse[k] = l;
        logp[k] = lp;
        float t, g;
        token_eval(c, k, lp, dl, &t, &g);
        term[k] = t;
        g_out[k] = g;
        cv = -g / S;
        cs[k] = cv;
      }
      c_s = cv;
    }
    __syncthreads();
    const float cv = c_s;
    uint4* dst = reinterpret_cast<uint4*>(Hs + (size_t)r * d);
    if (cv == 0.f) {
      for (int j = threadIdx.x; j < vec; j += blockDim.x) dst[j] = make_uint4(0, 0, 0, 0);
    } else {
      const uint4* src = reinterpret_cast<const uint4*>(Hc + (size_t)k * d);
      for (int j = threadIdx.x; j < vec; j += blockDim.x) {
        const uint4 hv = src[j];
        const uint32_t in[4] = {hv.x, hv.y, hv.z, hv.w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162*>(&in[e]);
          o[e] = pack_bf16(cv * __low2float(h2), cv * __high2float(h2));
        }
        dst[j] = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// dHidden of one row chunk from the float32 partial tiles of the K parts (kDh with
// k_splits > 1), slice p of `acc` holding part p's [chunk_rows, d] partial sums:
//   dH[k, :] = scale_k * (sum over parts in ascending order of acc[p][k - row0, :]) + g_k W[y_k, :]
// (one block per row).
__global__ void __launch_bounds__(128)
dh_finalize_kernel(const float* __restrict__ acc, const float* __restrict__ row_scale,
                   const float* __restrict__ g, const __nv_bfloat16* __restrict__ W,
                   const int32_t* __restrict__ targets, const int32_t* __restrict__ sel_idx,
                   const int32_t* __restrict__ n_sel, int cap, int row0, int chunk_rows, int d,
                   int V, int parts, __nv_bfloat16* __restrict__ dH,
                   const int32_t* __restrict__ flag, int run_if) {
  if (predicate_off(flag, run_if)) return;
  int n = *n_sel;
  n = n < cap ? n : cap;
  const int vec = d / 8;
  for (int r = blockIdx.x; r < chunk_rows; r += gridDim.x) {
    const int k = row0 + r;
    if (k >= n) break;
    const float scale = row_scale ? row_scale[k] : 1.f;
    const float gk = g[k];
    int y = targets[sel_idx[k]];
    if ((unsigned)y >= (unsigned)V) y = 0;  // such a token has g = 0
    const float4* a = reinterpret_cast<const float4*>(acc + (size_t)r * d);
    const uint4* wsrc = reinterpret_cast<const uint4*>(W + (size_t)y * d);
    uint4* dst = reinterpret_cast<uint4*>(dH + (size_t)k * d);
    const size_t slice4 = (size_t)chunk_rows * d / 4;  // float4 elements per part
    for (int j = threadIdx.x; j < vec; j += blockDim.x) {
      float4 a0 = a[2 * j], a1 = a[2 * j + 1];
      for (int q = 1; q < parts; ++q) {
        const float4 b0 = a[q * slice4 + 2 * j], b1 = a[q * slice4 + 2 * j + 1];
        a0.x += b0.x; a0.y += b0.y; a0.z += b0.z; a0.w += b0.w;
        a1.x += b1.x; a1.y += b1.y; a1.z += b1.z; a1.w += b1.w;
      }
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const uint4 wv = __ldg(wsrc + j);
      const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat162 w2 = *reinterpret_cast<const __nv_bfloat162*>(&ww[e]);
        o[e] = pack_bf16(fmaf(gk, __low2float(w2), scale * av[2 * e]),
                         fmaf(gk, __high2float(w2), scale * av[2 * e + 1]));
      }
      dst[j] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// Records that some chunk left the single-pass window (informational status bit).
__global__ void note_fallback_kernel(const int32_t* __restrict__ ovf, int n_chunks,
                                     uint32_t* status) {
  for (int c = threadIdx.x; c < n_chunks; c += blockDim.x)
    if (ovf[c] != 0) atomicOr(status, NAT_DEV_FALLBACK);
}

// One-hot part of dW: dW[y_k, :] += g_k h_k.  Tokens that share a target meet in the same
// row of dW; to keep the sum's order fixed (and with it the bits of dW) the tokens are first
// grouped by target, each group sorted by token index, and every row then receives its
// tokens in ascending order from a single thread per column:
//   count   tokens per target (integer atomics: the counts do not depend on their order)
//   scan    exclusive scan of the counts over the vocabulary -> group offsets
//   fill    every token takes a slot of its group (the slot order is arbitrary)
//   rank    every token counts the smaller indices of its group -> its sorted position
//   apply   one block per target and 1024-column slice walks the sorted group
__global__ void onehot_count_kernel(const int32_t* __restrict__ targets,
                                    const int32_t* __restrict__ sel_idx,
                                    const float* __restrict__ g, const int32_t* __restrict__ n_sel,
                                    int cap, int V, int32_t* __restrict__ count) {
  int n = *n_sel;
  n = n < cap ? n : cap;
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n; k += gridDim.x * blockDim.x) {
    if (g[k] == 0.f) continue;
    const int y = targets[sel_idx[k]];
    if ((unsigned)y < (unsigned)V) atomicAdd(&count[y], 1);
  }
}

// off[v] = number of tokens whose target is below v (off[V] = all of them); the counts are
// cleared on the way so that they can serve as the groups' fill cursors.
__global__ void __launch_bounds__(1024)
onehot_scan_kernel(int32_t* __restrict__ count, int V, int32_t* __restrict__ off) {
  __shared__ int warp_tot[2][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int carry = 0;
  for (int base = 0, tile = 0; base < V; base += 4096, ++tile) {
    const int v0 = base + (int)threadIdx.x * 4;
    int c[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      c[e] = v0 + e < V ? count[v0 + e] : 0;
      if (v0 + e < V) count[v0 + e] = 0;
    }
    const int sum = c[0] + c[1] + c[2] + c[3];
    int incl = sum;
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
    int e0 = carry + warp_excl + incl - sum;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (v0 + e < V) off[v0 + e] = e0;
      e0 += c[e];
    }
    carry += tile_total;
  }
  if (threadIdx.x == 0) off[V] = carry;
}

__global__ void onehot_fill_kernel(const int32_t* __restrict__ targets,
                                   const int32_t* __restrict__ sel_idx,
                                   const float* __restrict__ g, const int32_t* __restrict__ n_sel,
                                   int cap, int V, const int32_t* __restrict__ off,
                                   int32_t* __restrict__ cursor, int32_t* __restrict__ list) {
  int n = *n_sel;
  n = n < cap ? n : cap;
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n; k += gridDim.x * blockDim.x) {
    if (g[k] == 0.f) continue;
    const int y = targets[sel_idx[k]];
    if ((unsigned)y < (unsigned)V) list[off[y] + atomicAdd(&cursor[y], 1)] = k;
  }
}

__global__ void onehot_rank_kernel(const int32_t* __restrict__ targets,
                                   const int32_t* __restrict__ sel_idx, int V,
                                   const int32_t* __restrict__ off,
                                   const int32_t* __restrict__ list,
                                   int32_t* __restrict__ sorted) {
  const int n_live = off[V];
  for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < n_live; p += gridDim.x * blockDim.x) {
    const int k = list[p];
    const int y = targets[sel_idx[k]];
    const int lo = off[y], hi = off[y + 1];
    int rank = 0;
    for (int j = lo; j < hi; ++j) rank += list[j] < k ? 1 : 0;
    sorted[lo + rank] = k;
  }
}

// blockIdx.y selects a slice of 1024 columns (four per thread); rows are taken grid-stride.
__global__ void __launch_bounds__(256)
onehot_apply_kernel(const __nv_bfloat16* __restrict__ Hc, const float* __restrict__ g, int V,
                    int d, const int32_t* __restrict__ off, const int32_t* __restrict__ sorted,
                    float* __restrict__ dW) {
  const int col = (blockIdx.y * 256 + threadIdx.x) * 4;
  if (col >= d) return;
  for (int y = blockIdx.x; y < V; y += gridDim.x) {
    const int lo = off[y], hi = off[y + 1];
    if (lo == hi) continue;
    float* dst = dW + (size_t)y * d + col;
    float4 acc = *reinterpret_cast<const float4*>(dst);
    for (int e = lo; e < hi; ++e) {
      const int k = sorted[e];
      const float gk = g[k];
      const uint2 hv = *reinterpret_cast<const uint2*>(Hc + (size_t)k * d + col);
      const __nv_bfloat162 h01 = *reinterpret_cast<const __nv_bfloat162*>(&hv.x);
      const __nv_bfloat162 h23 = *reinterpret_cast<const __nv_bfloat162*>(&hv.y);
      acc.x = fmaf(gk, __low2float(h01), acc.x);
      acc.y = fmaf(gk, __high2float(h01), acc.y);
      acc.z = fmaf(gk, __low2float(h23), acc.z);
      acc.w = fmaf(gk, __high2float(h23), acc.w);
    }
    *reinterpret_cast<float4*>(dst) = acc;
  }
}

// ------------------------------------------------------------- host side
struct Layout {
  int cap_pad, n_tiles, n_splits, chunk_rows, n_chunks, ldz;
  int dh_splits;  // K parts of the dHidden contraction (1: direct epilogue)
  size_t off_term, off_g, off_zt, off_pm, off_ps, off_pe, off_mref, off_cs, off_ovf, off_prog,
      off_ohc, off_oho, off_ohl, off_ohs, off_hc, off_hs, off_dhacc, off_dz, total;
};

// Number of vocabulary splits.  A work unit of the vocabulary sweeps is (block of rows,
// split); the CTA pairs take units round-robin, so the sweep of a full row chunk lasts
// ceil(units / pairs) rounds of about n_tiles / splits tiles each.  Choose the split count
// that makes this product smallest with 8..32 tiles per unit (long enough to amortise the
// per-unit state, short enough to balance), preferring lengths near kTilesPerSplit on ties.
int pick_splits(int n_tiles, int m_units, int slots) {
  if (slots <= 0) slots = 74;  // CTA pairs of a whole B200; only a tuning assumption
  if (m_units <= 0) m_units = 1;
  int best = 0;
  double best_cost = 0.0;
  for (int s = 1; s <= n_tiles; ++s) {
    const int per = (n_tiles + s - 1) / s;
    if (per > 32) continue;
    if (per < 8 && best > 0) break;
    const long long units = (long long)m_units * s;
    const long long rounds = (units + slots - 1) / slots;
    const int gap = per > kTilesPerSplit ? per - kTilesPerSplit : kTilesPerSplit - per;
    const double cost = (double)rounds * ((double)n_tiles / s) * (1.0 + 1e-4 * gap);
    if (best == 0 || cost < best_cost) {
      best = s;
      best_cost = cost;
    }
  }
  return best > 0 ? best : 1;
}

int pair_slots();

// Number of K parts of the dHidden contraction.  Its work units are (512-row block,
// 256-column block) tiles over the whole vocabulary as K: few and long (256 for a full chunk
// at d = 4096), so the last round of the CTA pairs is mostly empty.  Cutting K into parts
// multiplies the units; every part has its own float32 slice of a scratch and a small pass
// adds the slices in part order (a fixed order: dHidden is reproducible).  The smallest count
// that fills the rounds to 95 % is taken (1 when CTA pairs are not available).
int pick_k_splits(int tiles, int kb, int slots) {
  if (slots <= 0 || tiles <= 0) return 1;
  int best = 1;
  double best_eff = 0.0;
  for (int s = 1; s <= 8; ++s) {
    if (s > 1 && kb / s < 64) break;
    const long long units = (long long)tiles * s;
    const double eff = (double)units / (double)(((units + slots - 1) / slots) * slots);
    if (eff > best_eff + 1e-9) {
      best = s;
      best_eff = eff;
    }
    if (eff >= 0.95) return s;
  }
  return best;
}

// Hidden sizes from which the single-pass sweep uses 512-row work units (see launch_tc).
bool wide_sweep(int d) { return d >= 2048; }

Layout make_layout(const nat_loss_params& p, int64_t cap) {
  Layout L;
  const int64_t c1 = cap > 0 ? cap : 1;
  L.cap_pad = (int)((c1 + kRowPad - 1) / kRowPad * kRowPad);
  L.n_tiles = (p.V + BN - 1) / BN;
  L.chunk_rows = L.cap_pad < kChunkRows ? L.cap_pad : kChunkRows;
  // tuned for the single-pass sweep, whose units cover 512 or 256 rows on CTA pairs
  L.n_splits = pick_splits(L.n_tiles, L.chunk_rows / (wide_sweep(p.d) ? 512 : 256), pair_slots());
  L.n_chunks = (L.cap_pad + L.chunk_rows - 1) / L.chunk_rows;
  L.ldz = (p.V + 63) / 64 * 64;
  L.dh_splits = pick_k_splits((L.chunk_rows / 512) * ((p.d + BN - 1) / BN), (p.V + BK - 1) / BK,
                              pair_slots());
  size_t off = sizeof(WorkspaceHead);
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes, 1024);
    return o;
  };
  L.off_term = take(sizeof(float) * L.cap_pad);
  L.off_g = take(sizeof(float) * L.cap_pad);
  L.off_zt = take(sizeof(float) * L.cap_pad);
  L.off_pm = take(sizeof(float) * (size_t)L.cap_pad * L.n_splits);
  L.off_ps = take(sizeof(float) * (size_t)L.cap_pad * L.n_splits);
  L.off_pe = take(sizeof(float) * (size_t)L.chunk_rows * L.n_tiles);
  L.off_mref = take(sizeof(float) * L.cap_pad);
  L.off_cs = take(sizeof(float) * L.cap_pad);
  L.off_ovf = take(sizeof(int32_t) * L.n_chunks);
  L.off_prog = take(sizeof(unsigned long long) * kMaxPairs);
  L.off_ohc = take(sizeof(int32_t) * (size_t)p.V);
  L.off_oho = take(sizeof(int32_t) * ((size_t)p.V + 1));
  L.off_ohl = take(sizeof(int32_t) * L.cap_pad);
  L.off_ohs = take(sizeof(int32_t) * L.cap_pad);
  off = align_up(off, 1024);
  L.off_hc = take(sizeof(__nv_bfloat16) * (size_t)L.cap_pad * p.d);
  L.off_hs = take(sizeof(__nv_bfloat16) * (size_t)L.chunk_rows * p.d);
  L.off_dhacc = take(L.dh_splits > 1 ? sizeof(float) * (size_t)L.dh_splits * L.chunk_rows * p.d : 0);
  L.off_dz = take(sizeof(__nv_bfloat16) * (size_t)L.chunk_rows * L.ldz);
  L.total = off;
  return L;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int get_encoder(EncodeTiledFn* out) {
  static EncodeTiledFn cached = nullptr;
  if (!cached) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    NAT_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !fn)
      return fail(NAT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cached = reinterpret_cast<EncodeTiledFn>(fn);
  }
  *out = cached;
  return NAT_OK;
}

// bf16 matrix [rows, inner] with the given row pitch; box = box_inner x box_rows
// elements, 128-byte swizzle, out-of-range elements read as zero.
int make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows,
             uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows) {
  EncodeTiledFn enc;
  int s = get_encoder(&enc);
  if (s != NAT_OK) return s;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(NAT_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return NAT_OK;
}

// float32 matrix [rows, inner] as a reduction target: box = 32 x 32 elements (128-byte rows).
int make_map_f32(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows) {
  EncodeTiledFn enc;
  int s = get_encoder(&enc);
  if (s != NAT_OK) return s;
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * 4};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(NAT_ERR_CUDA, "cuTensorMapEncodeTiled (float32) failed with code %d", (int)r);
  return NAT_OK;
}

// Per-device facts are cached per device index: one process may drive several GPUs.
constexpr int kMaxDevices = 64;

int current_device(int* dev) {
  NAT_CUDA(cudaGetDevice(dev));
  if (*dev < 0 || *dev >= kMaxDevices)
    return fail(NAT_ERR_UNSUPPORTED, "device index %d is beyond the %d this library tracks", *dev,
                kMaxDevices);
  return NAT_OK;
}

int sm_count(int* out) {
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  int s = current_device(&dev);
  if (s != NAT_OK) return s;
  int v = cached[dev].load();
  if (v == 0) {
    NAT_CUDA(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
    cached[dev].store(v);
  }
  *out = v;
  return NAT_OK;
}


// CTA pairs (cta_group::2) halve each CTA's share of the B operand and are used whenever
// the device can co-schedule 2-CTA clusters of this kernel on (nearly) all of its SMs;
// otherwise (e.g. a partitioned GPU) the single-CTA kernels run.
int pair_slots() {
  static std::atomic<int> cached[kMaxDevices];  // 0 = unknown, -1 = none, else the count
  int dev = 0;
  if (current_device(&dev) != NAT_OK) return 0;
  int slots = cached[dev].load();
  if (slots == 0) {
    slots = -1;
    int sms = 0;
    if (sm_count(&sms) == NAT_OK &&
        cudaFuncSetAttribute(nat_tc_kernel<kFwd, 2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)Ring<2, 1>::kSmem) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)sms, 1, 1);
      cfg.blockDim = dim3(threads_for(1), 1, 1);
      cfg.dynamicSmemBytes = Ring<2, 1>::kSmem;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&clusters, nat_tc_kernel<kFwd, 2, 1>, &cfg) == cudaSuccess &&
          clusters * 2 * 10 >= sms * 9)
        slots = clusters;
    }
    (void)cudaGetLastError();
    cached[dev].store(slots);
  }
  return slots > 0 ? slots : 0;
}

// ---- optional per-kernel timing (nat_trace_begin / nat_trace_end) ----------------
struct TraceSpan {
  int kind;
  cudaEvent_t t0, t1;
};
std::mutex g_trace_mutex;
bool g_trace_on = false;
std::vector<TraceSpan> g_trace_spans;

template <int MODE, int CTAS, int SUBS>
int launch_tc_impl(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c,
                   const TcParams& p, int max_units, cudaStream_t stream) {
  static std::atomic<bool> configured[kMaxDevices];
  int dev = 0;
  int sd = current_device(&dev);
  if (sd != NAT_OK) return sd;
  if (!configured[dev].load()) {
    NAT_CUDA(cudaFuncSetAttribute(nat_tc_kernel<MODE, CTAS, SUBS>,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)Ring<CTAS, SUBS>::kSmem));
    configured[dev].store(true);
  }
  int sms = 0;
  int s = sm_count(&sms);
  if (s != NAT_OK) return s;
  const int slots = CTAS == 2 ? pair_slots() : sms;
  const int groups = max_units < slots ? max_units : slots;
  if (groups <= 0) return NAT_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(groups * CTAS), 1, 1);
  cfg.blockDim = dim3(threads_for(SUBS), 1, 1);
  cfg.dynamicSmemBytes = Ring<CTAS, SUBS>::kSmem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  bool traced = false;
  TraceSpan span{MODE, nullptr, nullptr};
  {
    std::lock_guard<std::mutex> lock(g_trace_mutex);
    traced = g_trace_on;
  }
  if (traced) {
    NAT_CUDA(cudaEventCreate(&span.t0));
    NAT_CUDA(cudaEventCreate(&span.t1));
    NAT_CUDA(cudaEventRecord(span.t0, stream));
  }
  NAT_CUDA(cudaLaunchKernelEx(&cfg, nat_tc_kernel<MODE, CTAS, SUBS>, a, b, c, p));
  if (traced) {
    NAT_CUDA(cudaEventRecord(span.t1, stream));
    std::lock_guard<std::mutex> lock(g_trace_mutex);
    g_trace_spans.push_back(span);
  }
  return NAT_OK;
}

// `units128`: number of work units when the M dimension is cut into 128-row blocks
// (m_blocks128 * per_block); a pair covers two such blocks per unit.
template <int MODE>
int launch_tc(const CUtensorMap& a, const CUtensorMap& b1, const CUtensorMap& b2,
              const CUtensorMap& c, const TcParams& p, int m_blocks128, int per_block,
              cudaStream_t stream) {
  // Every launch gets a fresh epoch, so progress marks left by earlier launches (or
  // whatever the workspace held before) compare as "not there yet" or are overwritten
  // by their owner's first tile; either way they cannot stall this launch for long.
  static std::atomic<unsigned long long> epoch_counter{0};
  TcParams q = p;
  q.epoch = (epoch_counter.fetch_add(1) + 1) & 0x7FFFFFull;
  // dH and dW (long K) always take two A sub-tiles per CTA.  The single-pass sweep kE takes
  // two when the hidden size is large: its 512x256 tile fills tensor memory, so its epilogue
  // is exposed, which pays only while a tile's MMAs (proportional to d) dwarf it; for small d
  // it keeps 256x256 tiles whose epilogue overlaps the next tile.  kFwd / kDz keep one.
  if (pair_slots() > 0) {
    const bool two = MODE == kDh || MODE == kDw || (MODE == kE && wide_sweep(p.d));
    if (two)
      return launch_tc_impl<MODE, 2, (MODE == kFwd || MODE == kDz) ? 1 : 2>(
          a, b2, c, q, ((m_blocks128 + 3) / 4) * per_block, stream);
    return launch_tc_impl<MODE, 2, (MODE == kDh || MODE == kDw) ? 2 : 1>(
        a, b2, c, q, ((m_blocks128 + 1) / 2) * per_block, stream);
  }
  return launch_tc_impl<MODE, 1, 1>(a, b1, c, q, m_blocks128 * per_block, stream);
}

struct Ws {
  WorkspaceHead* head;
  float *term, *g, *zt, *pm, *ps, *pe, *mref, *cs, *dhacc;
  int32_t* ovf;
  unsigned long long* prog;
  int32_t *oh_count, *oh_off, *oh_list, *oh_sorted;  // grouping of the tokens by target
  __nv_bfloat16 *hc, *hs, *dz;
};

Ws carve(void* ws, const Layout& L) {
  char* b = reinterpret_cast<char*>(ws);
  Ws w;
  w.head = reinterpret_cast<WorkspaceHead*>(b);
  w.term = reinterpret_cast<float*>(b + L.off_term);
  w.g = reinterpret_cast<float*>(b + L.off_g);
  w.zt = reinterpret_cast<float*>(b + L.off_zt);
  w.pm = reinterpret_cast<float*>(b + L.off_pm);
  w.ps = reinterpret_cast<float*>(b + L.off_ps);
  w.pe = reinterpret_cast<float*>(b + L.off_pe);
  w.dhacc = reinterpret_cast<float*>(b + L.off_dhacc);
  w.mref = reinterpret_cast<float*>(b + L.off_mref);
  w.cs = reinterpret_cast<float*>(b + L.off_cs);
  w.ovf = reinterpret_cast<int32_t*>(b + L.off_ovf);
  w.prog = reinterpret_cast<unsigned long long*>(b + L.off_prog);
  w.oh_count = reinterpret_cast<int32_t*>(b + L.off_ohc);
  w.oh_off = reinterpret_cast<int32_t*>(b + L.off_oho);
  w.oh_list = reinterpret_cast<int32_t*>(b + L.off_ohl);
  w.oh_sorted = reinterpret_cast<int32_t*>(b + L.off_ohs);
  w.hc = reinterpret_cast<__nv_bfloat16*>(b + L.off_hc);
  w.hs = reinterpret_cast<__nv_bfloat16*>(b + L.off_hs);
  w.dz = reinterpret_cast<__nv_bfloat16*>(b + L.off_dz);
  return w;
}

TcParams base_params(const LossArgs& a, const Layout& L, const Ws& w) {
  TcParams p{};
  p.n_sel = a.n_sel;
  p.cap = (int)a.cap;
  p.row0 = 0;
  p.chunk_rows = L.cap_pad;
  p.d = a.p.d;
  p.V = a.p.V;
  p.n_splits = L.n_splits;
  p.cap_pad = L.cap_pad;
  p.targets = a.targets;
  p.sel_idx = a.sel_idx;
  p.part_m = w.pm;
  p.part_s = w.ps;
  p.zt = w.zt;
  p.g = w.g;
  p.lse = a.lse;
  p.dZ = w.dz;
  p.ldz = L.ldz;
  p.W = reinterpret_cast<const __nv_bfloat16*>(a.W);
  p.dH = reinterpret_cast<__nv_bfloat16*>(a.dHidden);
  p.dW = a.dW;
  p.status = &w.head->status;
  p.mref = w.mref;
  p.row_scale = nullptr;
  p.b_row0 = 0;
  p.k_splits = 1;
  p.flag = nullptr;
  p.run_if = 0;
  p.ovf = nullptr;
  p.progress = w.prog;
  p.epoch = 0;
  return p;
}

int gather(const LossArgs& a, const Layout& L, const Ws& w) {
  const int grid = L.cap_pad < 4096 ? L.cap_pad : 4096;
  gather_rows_kernel<<<grid, 128, 0, a.stream>>>(
      reinterpret_cast<const __nv_bfloat16*>(a.hidden), a.sel_idx, a.p.hidden_is_compact, a.n_sel,
      (int)a.cap, L.cap_pad, a.p.d, w.hc);
  NAT_LAUNCH_CHECK("gather_rows_kernel");
  return NAT_OK;
}

struct Maps {
  CUtensorMap hcK, wK, wK2, dzK, wMn, dzMn, hcMn, hsMn;  // wK2: 128-row boxes for CTA pairs
  CUtensorMap dzSt;  // the numerator scratch as a store target: 64 columns x 32 rows
  CUtensorMap dwRed;  // dW as a reduction target (valid only when the call has a dW)
  CUtensorMap dhAcc;  // the float32 scratch of the dHidden K parts: [parts x chunk_rows, d]
};

int encode_maps(const LossArgs& a, const Layout& L, const Ws& w, Maps* m) {
  int s;
  const uint64_t dpitch = (uint64_t)a.p.d * 2, zpitch = (uint64_t)L.ldz * 2;
  if ((s = make_map(&m->hcK, w.hc, a.p.d, L.cap_pad, dpitch, BK, BM)) != NAT_OK) return s;
  if ((s = make_map(&m->wK, a.W, a.p.d, a.p.V, dpitch, BK, BN)) != NAT_OK) return s;
  if ((s = make_map(&m->wK2, a.W, a.p.d, a.p.V, dpitch, BK, BN / 2)) != NAT_OK) return s;
  if ((s = make_map(&m->dzK, w.dz, a.p.V, L.chunk_rows, zpitch, BK, BM)) != NAT_OK) return s;
  if ((s = make_map(&m->wMn, a.W, a.p.d, a.p.V, dpitch, 64, BK)) != NAT_OK) return s;
  if ((s = make_map(&m->dzMn, w.dz, a.p.V, L.chunk_rows, zpitch, 64, BK)) != NAT_OK) return s;
  if ((s = make_map(&m->hcMn, w.hc, a.p.d, L.cap_pad, dpitch, 64, BK)) != NAT_OK) return s;
  if ((s = make_map(&m->hsMn, w.hs, a.p.d, L.chunk_rows, dpitch, 64, BK)) != NAT_OK) return s;
  if ((s = make_map(&m->dzSt, w.dz, a.p.V, L.chunk_rows, zpitch, 64, 32)) != NAT_OK) return s;
  m->dwRed = m->dzSt;
  if (a.dW != nullptr && (s = make_map_f32(&m->dwRed, a.dW, a.p.d, a.p.V)) != NAT_OK) return s;
  m->dhAcc = m->dzSt;
  if (L.dh_splits > 1 &&
      (s = make_map_f32(&m->dhAcc, w.dhacc, a.p.d, (uint64_t)L.dh_splits * L.chunk_rows)) != NAT_OK)
    return s;
  return NAT_OK;
}

// dHidden of one row chunk: the contraction (in K parts when that fills the device better)
// and, for K parts, the pass that forms dHidden from their float32 sum.
int launch_dh(const LossArgs& a, const Layout& L, const Ws& w, const Maps& m, TcParams p,
              const int32_t* flag, int run_if);

// The tensor maps depend only on the operands' addresses and shapes, which a trainer keeps
// from step to step, so the last few sets are remembered (encoding ten maps costs tens of
// microseconds of host time per call, a visible share of a small head's step).
struct MapsKey {
  const void *ws, *W, *dW;
  int d, V, cap_pad, chunk_rows, ldz, dev;
  bool operator==(const MapsKey& o) const {
    return ws == o.ws && W == o.W && dW == o.dW && d == o.d && V == o.V &&
           cap_pad == o.cap_pad && chunk_rows == o.chunk_rows && ldz == o.ldz && dev == o.dev;
  }
};
constexpr int kMapsCached = 8;
std::mutex g_maps_mutex;
MapsKey g_maps_key[kMapsCached];
Maps g_maps_val[kMapsCached];
bool g_maps_used[kMapsCached] = {false};
int g_maps_next = 0;

int make_maps(const LossArgs& a, const Layout& L, const Ws& w, Maps* m) {
  MapsKey key{a.workspace, a.W, a.dW, a.p.d, a.p.V, L.cap_pad, L.chunk_rows, L.ldz, 0};
  int s = current_device(&key.dev);
  if (s != NAT_OK) return s;
  {
    std::lock_guard<std::mutex> lock(g_maps_mutex);
    for (int i = 0; i < kMapsCached; ++i)
      if (g_maps_used[i] && g_maps_key[i] == key) {
        *m = g_maps_val[i];
        return NAT_OK;
      }
  }
  if ((s = encode_maps(a, L, w, m)) != NAT_OK) return s;
  std::lock_guard<std::mutex> lock(g_maps_mutex);
  g_maps_key[g_maps_next] = key;
  g_maps_val[g_maps_next] = *m;
  g_maps_used[g_maps_next] = true;
  g_maps_next = (g_maps_next + 1) % kMapsCached;
  return NAT_OK;
}

int finalize_grid(int rows) {
  const int g = (rows + 255) / 256;
  return g < 1 ? 1 : (g > 1184 ? 1184 : g);
}

int launch_dh(const LossArgs& a, const Layout& L, const Ws& w, const Maps& m, TcParams p,
              const int32_t* flag, int run_if) {
  int s;
  const int mb = L.chunk_rows / BM;
  const int nb_d = (a.p.d + BN - 1) / BN;
  p.flag = flag;
  p.run_if = run_if;
  const bool parts = L.dh_splits > 1 && pair_slots() > 0;
  p.k_splits = parts ? L.dh_splits : 1;
  if ((s = launch_tc<kDh>(m.dzK, m.wMn, m.wMn, parts ? m.dhAcc : m.hcK, p, mb, nb_d * p.k_splits,
                          a.stream)) != NAT_OK)
    return s;
  if (parts) {
    dh_finalize_kernel<<<L.chunk_rows < 4096 ? L.chunk_rows : 4096, 128, 0, a.stream>>>(
        w.dhacc, p.row_scale, w.g, reinterpret_cast<const __nv_bfloat16*>(a.W), a.targets,
        a.sel_idx, a.n_sel, (int)a.cap, p.row0, L.chunk_rows, a.p.d, a.p.V, p.k_splits,
        reinterpret_cast<__nv_bfloat16*>(a.dHidden), flag, run_if);
    NAT_LAUNCH_CHECK("dh_finalize_kernel");
  }
  return NAT_OK;
}

// The three two-pass backward launches for rows [row0, row0 + chunk_rows); `flag`
// (may be null) predicates them on the chunk having left the single-pass window.
int launch_two_pass_chunk(const LossArgs& a, const Layout& L, const Ws& w, const Maps& m,
                          int row0, const int32_t* flag) {
  int s;
  TcParams p = base_params(a, L, w);
  p.row0 = row0;
  p.chunk_rows = L.chunk_rows;
  p.b_row0 = row0;
  p.flag = flag;
  p.run_if = 1;
  const int mb = L.chunk_rows / BM;
  const int nb_d = (a.p.d + BN - 1) / BN;
  if ((s = launch_tc<kDz>(m.hcK, m.wK, m.wK2, m.hcK, p, mb, L.n_splits, a.stream)) != NAT_OK) return s;
  if ((s = launch_dh(a, L, w, m, p, flag, 1)) != NAT_OK) return s;
  return launch_tc<kDw>(m.dzMn, m.hcMn, m.hcMn, m.dwRed, p, (a.p.V + BM - 1) / BM, nb_d, a.stream);
}

int launch_onehot(const LossArgs& a, const Ws& w) {
  const int V = a.p.V, d = a.p.d, cap = (int)a.cap;
  const int tok_grid = (int)((a.cap + 255) / 256 < 1184 ? (a.cap + 255) / 256 : 1184);
  NAT_CUDA(cudaMemsetAsync(w.oh_count, 0, sizeof(int32_t) * (size_t)V, a.stream));
  onehot_count_kernel<<<tok_grid, 256, 0, a.stream>>>(a.targets, a.sel_idx, w.g, a.n_sel, cap, V,
                                                     w.oh_count);
  NAT_LAUNCH_CHECK("onehot_count_kernel");
  onehot_scan_kernel<<<1, 1024, 0, a.stream>>>(w.oh_count, V, w.oh_off);
  NAT_LAUNCH_CHECK("onehot_scan_kernel");
  onehot_fill_kernel<<<tok_grid, 256, 0, a.stream>>>(a.targets, a.sel_idx, w.g, a.n_sel, cap, V,
                                                    w.oh_off, w.oh_count, w.oh_list);
  NAT_LAUNCH_CHECK("onehot_fill_kernel");
  onehot_rank_kernel<<<tok_grid, 256, 0, a.stream>>>(a.targets, a.sel_idx, V, w.oh_off, w.oh_list,
                                                    w.oh_sorted);
  NAT_LAUNCH_CHECK("onehot_rank_kernel");
  const dim3 grid((unsigned)(V < 8192 ? V : 8192), (unsigned)((d + 1023) / 1024), 1);
  onehot_apply_kernel<<<grid, 256, 0, a.stream>>>(w.hc, w.g, V, d, w.oh_off, w.oh_sorted, a.dW);
  NAT_LAUNCH_CHECK("onehot_apply_kernel");
  return NAT_OK;
}

}  // namespace

size_t loss_bf16_workspace_bytes(const nat_loss_params& p, int64_t cap) {
  return make_layout(p, cap).total;
}

int loss_bf16_fwd(const LossArgs& a) {
  int s = require_sm100();
  if (s != NAT_OK) return s;
  const Layout L = make_layout(a.p, a.cap);
  const Ws w = carve(a.workspace, L);
  Maps m;  // encoded before anything is enqueued: a refusal leaves the stream untouched
  if (a.cap > 0 && (s = make_maps(a, L, w, &m)) != NAT_OK) return s;
  NAT_CUDA(cudaMemsetAsync(w.head, 0, sizeof(WorkspaceHead), a.stream));
  const TokenCtx c = make_token_ctx(a, &w.head->status);
  if (a.cap > 0) {
    if ((s = gather(a, L, w)) != NAT_OK) return s;
    const TcParams p = base_params(a, L, w);
    if ((s = launch_tc<kFwd>(m.hcK, m.wK, m.wK2, m.hcK, p, L.cap_pad / BM, L.n_splits, a.stream)) !=
        NAT_OK)
      return s;
    fwd_finalize_kernel<<<finalize_grid((int)a.cap), 256, 0, a.stream>>>(
        c, a.n_sel, (int)a.cap, 0, L.cap_pad, L.n_splits, L.cap_pad, w.pm, w.ps, w.zt, a.logp,
        a.lse, w.term, nullptr, nullptr, nullptr, 0);
    NAT_LAUNCH_CHECK("fwd_finalize_kernel");
  }
  return launch_loss_reduce(w.term, a.n_sel, a.cap, a.loss, w.head, a.stream);
}

int loss_bf16_bwd(const LossArgs& a) {
  int s = require_sm100();
  if (s != NAT_OK) return s;
  const Layout L = make_layout(a.p, a.cap);
  const Ws w = carve(a.workspace, L);
  Maps m;
  if (a.cap > 0 && (s = make_maps(a, L, w, &m)) != NAT_OK) return s;
  NAT_CUDA(cudaMemsetAsync(w.head, 0, sizeof(WorkspaceHead), a.stream));
  if (!a.p.accumulate_dW)
    NAT_CUDA(cudaMemsetAsync(a.dW, 0, sizeof(float) * (size_t)a.p.V * a.p.d, a.stream));
  if (a.cap == 0) return NAT_OK;
  const TokenCtx c = make_token_ctx(a, &w.head->status);
  if ((s = gather(a, L, w)) != NAT_OK) return s;
  if ((s = launch_grad_coeff(c, a.logp, a.n_sel, a.cap, a.dloss, w.g, a.stream)) != NAT_OK) return s;
  for (int row0 = 0; row0 < L.cap_pad; row0 += L.chunk_rows)
    if ((s = launch_two_pass_chunk(a, L, w, m, row0, nullptr)) != NAT_OK) return s;
  return launch_onehot(a, w);
}

// Forward and backward in one call with a single pass over S per row chunk.
int loss_bf16_fwd_bwd(const LossArgs& a) {
  int s = require_sm100();
  if (s != NAT_OK) return s;
  const Layout L = make_layout(a.p, a.cap);
  const Ws w = carve(a.workspace, L);
  Maps m;
  if (a.cap > 0 && (s = make_maps(a, L, w, &m)) != NAT_OK) return s;
  NAT_CUDA(cudaMemsetAsync(w.head, 0, sizeof(WorkspaceHead), a.stream));
  NAT_CUDA(cudaMemsetAsync(w.ovf, 0, sizeof(int32_t) * L.n_chunks, a.stream));
  if (!a.p.accumulate_dW)
    NAT_CUDA(cudaMemsetAsync(a.dW, 0, sizeof(float) * (size_t)a.p.V * a.p.d, a.stream));
  const TokenCtx c = make_token_ctx(a, &w.head->status);
  if (a.cap > 0) {
    if ((s = gather(a, L, w)) != NAT_OK) return s;
    const int mb = L.chunk_rows / BM;
    const int nb_d = (a.p.d + BN - 1) / BN;
    // Row references: the row maximum over the first vocabulary tile (a kFwd launch that
    // sees a vocabulary of one tile and writes its running maximum to mref).
    {
      TcParams p = base_params(a, L, w);
      p.V = a.p.V < BN ? a.p.V : BN;
      p.n_splits = 1;
      p.part_m = w.mref;
      if ((s = launch_tc<kFwd>(m.hcK, m.wK, m.wK2, m.hcK, p, L.cap_pad / BM, 1, a.stream)) != NAT_OK)
        return s;
    }
    for (int ci = 0; ci < L.n_chunks; ++ci) {
      const int row0 = ci * L.chunk_rows;
      int32_t* ovf = w.ovf + ci;
      TcParams p = base_params(a, L, w);
      p.row0 = row0;
      p.chunk_rows = L.chunk_rows;
      p.ovf = ovf;
      {
        // one work unit per (row block, vocabulary tile); partial row sums per tile, local
        // to the chunk
        TcParams pe = p;
        pe.n_splits = L.n_tiles;
        pe.part_s = w.pe;
        pe.cap_pad = L.chunk_rows;
        pe.progress = nullptr;
        if ((s = launch_tc<kE>(m.hcK, m.wK, m.wK2, m.dzSt, pe, mb, L.n_tiles, a.stream)) != NAT_OK)
          return s;
      }
      fused_finalize_kernel<<<L.chunk_rows < 2048 ? L.chunk_rows : 2048, 128, 0, a.stream>>>(
          c, a.n_sel, (int)a.cap, row0, L.chunk_rows, L.n_tiles, w.mref, w.pe, w.zt, a.dloss,
          a.logp, a.lse, w.term, w.g, w.cs, w.hc, w.hs, a.p.d, ovf);
      NAT_LAUNCH_CHECK("fused_finalize_kernel");
      p.ovf = nullptr;
      p.row_scale = w.cs;
      p.b_row0 = 0;  // Hs is local to the chunk
      if ((s = launch_dh(a, L, w, m, p, ovf, 0)) != NAT_OK) return s;
      p.flag = ovf;
      p.run_if = 0;
      if ((s = launch_tc<kDw>(m.dzMn, m.hsMn, m.hsMn, m.dwRed, p, (a.p.V + BM - 1) / BM, nb_d,
                              a.stream)) != NAT_OK)
        return s;
      // Predicated redo of the chunk by the two-pass kernels (no-ops unless *ovf != 0).
      TcParams pf = base_params(a, L, w);
      pf.row0 = row0;
      pf.chunk_rows = L.chunk_rows;
      pf.flag = ovf;
      pf.run_if = 1;
      if ((s = launch_tc<kFwd>(m.hcK, m.wK, m.wK2, m.hcK, pf, mb, L.n_splits, a.stream)) != NAT_OK)
        return s;
      fwd_finalize_kernel<<<finalize_grid(L.chunk_rows), 256, 0, a.stream>>>(
          c, a.n_sel, (int)a.cap, row0, L.chunk_rows, L.n_splits, L.cap_pad, w.pm, w.ps, w.zt,
          a.logp, a.lse, w.term, w.g, a.dloss, ovf, 1);
      NAT_LAUNCH_CHECK("fwd_finalize_kernel");
      if ((s = launch_two_pass_chunk(a, L, w, m, row0, ovf)) != NAT_OK) return s;
    }
    note_fallback_kernel<<<1, 128, 0, a.stream>>>(w.ovf, L.n_chunks, &w.head->status);
    NAT_LAUNCH_CHECK("note_fallback_kernel");
    if ((s = launch_onehot(a, w)) != NAT_OK) return s;
  }
  return launch_loss_reduce(w.term, a.n_sel, a.cap, a.loss, w.head, a.stream);
}

int trace_begin() {
  std::lock_guard<std::mutex> lock(g_trace_mutex);
  for (TraceSpan& sp : g_trace_spans) {
    cudaEventDestroy(sp.t0);
    cudaEventDestroy(sp.t1);
  }
  g_trace_spans.clear();
  g_trace_on = true;
  return NAT_OK;
}

int trace_end(float* ms_by_kind, int32_t* launches_by_kind) {
  std::vector<TraceSpan> spans;
  {
    std::lock_guard<std::mutex> lock(g_trace_mutex);
    g_trace_on = false;
    spans.swap(g_trace_spans);
  }
  for (int k = 0; k < NAT_TRACE_KINDS; ++k) {
    if (ms_by_kind) ms_by_kind[k] = 0.f;
    if (launches_by_kind) launches_by_kind[k] = 0;
  }
  int status = NAT_OK;
  for (TraceSpan& sp : spans) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(sp.t1);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, sp.t0, sp.t1);
    if (e != cudaSuccess) status = check_cuda(e, "nat_trace_end");
    if (sp.kind >= 0 && sp.kind < NAT_TRACE_KINDS) {
      if (ms_by_kind) ms_by_kind[sp.kind] += ms;
      if (launches_by_kind) launches_by_kind[sp.kind] += 1;
    }
    cudaEventDestroy(sp.t0);
    cudaEventDestroy(sp.t1);
  }
  return status;
}

}  // namespace nat
