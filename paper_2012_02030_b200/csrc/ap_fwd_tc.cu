// Masked attention of Section 3.2 for bf16 / fp16 tensors on the tcgen05 tensor cores.
//
// Persistent kernel, one CTA per SM, TWO query tiles in flight per CTA.  A work item is one
// (b, h, query tile of 128 rows).  The CTA runs two independent STREAMS; each stream owns one item
// at a time, with its own Q tile, K/V stages and bitmaps in shared memory, its own score buffer S
// and output accumulator O in tensor memory, its own producer warp, MMA-issuing warp and group of
// four softmax warps.  Nothing but the tensor pipe, the special-function units and a work counter
// is shared, so one stream's MMAs run under the other stream's softmax, and an item's first loads
// and its epilogue run under the other stream's rounds.
//
// A stream follows the schedule stored with the tile list: the ROUNDS of the item's (h, qt) list
// row.  A round holds up to eight non-empty groups of 16 key columns (slots), taken in list order
// from one or several key tiles, together with the bitmap of exactly those columns; groups without
// a kept entry never appear, so leaving them out is exact.  Per round:
//   S  = Q K_round^T         tcgen05.mma, N = 16 * slots, fp32 accumulator in TMEM
//   P  = exp2(c*S - c*m)     one thread per query row reads its S row from TMEM in two halves of
//                            64 columns (each an online-softmax step of its own), replaces pruned entries by -inf (the round's bitmap
//                            decides, exactly), keeps the running reference m and sum l of an
//                            online softmax, rescales O when m moved, and writes P as bf16 over S
//   O += P V_round           tcgen05.mma, A = P from TMEM, B = V (MN-major), one K step of 16 keys
//                            per slot; the first half's steps are issued as soon as the first
//                            half of P is written, i.e. under the softmax of the second half
// and after the item's last round O / l is written by the epilogue warps (zeros for rows that
// never saw a kept entry) while the stream goes on with its next item.
//
// Work distribution.  Items are numbered per CTA: item t is half t & 1 of unit
// blockIdx.x + (t >> 1) * gridDim.x, a unit being the pair (query tile n_qt-1-j, query tile j) of
// one (b, h).  The two producers draw item numbers from a counter in shared memory, so the stream
// that finishes first takes the next item (a causal late tile has a long list and an early one a
// short list).  Consecutive units belong to the same (b, h), so the CTAs running at any time share
// a few heads' K and V in L2.
//
// Warp roles (512 threads): warps 0-3 softmax of stream 0, warps 4-7 softmax of stream 1 (thread =
// query row = TMEM lane), warps 8-11 epilogue (both streams), warps 12/13 producers, warps 14/15
// MMA issuers (warp 14 owns the TMEM allocation).  TMEM (512 columns): S of stream x at column
// 128 x, O of stream x at column 256 + 128 x (at d = 64 two accumulators of 64 columns alternate
// there, so the next item's first O += P V need not wait for the epilogue).  Every wait is
// bounded; a wait that expires raises the device status word and the CTA winds down.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 512;
constexpr int kSubBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled sub-tile
constexpr uint32_t kTmemCols = 512;
constexpr bool kStagger = true;        // the streams' softmax phases keep apart (see the softmax warps)
#ifndef AP_STAGGER_CYCLES
#define AP_STAGGER_CYCLES 1200
#endif
constexpr uint32_t kStaggerCycles = AP_STAGGER_CYCLES;
constexpr int kRing = 4;              // per stream: slots for the rounds' info words and bitmaps

// per-round word published by the producer
constexpr uint32_t kInfoSlots = 15u;       // bits 0..3: slots of the round
constexpr uint32_t kInfoFirst = 1u << 4;   // first round of its item
constexpr uint32_t kInfoLast = 1u << 5;    // last round of its item
constexpr uint32_t kInfoFull = 1u << 6;    // every entry of the round is kept: no bitmap was copied
constexpr uint32_t kInfoStop = 1u << 7;    // no more work for this stream

// Shared-memory layout of a K or V stage.  Rows are the round's keys, a row's d elements are cut
// into halves of 64 (128 bytes, the swizzle span).
//   kSplit = false: [half][row / 8][8 rows][128 B]   one TMA box per half (3-D tensor map)
//   kSplit = true:  [row / 8][half][8 rows][128 B]   d = 128 only: one box brings both halves (5-D map)
// Per stream: kQBufs Q tiles, kStages K stages, kStages V stages.  Within a stream the chain
// S(g) -> softmax(g) -> O += P V(g) -> S(g+1) is serial (P lives in S's columns), so one stage is
// enough to keep the copies ahead: K(g+1) is copied under softmax(g), V(g+1) under S(g+1) and
// softmax(g+1).  d = 64 has room for two.
template <int D, bool kSplit>
struct Cfg {
  static_assert(!kSplit || D == 128, "the split layout is for d = 128");
  static constexpr int kSub = D / 64;                 // halves per row
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kStages = D == 64 ? 2 : 1;     // K / V ring depth of a stream
  static constexpr int kQBufs = D == 64 ? 2 : 1;
  static constexpr int kOBufs = D == 64 ? 2 : 1;      // output accumulators of a stream in TMEM
  static constexpr int kQOffset = 0;
  static constexpr int kKOffset = kQBufs * kTileBytes;
  static constexpr int kVOffset = kKOffset + kStages * kTileBytes;
  static constexpr int kStreamBytes = kVOffset + kStages * kTileBytes;
  static constexpr int kBarOffset = 2 * kStreamBytes;
  static constexpr int kHalfStride = kSplit ? 1024 : kSubBytes;          // half 0 -> half 1 of the same rows
  static constexpr int kSbo = kSplit ? 2048 : 1024;                      // one group of 8 rows -> the next
  static constexpr int kSlotStride = 2 * kSbo;                           // 16 rows (one slot) -> the next
  static_assert(kRing >= kStages + 2, "info / bitmap ring too short for the K ring");
};

// Tensor maps of one launch: Q in whole-tile boxes; K and V in boxes of 16, 32, 64 and 128 rows.
struct FwdMaps {
  CUtensorMap q;
  CUtensorMap k[4];
  CUtensorMap v[4];
};

struct StreamShared {
  alignas(16) uint32_t bitmap[kRing][kTile][4];  // the round's bitmap, row r = words [r][0..3]
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[2], v_full[2];                 // K / V rows of the stage have landed
  uint64_t k_empty[2], v_empty[2];               // S = Q K^T / O += P V of the stage has completed
  uint64_t b_full[kRing];                        // info word and bitmap of the round are valid
  uint64_t s_full;                               // S of a round is complete
  uint64_t p_full[2];                            // P of a half round is written (one arrival per softmax warp)
  uint64_t pv_done;                              // O += P V of a half round has completed
  uint64_t o_done[2], o_free[2];                 // per accumulator: O complete / O read out by the epilogue
  uint64_t ml_ready[4];                          // per item: the softmax warps have handed over l
  float l[4][kTile];                             // [item % 4][row]: sum of the row's weights
  int32_t ml_bh[4], ml_qt[4];                    // the item handed over (b * H + h, query tile); qt = -1: no more items
  uint32_t info[kRing];
  int32_t item_bh[kRing], item_qt[kRing];        // the item a round belongs to
};

struct Shared {
  StreamShared st[2];
  uint32_t tmem_base;
  int abort_flag;
  int next_item;  // work counter of the CTA
  uint32_t sm_start[2];  // cycle count (low word) at which stream x's softmax warps last began a round
};

// Development aid: with -DAP_FWD_TRACE thread block 0 records cycle stamps of its roles
// ([stream][role][round][point]; roles: 0 producer, 1 MMA issuer, 2..5 softmax warps), read back
// through ap_debug_fwd_trace.  Compiled out otherwise.
#ifdef AP_FWD_TRACE
constexpr int kTraceRounds = 256, kTracePoints = 16;
__device__ long long g_fwd_trace[2][6][kTraceRounds][kTracePoints];
#define AP_TRACE(x, role, g, k)                                                              \
  do {                                                                                       \
    if (blockIdx.x == 0 && lane == 0 && (g) < (uint32_t)kTraceRounds) g_fwd_trace[x][role][g][k] = clock64(); \
  } while (0)
#else
#define AP_TRACE(x, role, g, k) \
  do {                          \
  } while (0)
#endif
// the same from inside a single elected thread
#ifdef AP_FWD_TRACE
#define AP_TRACE1(x, role, g, k)                                                                      \
  do {                                                                                                \
    if (blockIdx.x == 0 && (g) < (uint32_t)kTraceRounds) g_fwd_trace[x][role][g][k] = clock64();      \
  } while (0)
#else
#define AP_TRACE1(x, role, g, k) \
  do {                           \
  } while (0)
#endif

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t lds_volatile(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void sts_volatile(uint32_t addr, uint32_t v) {
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// What every bounded wait needs.
struct WaitCtx {
  volatile int *abort_flag;
  unsigned *err;
  uint32_t max_polls;
};

// Bounded wait that also gives up as soon as another thread of the CTA has.  Each poll lets the
// hardware suspend the thread for up to a microsecond, so a waiting thread costs few issue slots.
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, const WaitCtx &w) {
  for (uint32_t i = 0; i < w.max_polls; ++i) {
    if (mbar_try_wait_for(bar, parity, 1000u)) return true;
    if (*w.abort_flag) return false;
  }
  *w.abort_flag = 1;
  atomicOr(w.err, kDevErrTimeout);
  return false;
}

// The same wait for a whole (converged) warp: one lane polls - 32 lanes polling one barrier would
// serialise - and the outcome is shared.
template <int kPollLane = 0>
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, int lane, const WaitCtx &w) {
  bool ok = true;
  if (lane == kPollLane && !mbar_try_wait(bar, parity)) ok = wait_or_abort(bar, parity, w);
  return __shfl_sync(0xffffffffu, ok ? 1 : 0, kPollLane) != 0;
}

// Two fp32 values rounded to the tensors' 16-bit type and packed (first value in the low half),
// and back: exactly the values the tensor cores will see.
template <bool kF16>
__device__ __forceinline__ uint32_t pack16x2(float lo, float hi) {
  if constexpr (kF16) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
  } else {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
  }
}
template <bool kF16>
__device__ __forceinline__ float2 unpack16x2(uint32_t pk) {
  if constexpr (kF16) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&pk));
  } else {
    return make_float2(__uint_as_float(pk << 16), __uint_as_float(pk & 0xffff0000u));
  }
}

// One online-softmax step of a thread's query row over kChunks 32-column chunks of S at `tmem_b`:
// pruned entries (bitmap bit 0) are replaced by -inf (exp2 of -inf is exactly 0), the row maximum
// is taken over kept entries, the exponent's reference follows it lazily, P = exp2(c*S - c*m) is
// written as 16-bit values over the first half of each chunk's columns of S (not yet waited for).
// Returns the new reference, the new sum and the factor by which the old sum (and the output
// accumulated so far) had to be scaled.
struct HalfStep {
  float m, l, alpha;
};
template <int kChunks, bool kMasked, bool kF16>
__device__ __forceinline__ HalfStep softmax_half(uint32_t tmem_b, uint2 bw, float m, float l, float scale_log2,
                                                 float ref_slack) {
  uint32_t xs[32 * kChunks];
#pragma unroll
  for (int c = 0; c < kChunks; ++c) tmem_ld32(tmem_b + 32 * c, &xs[32 * c]);
  tmem_wait_ld();
  if (kMasked) {
#pragma unroll
    for (int c = 0; c < kChunks; ++c) {
      const uint32_t w = c == 0 ? bw.x : bw.y;
#pragma unroll
      for (int e = 0; e < 32; ++e) xs[32 * c + e] = ((w >> e) & 1u) ? xs[32 * c + e] : 0xff800000u;  // -inf
    }
  }
  float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F, mx2 = -CUDART_INF_F, mx3 = -CUDART_INF_F;
#pragma unroll
  for (int e = 0; e < 32 * kChunks; e += 8) {
    mx0 = fmax3(mx0, __uint_as_float(xs[e]), __uint_as_float(xs[e + 1]));
    mx1 = fmax3(mx1, __uint_as_float(xs[e + 2]), __uint_as_float(xs[e + 3]));
    mx2 = fmax3(mx2, __uint_as_float(xs[e + 4]), __uint_as_float(xs[e + 5]));
    mx3 = fmax3(mx3, __uint_as_float(xs[e + 6]), __uint_as_float(xs[e + 7]));
  }
  const float half_max = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
  // The reference moves only when the maximum outgrows it by more than 2^8 in the exp2 domain
  // (weights stay <= 256, well inside bf16 and fp32 range), which saves most rescales of O.
  // O / l does not depend on the reference.
  const bool move = half_max > m + ref_slack;   // also true for the first kept entry (m = -inf)
  const float m_new = move ? half_max : m;
  const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
  const float alpha = move ? ex2_approx((m - m_safe) * scale_log2) : 1.f;  // 0 when m was -inf
  const float neg_mc = -m_safe * scale_log2;
  float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
  for (int c = 0; c < kChunks; ++c) {
    uint32_t pk[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const float p0 = ex2_approx(fmaf(__uint_as_float(xs[32 * c + 2 * e]), scale_log2, neg_mc));
      const float p1 = ex2_approx(fmaf(__uint_as_float(xs[32 * c + 2 * e + 1]), scale_log2, neg_mc));
      pk[e] = pack16x2<kF16>(p0, p1);
      // the row sum is taken over the rounded weights the MMA will use, so that
      // O / l is an exact convex combination of V rows whatever the rounding of P
      const float2 pr = unpack16x2<kF16>(pk[e]);
      sum0 += pr.x;
      sum1 += pr.y;
    }
    tmem_st16(tmem_b + 32 * c, pk);
  }
  return HalfStep{m_new, l * alpha + (sum0 + sum1), alpha};
}

// dbg_skip != 0 (test hook, see ap_debug_expire_waits): the producer of stream 0 leaves out the
// copies and the arrival of its first round, so that the waits on it run out.
template <int D, bool kSplit, bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
fwd_tc_kernel(const __grid_constant__ FwdMaps maps, uint16_t *__restrict__ O,
              const int32_t *__restrict__ round_ptr, const int32_t *__restrict__ round_rows,
              const uint8_t *__restrict__ round_info, const uint32_t *__restrict__ round_bitmap, int B, int H,
              int Lq, int n_qt, float scale_log2, unsigned *err, uint32_t max_polls, int dbg_skip) {
  using C = Cfg<D, kSplit>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Shared *sh = reinterpret_cast<Shared *>(smem + C::kBarOffset);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int x = 0; x < 2; ++x) {
      StreamShared &ss = sh->st[x];
      for (int i = 0; i < 2; ++i) {
        mbar_init(&ss.q_full[i], 1);
        mbar_init(&ss.q_empty[i], 1);
        mbar_init(&ss.k_full[i], 1);
        mbar_init(&ss.v_full[i], 1);
        mbar_init(&ss.k_empty[i], 1);
        mbar_init(&ss.v_empty[i], 1);
        mbar_init(&ss.p_full[i], 4);  // softmax warps of the stream
        mbar_init(&ss.o_done[i], 1);
        mbar_init(&ss.o_free[i], 4);  // epilogue warps
      }
      for (int i = 0; i < kRing; ++i) mbar_init(&ss.b_full[i], 1);
      mbar_init(&ss.s_full, 1);
      mbar_init(&ss.pv_done, 1);
      for (int i = 0; i < 4; ++i) mbar_init(&ss.ml_ready[i], 4);
    }
    sh->abort_flag = 0;
    sh->next_item = 0;
    sh->sm_start[0] = sh->sm_start[1] = (uint32_t)clock64() - 0x40000000u;
    fence_mbar_init();
  }
  if (warp == 14) {
    tmem_alloc(&sh->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  // Output accumulator of the n-th item of stream x.
  auto o_addr = [&](int x, uint32_t n) {
    return tmem + 256u + 128u * (uint32_t)x + (C::kOBufs == 2 ? 64u * (n & 1u) : 0u);
  };
  const WaitCtx wc{&sh->abort_flag, err, max_polls};
  // producers: the copies armed last (round numbers; -1: none), for the wind-down after an expired wait
  int armed_q = -1, armed_k = -1, armed_v = -1;

  if (warp == 12 || warp == 13) {
    // ------------------------------------------------------------ producer of stream x
    const int x = warp - 12;
    StreamShared &ss = sh->st[x];
    unsigned char *q_s = smem + x * C::kStreamBytes + C::kQOffset;
    unsigned char *k_s = smem + x * C::kStreamBytes + C::kKOffset;
    unsigned char *v_s = smem + x * C::kStreamBytes + C::kVOffset;
    if (lane < 4) {
      prefetch_tensormap(&maps.k[lane]);
      prefetch_tensormap(&maps.v[lane]);
    }
    if (lane == 4) prefetch_tensormap(&maps.q);
    bool ok = true;
    uint32_t g = 0, n = 0;   // rounds / non-empty items of this stream so far
    const int n_half = (n_qt + 1) / 2, n_units = B * H * n_half;
    const int item_step = (int)gridDim.x;
    struct ItemRef {
      int bh, qt, rho0, rho1;  // rounds [rho0, rho1): loaded here, first read when the item begins
      bool in_range, exists;   // !exists: no such item (the unit's halves coincide)
    };
    // The unit's (j, bh, h = bh % H) are stepped from the unit last looked at to the one wanted
    // instead of divided out of the unit number (item numbers only grow).
    int cur_k = 0, cur_u = (int)blockIdx.x, cur_j = cur_u % n_half, cur_bh = cur_u / n_half, cur_h = cur_bh % H;
    const int step_j = item_step % n_half, step_bh = item_step / n_half, step_h = step_bh % H;
    // Draws the next item number of the CTA and looks its rounds up.
    auto next_item = [&]() {
      int t = 0;
      if (lane == 0) t = atomicAdd(&sh->next_item, 1);
      t = __shfl_sync(0xffffffffu, t, 0);
      const int k = t >> 1;
      while (cur_k < k && cur_u < n_units) {
        ++cur_k;
        cur_u += item_step;
        cur_j += step_j;
        cur_bh += step_bh;
        cur_h += step_h;
        if (cur_j >= n_half) {
          cur_j -= n_half;
          ++cur_bh;
          ++cur_h;
        }
        if (cur_h >= H) cur_h -= H;
      }
      ItemRef it;
      it.in_range = cur_k == k && cur_u < n_units;
      it.bh = 0, it.qt = 0, it.rho0 = 0, it.rho1 = 0, it.exists = false;
      if (it.in_range) {
        const int j = cur_j;
        it.bh = cur_bh;
        it.qt = (t & 1) ? j : n_qt - 1 - j;
        if (!(t & 1) || j != n_qt - 1 - j) {
          const int lr = cur_h * n_qt + it.qt;
          it.rho0 = (int)ldg_now_u32(round_ptr + lr);
          it.rho1 = (int)ldg_now_u32(round_ptr + lr + 1);
          it.exists = true;
        }
      }
      return it;
    };
    // One piece of a stage: (16 << lg) consecutive key rows from `row` on, to slot `q` of the stage.
    auto load_piece = [&](unsigned char *stage, const CUtensorMap *m, uint64_t *bar, int q, int row, int bh) {
      if (kSplit) {
        tma_load_5d(stage + q * C::kSlotStride, m, bar, 0, 0, 0, row >> 3, bh);
      } else {
#pragma unroll
        for (int s = 0; s < C::kSub; ++s)
          tma_load_3d(stage + s * kSubBytes + q * C::kSlotStride, m, bar, 64 * s, row, bh);
      }
    };
    auto wait_free = [&](uint64_t *bar, uint32_t ph) {
      if (lane == 0) ok = wait_or_abort(bar, ph ^ 1u, wc);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    };
    // A run of slots (key rows following one another) is copied by the lane of its first slot, in
    // pieces of 8, 4, 2 or 1 slots.
    auto load_run = [&](unsigned char *stage, const CUtensorMap *m4, uint64_t *bar, int row, int run, int bh) {
      int q = lane, r = row, left = run;
      while (left > 0) {
        const int lg = left >= 8 ? 3 : left >= 4 ? 2 : left >= 2 ? 1 : 0;
        load_piece(stage, m4 + lg, bar, q, r, bh);
        q += 1 << lg;
        r += 16 << lg;
        left -= 1 << lg;
      }
    };
    // Items are drawn one ahead: the look-ups of the next item are in flight while this one runs,
    // and the slot rows and info byte of its first round are fetched during this item's last round.
    ItemRef next = next_item();
    int pf_valid = 0, pf_row = -1;
    uint32_t pf_info = 0u;
    while (next.in_range && ok) {
      const ItemRef cur = next;
      next = next_item();
      if (!cur.exists) continue;
      const int bh = cur.bh, qt = cur.qt, rho0 = cur.rho0, n_rounds = cur.rho1 - cur.rho0;
      if (n_rounds == 0) {
        // nothing kept in this query tile: its output rows are zero (nobody else sees the item)
        const int rows = min(kTile, Lq - qt * kTile);
        uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + (size_t)qt * kTile) * D);
        for (int i = lane; i < rows * (D / 8); i += 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        continue;
      }
      // Q of this item into its buffer (free once the last S = Q K^T of item n - kQBufs has completed)
      const int qb = (int)(n % C::kQBufs);
      const uint32_t q_use = n / C::kQBufs;
      if (lane == 0) {
        ok = wait_or_abort(&ss.q_empty[qb], (q_use & 1u) ^ 1u, wc);
        if (ok) {
          mbar_arrive_expect_tx(&ss.q_full[qb], C::kTileBytes);
#pragma unroll
          for (int s = 0; s < C::kSub; ++s)
            tma_load_3d(q_s + qb * C::kTileBytes + s * kSubBytes, &maps.q, &ss.q_full[qb], 64 * s, qt * kTile, bh);
          armed_q = (int)n;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      // slot rows (lanes 0..7) and info byte of a round are fetched one round ahead
      int next_row = pf_row;
      uint32_t next_info = pf_info;
      if (!pf_valid) {
        next_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)rho0 * 8 + lane) : -1;
        next_info = ldg_now_u8(round_info + rho0);
      }
      pf_valid = 0;
      for (int v = 0; v < n_rounds && ok; ++v, ++g) {
        const int row = next_row;
        const uint32_t rinfo = next_info;
        if (v + 1 < n_rounds) {
          next_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)(rho0 + v + 1) * 8 + lane) : -1;
          next_info = ldg_now_u8(round_info + rho0 + v + 1);
        } else if (next.in_range && next.exists && next.rho1 > next.rho0) {
          pf_valid = 1;
          pf_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)next.rho0 * 8 + lane) : -1;
          pf_info = ldg_now_u8(round_info + next.rho0);
        }
        const int st = (int)(g % C::kStages);
        const uint32_t ph = (g / C::kStages) & 1u;
        const int ng = (int)(rinfo & 15u);
        const bool full = (rinfo & 0x80u) != 0u;
        // slots whose key rows follow one another form a run
        const int row_before = __shfl_up_sync(0xffffffffu, row, 1);
        const bool head = lane < ng && (lane == 0 || row != row_before + 16);
        const uint32_t heads = __ballot_sync(0xffffffffu, head);
        const uint32_t later = lane < 31 ? heads >> (lane + 1) : 0u;
        const int run = head ? (later ? __ffs((int)later) : ng - lane) : 0;  // slots in this lane's run
        const int si = (int)(g % kRing);
        // K of round g: its stage is free once S of round g - kStages has completed.  The info slot
        // last served round g - kRing, whose softmax was over before S of round g - kStages was issued.
        wait_free(&ss.k_empty[st], ph);
        if (!ok) break;
        AP_TRACE(x, 0, g, 0);
        const uint32_t bytes = (uint32_t)ng * 16u * D * 2u;
        const bool skip = dbg_skip != 0 && x == 0 && g == 0;
        if (lane == 0) {
          ss.info[si] = (uint32_t)ng | (v == 0 ? kInfoFirst : 0u) | (v + 1 == n_rounds ? kInfoLast : 0u) |
                        (full ? kInfoFull : 0u);
          ss.item_bh[si] = bh;
          ss.item_qt[si] = qt;
          if (!skip) {
            mbar_arrive_expect_tx(&ss.k_full[st], bytes);
            armed_k = (int)g;
            if (full) {
              mbar_arrive(&ss.b_full[si]);
            } else {
              mbar_arrive_expect_tx(&ss.b_full[si], kBitmapWords * 4);
              bulk_load(&ss.bitmap[si][0][0], round_bitmap + (size_t)(rho0 + v) * kBitmapWords, kBitmapWords * 4,
                        &ss.b_full[si]);
            }
          }
        }
        __syncwarp();
        if (!skip) load_run(k_s + st * C::kTileBytes, maps.k, &ss.k_full[st], row, run, bh);
        AP_TRACE(x, 0, g, 1);
        // V of round g: its stage is free once O += P V of round g - kStages has completed, which is
        // before S of round g + 1 - kStages, the next thing this warp waits for
        wait_free(&ss.v_empty[st], ph);
        if (!ok) break;
        AP_TRACE(x, 0, g, 2);
        if (!skip) {
          if (lane == 0) {
            mbar_arrive_expect_tx(&ss.v_full[st], bytes);
            armed_v = (int)g;
          }
          __syncwarp();
          load_run(v_s + st * C::kTileBytes, maps.v, &ss.v_full[st], row, run, bh);
        }
        AP_TRACE(x, 0, g, 3);
      }
      ++n;
    }
    // no more work: one more round carries the stop word
    if (ok) {
      const int st = (int)(g % C::kStages);
      const uint32_t ph = (g / C::kStages) & 1u;
      wait_free(&ss.k_empty[st], ph);
      if (ok && lane == 0) {
        ss.info[g % kRing] = kInfoStop;
        mbar_arrive(&ss.k_full[st]);
        mbar_arrive(&ss.b_full[g % kRing]);
      }
    }
  } else if (warp >= 14) {
    // ------------------------------------------------------------ MMA issuer of stream x
    // One thread walks the stream's rounds.  Per round it issues O += P V in two halves as the
    // softmax hands P over, and right behind the second half the next round's S = Q K^T, whose
    // operands it has checked for while the softmax was busy.  The tensor pipe runs one thread's
    // instructions in order, so that S may overwrite the columns P was read from without a wait in
    // between.  Every instruction between a hand-over and the MMAs it releases is on the stream's
    // critical path, so this thread's code is kept short: descriptors are prepared once, nothing is
    // shared with other lanes.
    const int x = warp - 14;
    if (lane == 0) {
      StreamShared &ss = sh->st[x];
      const uint32_t q_addr = smem_u32(smem + x * C::kStreamBytes + C::kQOffset);
      const uint32_t k_addr = smem_u32(smem + x * C::kStreamBytes + C::kKOffset);
      const uint32_t v_addr = smem_u32(smem + x * C::kStreamBytes + C::kVOffset);
      const uint32_t tmem_s = tmem + 128u * (uint32_t)x;
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true, kF16);
      bool ok = true;
      uint32_t n = 0;  // non-empty items finished so far
      auto wait = [&](uint64_t *bar, uint32_t parity) {
        if (!mbar_try_wait(bar, parity)) ok = wait_or_abort(bar, parity, wc);
        return ok;
      };
      // waits for K of round g (and Q if the round opens an item) and returns the round's info word
      auto operands_of = [&](uint32_t g) {
        if (!wait(&ss.k_full[g % C::kStages], (g / C::kStages) & 1u)) return kInfoStop;
        const uint32_t info = ss.info[g % kRing];
        if (!(info & kInfoStop) && (info & kInfoFirst)) {
          // the item this round opens: item n, or n + 1 while item n's last round is still under way
          const uint32_t item = n + (g > 0 && (ss.info[(g - 1) % kRing] & kInfoLast) ? 1u : 0u);
          if (!wait(&ss.q_full[item % C::kQBufs], (item / C::kQBufs) & 1u)) return kInfoStop;
        }
        return info;
      };
      // Low descriptor words of every operand tile this thread will ever name (the stages are few).
      uint32_t q_lo[C::kQBufs][D / 16], k_lo[C::kStages][D / 16], v_lo[C::kStages][8];
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int sub = ks / 4, off = (ks % 4) * 32;  // D/16 steps of K = 16 (32 bytes inside the swizzled rows)
#pragma unroll
        for (int b = 0; b < C::kQBufs; ++b)
          q_lo[b][ks] = smem_desc_lo(q_addr + b * C::kTileBytes + sub * kSubBytes + off, 16);
#pragma unroll
        for (int b = 0; b < C::kStages; ++b)
          k_lo[b][ks] = smem_desc_lo(k_addr + b * C::kTileBytes + sub * C::kHalfStride + off, 16);
      }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
#pragma unroll
        for (int b = 0; b < C::kStages; ++b)
          v_lo[b][ks] = smem_desc_lo(v_addr + b * C::kTileBytes + ks * C::kSlotStride, C::kHalfStride);
      constexpr uint32_t q_hi = smem_desc_hi_sw128(1024), kv_hi = smem_desc_hi_sw128(C::kSbo);
      // S = Q K^T of round g of item `item` (N = 16 ng), announced on s_full first: the softmax waits for it
      auto issue_s = [&](uint32_t g, uint32_t info, uint32_t item) {
        const int st = (int)(g % C::kStages), qb = (int)(item % C::kQBufs);
        const uint32_t idesc_qk = idesc_bf16_f32(128, 16 * (int)(info & kInfoSlots), false, false, kF16);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t ql = C::kQBufs == 2 && qb ? q_lo[C::kQBufs - 1][ks] : q_lo[0][ks];
          const uint32_t kl = C::kStages == 2 && st ? k_lo[C::kStages - 1][ks] : k_lo[0][ks];
          mma_ss(tmem_s, smem_desc_join(ql, q_hi), smem_desc_join(kl, kv_hi), idesc_qk, ks > 0);
        }
        mma_commit(&ss.s_full);
        mma_commit(&ss.k_empty[st]);
        if (info & kInfoLast) mma_commit(&ss.q_empty[qb]);
      };
      uint32_t info = operands_of(0);
      if (ok && !(info & kInfoStop)) {
        tc_fence_after_sync();
        issue_s(0, info, 0);
        AP_TRACE1(x, 1, 0u, 0);
      }
      for (uint32_t g = 0; ok && !(info & kInfoStop); ++g) {
        const int st = (int)(g % C::kStages);
        const uint32_t ph = (g / C::kStages) & 1u;
        const int ng = (int)(info & kInfoSlots);
        const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
        // O += P V.  What is ready early first; P, which the softmax has just finished, last.
        if (!wait(&ss.v_full[st], ph)) break;
        // the first round of an item overwrites O: the epilogue of the item that used the accumulator
        // before must have read it
        const uint32_t ob = C::kOBufs == 2 ? (n & 1u) : 0u;
        if (first && n >= (uint32_t)C::kOBufs && !wait(&ss.o_free[ob], ((n / C::kOBufs) - 1u) & 1u)) break;
        const uint32_t o_acc = o_addr(x, n);
        AP_TRACE1(x, 1, g, 2);
        // One K step of 16 keys per slot.  P (16-bit) of a 32-column chunk is written over the
        // first 16 columns of that chunk of S, so slot q's eight columns of P start at column
        // 32 (q / 2) + 8 (q % 2).  The item's first step overwrites the accumulator.
        auto issue_pv = [&](int half) {
#pragma unroll
          for (int ks = 4 * half; ks < 4 * half + 4; ++ks) {
            const uint32_t vl = C::kStages == 2 && st ? v_lo[C::kStages - 1][ks] : v_lo[0][ks];
            if (ks < ng)
              mma_ts(o_acc, tmem_s + 32 * (ks >> 1) + 8 * (ks & 1), smem_desc_join(vl, kv_hi), idesc_pv,
                     (first && ks == 0) ? 0u : 1u);
          }
        };
        if (!wait(&ss.p_full[0], g & 1u)) break;
        AP_TRACE1(x, 1, g, 3);
        tc_fence_after_sync();
        issue_pv(0);
        mma_commit(&ss.pv_done);
        // while the softmax works on the second half: the next round's operands (they do not
        // depend on this round's P)
        const uint32_t info_next = operands_of(g + 1);
        if (!ok) break;
        AP_TRACE1(x, 1, g, 6);
        if (last) ++n;
        if (!wait(&ss.p_full[1], g & 1u)) break;
        AP_TRACE1(x, 1, g, 4);
        tc_fence_after_sync();
        issue_pv(1);
        if (!(info_next & kInfoStop)) issue_s(g + 1, info_next, n);
        AP_TRACE1(x, 1, g + 1, 0);
        // (completion of these is signalled once the MMAs issued so far, S included, are through:
        // nobody waits for them as urgently as the softmax for S)
        mma_commit(&ss.pv_done);
        mma_commit(&ss.v_empty[st]);
        if (last) mma_commit(&ss.o_done[ob]);
        AP_TRACE1(x, 1, g, 5);
        info = info_next;
      }
    }
    __syncwarp();
  } else if (warp < 8) {
    // ------------------------------------------------------------ softmax of stream x
    const int x = warp >> 2;
    StreamShared &ss = sh->st[x];
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tmem_s = tmem + 128u * (uint32_t)x + lane_addr;
    uint32_t tmem_og = o_addr(x, 0) + lane_addr;  // the current item's output accumulator
    const float ref_slack = 8.f / scale_log2;
    const uint32_t start_mine = smem_u32(&sh->sm_start[x]), start_other = smem_u32(&sh->sm_start[1 - x]);
    const bool flag_writer = (warp & 3) == 0 && lane == 0;
    bool ok = true;
    uint32_t n = 0;
    float m = -CUDART_INF_F, l = 0.f;       // exponent reference and running sum of weights of this row
    bool o_started = false;                  // an earlier half round of the item added to the accumulator
    int cur_bh = 0, cur_qt = 0;
    for (uint32_t g = 0; ok; ++g) {
      const int si = (int)(g % kRing);       // info / bitmap slot of the round
      ok = warp_wait(&ss.b_full[si], (g / kRing) & 1u, lane, wc);
      if (!ok) break;
      const uint32_t info = ss.info[si];
      if (info & kInfoStop) break;
      const int ng = (int)(info & kInfoSlots);
      const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
      const bool tile_full = (info & kInfoFull) != 0u;
      if (first) {
        cur_bh = ss.item_bh[si];
        cur_qt = ss.item_qt[si];
        m = -CUDART_INF_F;
        l = 0.f;
        o_started = false;
        tmem_og = o_addr(x, n) + lane_addr;
      }
      AP_TRACE(x, 2 + (warp & 3), g, 0);
      ok = warp_wait(&ss.s_full, g & 1u, lane, wc);
      if (!ok) break;
      AP_TRACE(x, 2 + (warp & 3), g, 1);
      // The two streams keep their softmax phases apart by at least half a round.  Left alone they
      // fall into lockstep (their MMAs share the tensor pipe and complete together), and then
      // both compute while the tensor pipe idles and both wait while it works.  Started a
      // half round apart, one stream's MMAs run under the other's exponentials, while two
      // warps per scheduler still overlap enough to hide each other's latencies.  A hint only: the
      // wait is short and bounded, and nothing depends on it.  (Stream 1 looks a moment later, so
      // that of two streams arriving together stream 0 goes first.)
      if (kStagger) {
        if (x == 1) __nanosleep(64);
        for (int i = 0; i < 48; ++i) {  // (one read serves the warp)
          if ((uint32_t)clock64() - lds_volatile(start_other) >= kStaggerCycles) break;
          __nanosleep(32);
        }
        if (flag_writer) sts_volatile(start_mine, (uint32_t)clock64());
      }
      AP_TRACE(x, 2 + (warp & 3), g, 2);
      tc_fence_after_sync();
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        // this half's slots 4 half .. 4 half + n_sl - 1: one or two 32-column chunks
        const int n_sl = min(max(ng - 4 * half, 0), 4);
        if (n_sl > 0) {
          const uint32_t tmem_b = tmem_s + 64u * (uint32_t)half;
          uint2 bw = make_uint2(0xffffffffu, 0xffffffffu);   // bitmap words of the two chunks
          if (!tile_full) bw = *reinterpret_cast<const uint2 *>(&ss.bitmap[si][r][2 * half]);
          // Straight-line code per case (one or two chunks, masked or not): the chunks' loads,
          // maxima, exponentials and stores interleave freely, which is worth far more than
          // skipping the occasional chunk in which a warp's 32 rows keep nothing.
          HalfStep st{m, l, 1.f};
          if (n_sl > 2) {
            if (tile_full) st = softmax_half<2, false, kF16>(tmem_b, bw, m, l, scale_log2, ref_slack);
            else st = softmax_half<2, true, kF16>(tmem_b, bw, m, l, scale_log2, ref_slack);
          } else {
            st = softmax_half<1, true, kF16>(tmem_b, bw, m, l, scale_log2, ref_slack);
          }
          // Rescale the running output where the reference moved (rare: the reference is lazy).
          // O += P V of the half round before may still be running: wait for it first.  (It cannot
          // be further ahead: the step after it needs the P being handed over below.)  P of this
          // half is already in TMEM but not handed over yet, so the order is free.
          if (o_started && __any_sync(0xffffffffu, st.alpha != 1.f)) {
            ok = warp_wait(&ss.pv_done, (2u * g + (uint32_t)half - 1u) & 1u, lane, wc);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(tmem_og + 32 * c, o);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * st.alpha);
              tmem_st32(tmem_og + 32 * c, o);
            }
          }
          m = st.m;
          l = st.l;
          o_started = true;
          tmem_wait_st();
        }
        // one arrival per warp (32 lanes arriving one by one would take hundreds of cycles)
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&ss.p_full[half]);
        AP_TRACE(x, 2 + (warp & 3), g, 3 + half);
      }
      if (!ok) break;
      if (!last) continue;
      // The item's rounds are over for these warps: they hand l to the epilogue warps and go on with
      // the stream's next item.  The slot of the hand-over ring was last used by item n - 4, whose
      // epilogue read it before it released that item's accumulator, which the first O += P V of
      // item n - 4 + kOBufs waited for; that step was issued before S of this item.
      ss.l[n & 3u][r] = l;
      if ((threadIdx.x & 127) == 0) {
        ss.ml_bh[n & 3u] = cur_bh;
        ss.ml_qt[n & 3u] = cur_qt;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&ss.ml_ready[n & 3u]);
      ++n;
    }
    // no more items: tell the epilogue warps (the slot is free by the argument above)
    if (ok) {
      if ((threadIdx.x & 127) == 0) ss.ml_qt[n & 3u] = -1;
      __syncwarp();
      if (lane == 0) mbar_arrive(&ss.ml_ready[n & 3u]);
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------ epilogue (both streams)
    // Per finished item: O / l, rounded once to the tensors' type.  Each warp serves its 32 rows of
    // whichever stream hands an item over next.
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    uint32_t n0 = 0u, n1 = 0u;             // items of stream 0 / 1 taken so far
    bool live0 = true, live1 = true;       // the stream has not sent its end marker yet
    bool ok = true;
    while (ok && (live0 || live1)) {
      // lane 0 polls the two streams' hand-over barriers in turn
      int x = -1;
      if (lane == 0) {
        for (uint32_t i = 0; i < wc.max_polls && x < 0; ++i) {
          if (live0 && mbar_try_wait(&sh->st[0].ml_ready[n0 & 3u], (n0 >> 2) & 1u)) x = 0;
          if (x < 0 && live1 && mbar_try_wait(&sh->st[1].ml_ready[n1 & 3u], (n1 >> 2) & 1u)) x = 1;
          if (x < 0) {
            if (*wc.abort_flag) break;
            if (i > 1024) __nanosleep(64);
          }
        }
        if (x < 0 && !*wc.abort_flag) {
          *wc.abort_flag = 1;
          atomicOr(err, kDevErrTimeout);
        }
      }
      x = __shfl_sync(0xffffffffu, x, 0);
      if (x < 0) {
        ok = false;
        break;
      }
      StreamShared &ss = sh->st[x];
      const uint32_t n = x == 0 ? n0 : n1;
      if (x == 0) ++n0; else ++n1;
      const int item_qt = ss.ml_qt[n & 3u], item_bh = ss.ml_bh[n & 3u];
      if (item_qt < 0) {
        if (x == 0) live0 = false; else live1 = false;
        continue;
      }
      const float l = ss.l[n & 3u][r];
      const int i = item_qt * kTile + r;
      uint16_t *orow = O + ((size_t)item_bh * Lq + i) * D;
      // a row without kept entries has l = 0 and P = 0 throughout: exact zeros (its accumulator may
      // never have been written)
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const uint32_t ob = C::kOBufs == 2 ? (n & 1u) : 0u;
      ok = warp_wait(&ss.o_done[ob], (n / C::kOBufs) & 1u, lane, wc);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t o_acc = o_addr(x, n) + lane_addr;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(o_acc + 32 * c, o);
        tmem_wait_ld();
        if (c == D / 32 - 1) {  // this thread's rows of O are in registers: the next item may overwrite them
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&ss.o_free[ob]);
        }
        if (i < Lq) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int j = 8 * q + 2 * e;
              const float x0 = inv > 0.f ? __uint_as_float(o[j]) * inv : 0.f;
              const float x1 = inv > 0.f ? __uint_as_float(o[j + 1]) * inv : 0.f;
              pk[e] = pack16x2<kF16>(x0, x1);
            }
            *reinterpret_cast<uint4 *>(orow + 32 * c + 8 * q) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if ((warp == 12 || warp == 13) && lane == 0 && *wc.abort_flag) {
    // A wait expired somewhere in the CTA and every role has left its loop.  Copies this producer
    // armed may still be in flight: wait (bounded) for the most recent ones before the CTA's shared
    // memory is given up (earlier ones completed before these were armed).
    StreamShared &ss = sh->st[warp - 12];
    if (armed_q >= 0) mbar_wait(&ss.q_full[armed_q % C::kQBufs], ((uint32_t)armed_q / C::kQBufs) & 1u, 1u << 16);
    for (int a = armed_k - 1; a <= armed_k; ++a)
      if (a >= 0) {
        mbar_wait(&ss.k_full[a % C::kStages], ((uint32_t)a / C::kStages) & 1u, 1u << 16);
        mbar_wait(&ss.b_full[a % kRing], ((uint32_t)a / kRing) & 1u, 1u << 16);
      }
    for (int a = armed_v - 1; a <= armed_v; ++a)
      if (a >= 0) mbar_wait(&ss.v_full[a % C::kStages], ((uint32_t)a / C::kStages) & 1u, 1u << 16);
  }
  __syncthreads();
  if (warp == 14) tmem_dealloc(tmem, kTmemCols);
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    cached[dev] = n;
  }
  return cached[dev];
}

template <int D, bool kSplit, bool kF16>
cudaError_t launch(const FwdMaps &maps, void *O, const ap_tiles &t, int B, int H, int Lq, float scale,
                   unsigned *err, cudaStream_t s) {
  using C = Cfg<D, kSplit>;
  constexpr int kSmemBytes = C::kBarOffset + (int)sizeof(Shared) + 1024;  // + alignment slack
  static_assert(kSmemBytes > 114 * 1024 && kSmemBytes <= 227 * 1024, "one CTA per SM, within the limit");
  auto kern = fwd_tc_kernel<D, kSplit, kF16>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int n_units = B * H * ((t.n_qt + 1) / 2);  // pairs of query tiles, see the producer
  const float scale_log2 = scale * 1.4426950408889634f;
  const DebugKnobs dbg = debug_knobs();
  // the test hook runs on one CTA only (a tiny grid is all it is meant for)
  kern<<<dbg.skip_arrive ? 1 : (n_units < sms ? n_units : sms), kThreads, kSmemBytes, s>>>(
      maps, static_cast<uint16_t *>(O), t.round_ptr, t.round_rows, t.round_info, t.round_bitmap, B, H, Lq,
      t.n_qt, scale_log2, err, dbg.max_polls, dbg.skip_arrive);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

#ifdef AP_FWD_TRACE
extern "C" int ap_debug_fwd_trace(long long *host_out, size_t bytes) {
  return (int)cudaMemcpyFromSymbol(host_out, g_fwd_trace, bytes < sizeof(g_fwd_trace) ? bytes : sizeof(g_fwd_trace));
}
#endif

cudaError_t launch_fwd_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                          int Lq, int Lk, int d, int f16, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  // d = 128 with whole groups of eight key rows: both halves of a row come with one box
  const bool split = d == 128 && Lk % 8 == 0;
  FwdMaps maps;
  bool ok = make_tile_map_bf16(&maps.q, Q, B * H, Lq, d);
  for (int i = 0; i < 4 && ok; ++i) {
    const int rows = 16 << i;
    ok = split ? make_split_map_bf16_d128(&maps.k[i], K, B * H, Lk, rows) &&
                     make_split_map_bf16_d128(&maps.v[i], V, B * H, Lk, rows)
               : make_tile_map_bf16(&maps.k[i], K, B * H, Lk, d, rows) &&
                     make_tile_map_bf16(&maps.v[i], V, B * H, Lk, d, rows);
  }
  if (!ok) return cudaErrorUnknown;
  if (f16) {
    if (d == 64) return launch<64, false, true>(maps, O, t, B, H, Lq, scale, err, s);
    return split ? launch<128, true, true>(maps, O, t, B, H, Lq, scale, err, s)
                 : launch<128, false, true>(maps, O, t, B, H, Lq, scale, err, s);
  }
  if (d == 64) return launch<64, false, false>(maps, O, t, B, H, Lq, scale, err, s);
  return split ? launch<128, true, false>(maps, O, t, B, H, Lq, scale, err, s)
               : launch<128, false, false>(maps, O, t, B, H, Lq, scale, err, s);
}

}  // namespace ap
