// Masked attention of Section 3.2 for bf16 / fp16 tensors on the tcgen05 tensor cores.
//
// Persistent kernel, one CTA per SM.  A work item is one (b, h, query tile of 128 rows); the CTA
// works through its items as ONE sequence of rounds that runs on across item boundaries.  The
// rounds are the schedule stored with the tile list: a round of an item's (h, qt) list row holds
// up to eight non-empty groups of 16 key columns (slots), taken in list order from one or several
// key tiles, together with the bitmap of exactly those columns; groups without a kept entry never
// appear, so leaving them out is exact.  Per round:
//   S  = Q K_round^T         tcgen05.mma, N = 16 * slots, fp32 accumulator in TMEM
//   P  = exp2(c*S - c*m)     two threads per query row, one per half of the round's columns: read
//                            64 scores from TMEM, replace pruned entries by -inf (the round's
//                            bitmap decides, exactly), agree on the row's exponent reference m,
//                            rescale O when m moved, write P as 16-bit values over S
//   O += P V_round           tcgen05.mma, A = P from TMEM, B = V (MN-major), one K step of 16 keys
//                            per slot
// and after an item's last round O / l is written by the epilogue warps (zeros for rows that never
// saw a kept entry) while the rounds of the next item are already under way.
//
// What overlaps.  TMEM (512 columns) holds two score buffers S[0], S[1] (rounds alternate) and two
// output accumulators O[0], O[1] (items alternate).  All eight softmax warps work on one round at
// a time; while they do, the tensor pipe runs O += P V of the round before and S of the round
// after next, issued back to back by one thread (in order on the pipe, so S may overwrite the
// columns P was just read from).  Softmax and MMAs therefore alternate between the two buffers by
// construction: neither the special-function units (one exponential per score) nor the tensor
// pipe, which need about the same time per round, waits for the other for long.  Because the
// accumulators alternate by item, an item's first O += P V need not wait for the epilogue of the
// item before, and the producer runs ahead across item boundaries (Q double-buffered).
//
// One reference per row.  The two threads of a row share one online softmax: the same exponent
// reference m (so both halves of P can feed one accumulator), separate partial sums l that the
// epilogue adds.  Each publishes the maximum of its half in shared memory and reads the other's
// (a bounded spin that normally finds the value there); the reference moves lazily, only when
// the row's maximum outgrows it by 2^8, so rescaling O is rare.
//
// Work distribution.  Item t of a CTA is half t & 1 of unit blockIdx.x + (t >> 1) * gridDim.x, a
// unit being the pair (query tile n_qt-1-j, query tile j) of one (b, h): a causal late tile has a
// long list and an early one a short list, so units weigh about the same, and consecutive units
// belong to the same (b, h), so the CTAs running at any time share a few heads' K and V in L2.
//
// Warp roles (448 threads): warps 0-7 softmax (warp w: rows 32 (w & 3) .., column half w >> 2;
// thread = TMEM lane), warps 8-11 epilogue, warp 12 producer (TMA), lane 0 of warp 13 the MMA
// issuer (warp 13 owns the TMEM allocation).  Every wait is bounded; a wait that expires raises
// the device status word and the CTA winds down.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 448;
constexpr int kSubBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled sub-tile
constexpr uint32_t kTmemCols = 512;
constexpr int kRing = 4;              // slots for the rounds' info words and bitmaps
constexpr int kMaxStages = 4;

// per-round word published by the producer
constexpr uint32_t kInfoSlots = 15u;       // bits 0..3: slots of the round
constexpr uint32_t kInfoFirst = 1u << 4;   // first round of its item
constexpr uint32_t kInfoLast = 1u << 5;    // last round of its item
constexpr uint32_t kInfoFull = 1u << 6;    // every entry of the round is kept: no bitmap was copied
constexpr uint32_t kInfoStop = 1u << 7;    // no more work for this CTA

// Shared-memory layout of a K or V stage.  Rows are the round's keys, a row's d elements are cut
// into halves of 64 (128 bytes, the swizzle span).
//   kSplit = false: [half][row / 8][8 rows][128 B]   one TMA box per half (3-D tensor map)
//   kSplit = true:  [row / 8][half][8 rows][128 B]   d = 128 only: one box brings both halves (5-D map)
template <int D, bool kSplit>
struct Cfg {
  static_assert(!kSplit || D == 128, "the split layout is for d = 128");
  static constexpr int kSub = D / 64;                 // halves per row
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kStages = D == 64 ? 4 : 2;     // K / V ring depth
  static constexpr int kKOffset = 2 * kTileBytes;     // after the two Q buffers
  static constexpr int kVOffset = kKOffset + kStages * kTileBytes;
  static constexpr int kBarOffset = kVOffset + kStages * kTileBytes;
  static constexpr int kHalfStride = kSplit ? 1024 : kSubBytes;          // half 0 -> half 1 of the same rows
  static constexpr int kSbo = kSplit ? 2048 : 1024;                      // one group of 8 rows -> the next
  static constexpr int kSlotStride = 2 * kSbo;                           // 16 rows (one slot) -> the next
  static_assert(kStages == kMaxStages || kStages == 2, "ring discipline, see the producer");
};

// Tensor maps of one launch: Q in whole-tile boxes; K and V in boxes of 16, 32, 64 and 128 rows.
struct FwdMaps {
  CUtensorMap q;
  CUtensorMap k[4];
  CUtensorMap v[4];
};

struct Shared {
  alignas(16) uint32_t bitmap[kRing][kTile][4];       // the round's bitmap, row r = words [r][0..3]
  uint32_t xch[2][2][kTile];                          // [score buffer][column half][row]: the half's maximum, tagged
  float l[4][2][kTile];                               // [item % 4][column half][row]: partial sum of the row's weights
  uint64_t q_full[2];
  uint64_t k_full[kMaxStages], v_full[kMaxStages];    // K / V rows of the stage have landed
  uint64_t b_full[kRing];                             // info word and bitmap of the round are valid
  uint64_t mma_done[4];                               // event e (slot e % 4): S of round e and O += P V of round e - 2 have completed
  uint64_t p_full[2];                                 // per score buffer: P written (8 warps)
  uint64_t o_done[2], o_free[2];                      // per accumulator: O complete / O read out by the epilogue
  uint64_t ml_ready[4];                               // per item: the softmax warps have handed over l
  int32_t ml_bh[4], ml_qt[4];                         // the item handed over (b * H + h, query tile); qt = -1: no more items
  uint32_t info[kRing];
  int32_t item_bh[kRing], item_qt[kRing];             // the item a round belongs to
  uint32_t tmem_base;
  int abort_flag;
};

// Development aid: with -DAP_FWD_TRACE thread block 0 records cycle stamps of its roles
// ([0][role][round][point]; roles: 0 producer, 1 MMA issuer, 2..5 softmax warps 0, 1, 4, 5), read back
// through ap_debug_fwd_trace.  Compiled out otherwise.
#ifdef AP_FWD_TRACE
constexpr int kTraceRounds = 256, kTracePoints = 16;
__device__ long long g_fwd_trace[1][6][kTraceRounds][kTracePoints];
#define AP_TRACE(sx, role, g, k)                                                              \
  do {                                                                                       \
    if (blockIdx.x == 0 && lane == 0 && (g) < (uint32_t)kTraceRounds) g_fwd_trace[sx][role][g][k] = clock64(); \
  } while (0)
#else
#define AP_TRACE(sx, role, g, k) \
  do {                          \
  } while (0)
#endif
// the same from inside a single elected thread
#ifdef AP_FWD_TRACE
#define AP_TRACE1(sx, role, g, k)                                                                      \
  do {                                                                                                \
    if (blockIdx.x == 0 && (g) < (uint32_t)kTraceRounds) g_fwd_trace[sx][role][g][k] = clock64();      \
  } while (0)
#else
#define AP_TRACE1(sx, role, g, k) \
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

// First half of a thread's softmax step over kChunks 32-column chunks of S at `tmem_b`: the scores
// come into registers, pruned entries (bitmap bit 0) are replaced by -inf (exp2 of -inf is
// exactly 0); returns the maximum over kept entries.
template <int kChunks, bool kMasked>
__device__ __forceinline__ float load_mask_max(uint32_t tmem_b, uint2 bw, uint32_t (&xs)[64]) {
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
  return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
}

// Second half: P = exp2(c*S - c*m) as 16-bit values over the first half of each chunk's columns of
// S (the stores are not waited for here); returns the sum of the weights as the MMA will see them.
template <int kChunks, bool kF16>
__device__ __forceinline__ float exp_store(uint32_t tmem_b, const uint32_t (&xs)[64], float scale_log2, float neg_mc) {
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
  return sum0 + sum1;
}

// The maximum of a row half as it is exchanged between the row's two threads: the two lowest bits
// of the value carry a tag (which use of the slot this is), so one 32-bit store publishes both, and
// both threads then work with the same (slightly truncated) values.  -inf travels as the most
// negative finite number.
constexpr uint32_t kXchMinusInf = 0xff7ffffcu;
__device__ __forceinline__ uint32_t xch_encode(float v, uint32_t tag) {
  const uint32_t bits = v == -CUDART_INF_F ? kXchMinusInf : (__float_as_uint(v) & ~3u);
  return bits | tag;
}
__device__ __forceinline__ float xch_decode(uint32_t w) {
  const uint32_t bits = w & ~3u;
  return bits == kXchMinusInf ? -CUDART_INF_F : __uint_as_float(bits);
}

// dbg_skip != 0 (test hook, see ap_debug_expire_waits): the producer leaves out the copies and the
// arrivals of its first round, so that the waits on it run out.
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
  unsigned char *q_s = smem;
  unsigned char *k_s = smem + C::kKOffset;
  unsigned char *v_s = smem + C::kVOffset;
  Shared *sh = reinterpret_cast<Shared *>(smem + C::kBarOffset);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh->q_full[i], 1);
      mbar_init(&sh->p_full[i], 8);  // softmax warps
      mbar_init(&sh->o_done[i], 1);
      mbar_init(&sh->o_free[i], 4);  // epilogue warps
    }
    for (int i = 0; i < kMaxStages; ++i) {
      mbar_init(&sh->k_full[i], 1);
      mbar_init(&sh->v_full[i], 1);
    }
    for (int i = 0; i < kRing; ++i) mbar_init(&sh->b_full[i], 1);
    for (int i = 0; i < 4; ++i) mbar_init(&sh->mma_done[i], 1);
    for (int i = 0; i < 4; ++i) mbar_init(&sh->ml_ready[i], 8);
    sh->abort_flag = 0;
    fence_mbar_init();
  }
  // exchange slots start with the tag of their fourth use, which the first three never ask for
  for (int i = threadIdx.x; i < 2 * 2 * kTile; i += kThreads) (&sh->xch[0][0][0])[i] = kXchMinusInf | 3u;
  if (warp == 13) {
    tmem_alloc(&sh->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  // score buffer of round g, output accumulator of the n-th item
  auto s_addr = [&](uint32_t g) { return tmem + 128u * (g & 1u); };
  auto o_addr = [&](uint32_t n) { return tmem + 256u + 128u * (n & 1u); };
  const WaitCtx wc{&sh->abort_flag, err, max_polls};
  // producer: the copies armed last (item / round numbers; -1: none), for the wind-down after an expired wait
  int armed_q = -1, armed_k = -1, armed_v = -1;

  if (warp == 12) {
    // ------------------------------------------------------------ producer
    if (lane < 4) {
      prefetch_tensormap(&maps.k[lane]);
      prefetch_tensormap(&maps.v[lane]);
    }
    if (lane == 4) prefetch_tensormap(&maps.q);
    bool ok = true;
    uint32_t g = 0, n = 0;   // rounds / non-empty items so far
    const int n_half = (n_qt + 1) / 2, n_units = B * H * n_half;
    const int item_step = (int)gridDim.x;
    struct ItemRef {
      int bh, qt, rho0, rho1;  // rounds [rho0, rho1): loaded here, first read when the item begins
      bool in_range, exists;   // !exists: no such item (the unit's halves coincide)
    };
    // (called for t = 0, 1, 2, ... in turn: the unit's (j, bh, h = bh % H) are stepped from one unit
    // of this CTA to the next instead of divided out of the unit number every time)
    int cur_u = (int)blockIdx.x, cur_j = cur_u % n_half, cur_bh = cur_u / n_half, cur_h = cur_bh % H;
    const int step_j = item_step % n_half, step_bh = item_step / n_half, step_h = step_bh % H;
    auto item_ref = [&](int t) {
      ItemRef it;
      if (t >= 2 && !(t & 1)) {  // the next unit
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
      const int u = cur_u;
      it.in_range = u < n_units;
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
    // Ring discipline.  K and V of round g go to stage g % kStages, its info word and bitmap to
    // slot g % kRing.  K may be overwritten once S = Q K^T of round g - kStages has completed
    // (event g - kStages), V once O += P V of that round has (event g - kStages + 2).  The info slot
    // last served round g - kRing, whose softmax must be over: with kStages == kRing that is what
    // the V condition says; with a ring of two, S of round g - 2 could only be issued behind
    // O += P V of round g - 4, i.e. after that round's softmax, so the K condition implies it.
    // (Completion of MMAs is announced once per round, as event e = "S of round e and O += P V of
    // round e - 2 are complete": a commit costs the tensor pipe about two MMAs' time, so the MMA
    // thread makes one per round and everybody derives what they need from it.)
    // Events complete in order and a slot's phase bit only tells the two most recent uses apart,
    // so an event at or before the newest one already seen is known to be over and is not waited
    // for; a newer one cannot be more than a slot's period ahead, because the MMAs after it need
    // copies this warp has not issued yet.
    int seen_event = -1;
    auto wait_event = [&](int e) {
      if (e <= seen_event) return;
      seen_event = e;
      if (lane == 0) {
        uint64_t *bar = &sh->mma_done[e & 3];
        const uint32_t parity = ((uint32_t)e >> 2) & 1u;
        ok = mbar_try_wait(bar, parity) || wait_or_abort(bar, parity, wc);
      }
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
    // V of a round is copied one round later than its K: K only needs S = Q K^T of the round that
    // used the stage before to be over, V needs that round's O += P V, which comes much later;
    // issued in round order, the V copy would hold back the next round's K.
    bool pv_valid = false;
    int pv_st = 0, pv_ng = 0, pv_row = 0, pv_run = 0, pv_bh = 0, pv_g = 0;
    auto issue_v = [&]() {
      if (C::kStages != kRing) wait_event(pv_g - C::kStages + 2);
      if (!ok) return;
      if (lane == 0) {
        mbar_arrive_expect_tx(&sh->v_full[pv_st], (uint32_t)pv_ng * 16u * D * 2u);
        armed_v = pv_g;
      }
      __syncwarp();
      load_run(v_s + pv_st * C::kTileBytes, maps.v, &sh->v_full[pv_st], pv_row, pv_run, pv_bh);
      pv_valid = false;
    };
    // the rounds of an item are looked up two items ahead: the loads of item t + 2 are issued when
    // item t begins and their results first touched when item t + 1 does
    int q_last[2] = {-1, -1};  // last round of the item that used each Q buffer before
    ItemRef next = item_ref(0);
    ItemRef next2 = item_ref(1);
    // ... and the slot rows and info byte of its first round while the current item is under way
    int pf_t = -1, pf_row = -1;
    uint32_t pf_info = 0u;
    for (int t = 0; next.in_range && ok; ++t) {
      const ItemRef cur = next;
      next = next2;
      next2 = item_ref(t + 2);
      if (!cur.exists) continue;
      const int bh = cur.bh, qt = cur.qt, rho0 = cur.rho0, n_rounds = cur.rho1 - cur.rho0;
      if (n_rounds == 0) {
        // nothing kept in this query tile: its output rows are zero (nobody else sees the item)
        const int rows = min(kTile, Lq - qt * kTile);
        uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + (size_t)qt * kTile) * D);
        for (int i = lane; i < rows * (D / 8); i += 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        continue;
      }
      // Q of this item into its buffer (free once the last S = Q K^T of item n - 2 has completed)
      const int qb = (int)(n & 1u);
      wait_event(q_last[qb]);
      q_last[qb] = (int)g + n_rounds - 1;
      if (lane == 0) {
        if (ok) {
          mbar_arrive_expect_tx(&sh->q_full[qb], C::kTileBytes);
#pragma unroll
          for (int s = 0; s < C::kSub; ++s)
            tma_load_3d(q_s + qb * C::kTileBytes + s * kSubBytes, &maps.q, &sh->q_full[qb], 64 * s, qt * kTile, bh);
          armed_q = (int)n;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      // slot rows (lanes 0..7) and info byte of a round are fetched one round ahead
      int next_row = pf_row;
      uint32_t next_info = pf_info;
      if (pf_t != t) {
        next_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)rho0 * 8 + lane) : -1;
        next_info = ldg_now_u8(round_info + rho0);
      }
      for (int v = 0; v < n_rounds && ok; ++v, ++g) {
        const int row = next_row;
        const uint32_t rinfo = next_info;
        if (v + 1 < n_rounds) {
          next_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)(rho0 + v + 1) * 8 + lane) : -1;
          next_info = ldg_now_u8(round_info + rho0 + v + 1);
        } else if (next.exists && next.rho1 > next.rho0) {
          pf_t = t + 1;
          pf_row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)next.rho0 * 8 + lane) : -1;
          pf_info = ldg_now_u8(round_info + next.rho0);
        }
        const int st = (int)(g % C::kStages);
        const int ng = (int)(rinfo & 15u);
        const bool full = (rinfo & 0x80u) != 0u;
        // slots whose key rows follow one another form a run
        const int row_before = __shfl_up_sync(0xffffffffu, row, 1);
        const bool head = lane < ng && (lane == 0 || row != row_before + 16);
        const uint32_t heads = __ballot_sync(0xffffffffu, head);
        const uint32_t later = lane < 31 ? heads >> (lane + 1) : 0u;
        const int run = head ? (later ? __ffs((int)later) : ng - lane) : 0;  // slots in this lane's run
        const int si = (int)(g % kRing);
        wait_event((int)g - C::kStages);
        if (ok && C::kStages == kRing) wait_event((int)g - C::kStages + 2);
        if (!ok) break;
        AP_TRACE(0, 0, g, 0);
        const uint32_t bytes = (uint32_t)ng * 16u * D * 2u;
        const bool skip = dbg_skip != 0 && g == 0;
        if (lane == 0 && !skip) {
          sh->info[si] = (uint32_t)ng | (v == 0 ? kInfoFirst : 0u) | (v + 1 == n_rounds ? kInfoLast : 0u) |
                         (full ? kInfoFull : 0u);
          sh->item_bh[si] = bh;
          sh->item_qt[si] = qt;
          mbar_arrive_expect_tx(&sh->k_full[st], bytes);
          armed_k = (int)g;
          if (full) {
            mbar_arrive(&sh->b_full[si]);
          } else {
            mbar_arrive_expect_tx(&sh->b_full[si], kBitmapWords * 4);
            bulk_load(&sh->bitmap[si][0][0], round_bitmap + (size_t)(rho0 + v) * kBitmapWords, kBitmapWords * 4,
                      &sh->b_full[si]);
          }
        }
        __syncwarp();
        if (!skip) load_run(k_s + st * C::kTileBytes, maps.k, &sh->k_full[st], row, run, bh);
        AP_TRACE(0, 0, g, 1);
        if (pv_valid) issue_v();
        if (!ok) break;
        if (!skip) {
          pv_valid = true;
          pv_st = st, pv_ng = ng, pv_row = row, pv_run = run, pv_bh = bh, pv_g = (int)g;
        }
      }
      ++n;
    }
    if (ok && pv_valid) issue_v();
    // no more work: one more stage carries the stop word
    if (ok) {
      const int st = (int)(g % C::kStages);
      wait_event((int)g - C::kStages);
      if (ok && C::kStages == kRing) wait_event((int)g - C::kStages + 2);
      if (ok && lane == 0) {
        sh->info[g % kRing] = kInfoStop;
        mbar_arrive(&sh->k_full[st]);
        mbar_arrive(&sh->b_full[g % kRing]);
      }
    }
  } else if (warp == 13) {
    // ------------------------------------------------------------ MMA issuer
    // One thread walks the rounds.  It keeps S two rounds ahead of O += P V: the scores of round
    // g + 2 are issued right behind O += P V of round g, into the buffer that step has just read P
    // from (in order on the tensor pipe, so no wait in between).  Every instruction between a
    // hand-over and the MMAs it releases is on the critical path, so this thread's code is kept
    // short: descriptors are prepared once, nothing is shared with other lanes.
    if (lane == 0) {
      const uint32_t q_addr = smem_u32(q_s), k_addr = smem_u32(k_s), v_addr = smem_u32(v_s);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true, kF16);
      bool ok = true;
      auto wait = [&](uint64_t *bar, uint32_t parity) {
        if (!mbar_try_wait(bar, parity)) ok = wait_or_abort(bar, parity, wc);
        return ok;
      };
      // Low descriptor words of the Q buffers and of the first K / V stage (a later stage adds its
      // distance, in units of 16 bytes, to the address field: stage bases are multiples of 1024 bytes
      // and shared memory ends below 256 KB, so the sum stays inside the field).  With these in
      // registers, issuing a round's MMAs takes a few instructions per MMA; this thread shares its
      // scheduler with two busy softmax warps and every instruction of its own costs it a turn.
      uint32_t q_lo[2][D / 16], k_lo[D / 16], v_lo[8];
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int sub = ks / 4, off = (ks % 4) * 32;  // D/16 steps of K = 16 (32 bytes inside the swizzled rows)
#pragma unroll
        for (int b = 0; b < 2; ++b) q_lo[b][ks] = smem_desc_lo(q_addr + b * C::kTileBytes + sub * kSubBytes + off, 16);
        k_lo[ks] = smem_desc_lo(k_addr + sub * C::kHalfStride + off, 16);
      }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) v_lo[ks] = smem_desc_lo(v_addr + ks * C::kSlotStride, C::kHalfStride);
      static_assert(C::kTileBytes % 1024 == 0, "stage distance in descriptor units");
      constexpr uint32_t kStageUnits = C::kTileBytes >> 4;
      constexpr uint32_t q_hi = smem_desc_hi_sw128(1024), kv_hi = smem_desc_hi_sw128(C::kSbo);
      // ---- the S side: a cursor over the rounds whose scores have not been issued yet
      uint32_t s_g = 0, s_items = 0;  // s_items: items whose last S was issued
      bool s_stop = false;
      // what O += P V needs to know of the (at most two) rounds whose S is under way; entry g & 1
      uint32_t q_info[2] = {0u, 0u};
      auto s_advance = [&]() {
        if (s_stop) return;
        const int st = (int)(s_g % C::kStages);
        if (!wait(&sh->k_full[st], (s_g / C::kStages) & 1u)) return;
        const uint32_t info = sh->info[s_g % kRing];
        if (info & kInfoStop) {
          s_stop = true;
          return;
        }
        const int qb = (int)(s_items & 1u);
        if ((info & kInfoFirst) && !wait(&sh->q_full[qb], (s_items >> 1) & 1u)) return;
        const uint32_t idesc_qk = idesc_bf16_f32(128, 16 * (int)(info & kInfoSlots), false, false, kF16);
        const uint32_t d_tmem = s_addr(s_g);
        const uint32_t k_units = (uint32_t)st * kStageUnits;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          mma_ss(d_tmem, smem_desc_join(qb ? q_lo[1][ks] : q_lo[0][ks], q_hi), smem_desc_join(k_lo[ks] + k_units, kv_hi),
                 idesc_qk, ks > 0);
        if (info & kInfoLast) ++s_items;
        AP_TRACE1(0, 1, s_g, 0);
        if (s_g & 1u) q_info[1] = info; else q_info[0] = info;
        ++s_g;
      };
      // events 0 and 1: the first two rounds' scores (event 1 is announced even if there is no
      // second round, so that the slots' phases stay in step with the event numbers)
      s_advance();
      mma_commit(&sh->mma_done[0]);
      if (ok) s_advance();
      mma_commit(&sh->mma_done[1]);
      uint32_t n = 0;  // items whose O += P V is complete
      for (uint32_t g = 0; ok && g < s_g; ++g) {
        const int st = (int)(g % C::kStages);
        const uint32_t sb = g & 1u;
        const uint32_t info = sb ? q_info[1] : q_info[0];
        const int ng = (int)(info & kInfoSlots);
        const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
        // O += P V.  What is ready early first; P, which the softmax has just finished, last.
        if (!wait(&sh->v_full[st], (g / C::kStages) & 1u)) break;
        // the first round of an item overwrites O: the epilogue of the item before last, which used
        // this accumulator, must have read it
        const uint32_t ob = n & 1u;
        if (first && n >= 2u && !wait(&sh->o_free[ob], ((n >> 1) - 1u) & 1u)) break;
        const uint32_t o_acc = o_addr(n), p_base = s_addr(g);
        const uint32_t v_units = (uint32_t)st * kStageUnits;
        AP_TRACE1(0, 1, g, 1);
        if (!wait(&sh->p_full[sb], (g >> 1) & 1u)) break;
        AP_TRACE1(0, 1, g, 2);
        tc_fence_after_sync();
        // One K step of 16 keys per slot.  P (16-bit) of a 32-column chunk is written over the
        // first 16 columns of that chunk of S, so slot q's eight columns of P start at column
        // 32 (q / 2) + 8 (q % 2).  The item's first step overwrites the accumulator.
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          if (ks < ng)
            mma_ts(o_acc, p_base + 32 * (ks >> 1) + 8 * (ks & 1), smem_desc_join(v_lo[ks] + v_units, kv_hi), idesc_pv,
                   (first && ks == 0) ? 0u : 1u);
        }
        AP_TRACE1(0, 1, g, 4);
        // the scores two rounds ahead, into the buffer just read
        s_advance();
        if (!ok) break;
        // event g + 2: everything issued so far is through
        mma_commit(&sh->mma_done[(g + 2u) & 3u]);
        if (last) {
          // (the epilogue may come to look long after the event: it gets a barrier of its own, once per item)
          mma_commit(&sh->o_done[ob]);
          ++n;
        }
        AP_TRACE1(0, 1, g, 3);
      }
    }
    __syncwarp();
  } else if (warp < 8) {
    // ------------------------------------------------------------ softmax
    const int half = warp >> 2;              // this thread's half of a round's columns: chunks 2 half, 2 half + 1
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const float ref_slack = 8.f / scale_log2;
    const bool tracer = (warp & 3) < 2;      // (development aid: the warps whose cycle stamps are kept)
    (void)tracer;
    bool ok = true;
    uint32_t n = 0;
    float m = -CUDART_INF_F, l = 0.f;       // the row's exponent reference; this half's sum of weights
    bool o_started = false;                  // an earlier round of the item added to the accumulator
    int cur_bh = 0, cur_qt = 0;
    uint32_t tmem_og = 0;                    // this thread's 64 (d = 128) or 32 columns of the item's accumulator
    // What the softmax needs to know of a round (its info word, the item on an item's first round,
    // this thread's two bitmap words) is read one round ahead, while the round before is worked
    // on, so that these shared-memory round trips are off the chain S -> softmax -> O += P V.
    struct RoundHead {
      uint32_t info;
      uint2 bw;
      int bh, qt;
    };
    auto read_head = [&](uint32_t g) {
      RoundHead hd;
      hd.info = kInfoStop, hd.bw = make_uint2(0xffffffffu, 0xffffffffu), hd.bh = 0, hd.qt = 0;
      const int si = (int)(g % kRing);
      ok = warp_wait(&sh->b_full[si], (g / kRing) & 1u, lane, wc);
      if (!ok) return hd;
      hd.info = sh->info[si];
      if (hd.info & kInfoStop) return hd;
      if (!(hd.info & kInfoFull)) hd.bw = *reinterpret_cast<const uint2 *>(&sh->bitmap[si][r][2 * half]);
      if (hd.info & kInfoFirst) {
        hd.bh = sh->item_bh[si];
        hd.qt = sh->item_qt[si];
      }
      return hd;
    };
    RoundHead head = read_head(0);
    for (uint32_t g = 0; ok; ++g) {
      const uint32_t sb = g & 1u;
      const uint32_t info = head.info;
      if (info & kInfoStop) break;
      const uint2 bw = head.bw;
      const int ng = (int)(info & kInfoSlots);
      const bool last = (info & kInfoLast) != 0u;
      const bool tile_full = (info & kInfoFull) != 0u;
      if (info & kInfoFirst) {
        cur_bh = head.bh;
        cur_qt = head.qt;
        m = -CUDART_INF_F;
        l = 0.f;
        o_started = false;
        tmem_og = o_addr(n) + lane_addr + (uint32_t)(half * (D / 2));
      }
      const int n_sl = min(max(ng - 4 * half, 0), 4);   // this half's slots
      const uint32_t tmem_b = s_addr(g) + lane_addr + 64u * (uint32_t)half;
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 0);
      ok = warp_wait(&sh->mma_done[g & 3u], (g >> 2) & 1u, lane, wc);
      if (!ok) break;
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 1);
      tc_fence_after_sync();
      // Straight-line code per case (two chunks, one chunk, none; masked or not): the chunks'
      // loads, maxima, exponentials and stores interleave freely.
      uint32_t xs[64];
      float my_max = -CUDART_INF_F;
      if (n_sl > 2) {
        my_max = tile_full ? load_mask_max<2, false>(tmem_b, bw, xs) : load_mask_max<2, true>(tmem_b, bw, xs);
      } else if (n_sl > 0) {
        my_max = load_mask_max<1, true>(tmem_b, bw, xs);
      }
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 4);
      // The row's two threads exchange the maxima of their halves: each publishes its own under the
      // tag of this use of the slot and reads the other's as soon as it carries the same tag.
      const uint32_t tag = (g >> 1) & 3u;
      const uint32_t mine = xch_encode(my_max, tag);
      sts_volatile(smem_u32(&sh->xch[sb][half][r]), mine);
      // (meanwhile: the next round's head)
      head = read_head(g + 1);
      if (!ok) break;
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 5);
      uint32_t theirs = 0u;
      {
        const uint32_t addr = smem_u32(&sh->xch[sb][1 - half][r]);
        bool got = false;
        for (uint32_t i = 0; i < wc.max_polls && !got; ++i) {
          theirs = lds_volatile(addr);
          got = (theirs & 3u) == tag;
          if (!got && (i & 63u) == 63u && *wc.abort_flag) break;
        }
        if (!__all_sync(0xffffffffu, got)) {  // the other warp is gone: give up as every wait does
          if (!*wc.abort_flag) {
            *wc.abort_flag = 1;
            atomicOr(err, kDevErrTimeout);
          }
          ok = false;
          break;
        }
      }
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 2);
      const float row_max = fmaxf(xch_decode(mine), xch_decode(theirs));
      // The reference follows the row's maximum lazily: it moves only when the maximum outgrows it
      // by more than 2^8 in the exp2 domain (weights stay <= 256, well inside bf16 and fp32
      // range), which saves most rescales of O.  O / l does not depend on the reference.
      const bool move = row_max > m + ref_slack;   // also true for the first kept entry (m = -inf)
      const float m_new = move ? row_max : m;
      const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
      const float alpha = move ? ex2_approx((m - m_safe) * scale_log2) : 1.f;  // 0 when m was -inf
      const float neg_mc = -m_safe * scale_log2;
      m = m_new;
      // Rescale this thread's columns of the running output where the reference moved.  O += P V of
      // the round before may still be running: wait for it first.  (It cannot be further ahead: the
      // step after it needs the P written below.)
      if (o_started && __any_sync(0xffffffffu, alpha != 1.f)) {
        ok = warp_wait(&sh->mma_done[(g + 1u) & 3u], ((g + 1u) >> 2) & 1u, lane, wc);  // event g + 1: O += P V of round g - 1
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < D / 64; ++c) {
          uint32_t o[32];
          tmem_ld32(tmem_og + 32 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st32(tmem_og + 32 * c, o);
        }
      }
      float sum = 0.f;
      if (n_sl > 2) sum = exp_store<2, kF16>(tmem_b, xs, scale_log2, neg_mc);
      else if (n_sl > 0) sum = exp_store<1, kF16>(tmem_b, xs, scale_log2, neg_mc);
      l = l * alpha + sum;
      o_started = true;
      tmem_wait_st();
      // one arrival per warp (32 lanes arriving one by one would take hundreds of cycles)
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->p_full[sb]);
      if (tracer) AP_TRACE(0, 2 + (warp & 1) + 2 * half, g, 3);
      if (!last) continue;
      // The item's rounds are over for the softmax warps: they hand their partial sums to the
      // epilogue warps and go on with the next item.  The slot of the hand-over ring was last used by
      // item n - 4, whose epilogue read it before it released that item's accumulator, which the
      // first O += P V of item n - 2 waited for; that step was issued before the last S of this item.
      sh->l[n & 3u][half][r] = l;
      if (threadIdx.x == 0) {
        sh->ml_bh[n & 3u] = cur_bh;
        sh->ml_qt[n & 3u] = cur_qt;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ml_ready[n & 3u]);
      ++n;
    }
    // no more items: tell the epilogue warps (the slot is free by the argument above)
    if (ok) {
      if (threadIdx.x == 0) sh->ml_qt[n & 3u] = -1;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ml_ready[n & 3u]);
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------ epilogue
    // Per finished item: O / (l_0 + l_1), rounded once to the tensors' type.
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    bool ok = true;
    for (uint32_t n = 0; ok; ++n) {
      ok = warp_wait(&sh->ml_ready[n & 3u], (n >> 2) & 1u, lane, wc);
      if (!ok) break;
      const int item_qt = sh->ml_qt[n & 3u], item_bh = sh->ml_bh[n & 3u];
      if (item_qt < 0) break;
      const float l = sh->l[n & 3u][0][r] + sh->l[n & 3u][1][r];
      const int i = item_qt * kTile + r;
      uint16_t *orow = O + ((size_t)item_bh * Lq + i) * D;
      // a row without kept entries has l = 0 and P = 0 throughout: exact zeros (its accumulator may
      // never have been written)
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const uint32_t ob = n & 1u;
      ok = warp_wait(&sh->o_done[ob], (n >> 1) & 1u, lane, wc);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t o_acc = o_addr(n) + lane_addr;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(o_acc + 32 * c, o);
        tmem_wait_ld();
        if (c == D / 32 - 1) {  // this thread's rows of O are in registers: the item after next may overwrite them
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh->o_free[ob]);
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
  if (warp == 12 && lane == 0 && *wc.abort_flag) {
    // A wait expired somewhere in the CTA and every role has left its loop.  Copies the producer
    // armed may still be in flight: wait (bounded) for the most recent ones before the CTA's shared
    // memory is given up (earlier ones completed before these were armed).
    if (armed_q >= 0) mbar_wait(&sh->q_full[armed_q & 1], ((uint32_t)armed_q >> 1) & 1u, 1u << 16);
    for (int a = armed_k - 1; a <= armed_k; ++a)
      if (a >= 0) {
        mbar_wait(&sh->k_full[a % C::kStages], ((uint32_t)a / C::kStages) & 1u, 1u << 16);
        mbar_wait(&sh->b_full[a % kRing], ((uint32_t)a / kRing) & 1u, 1u << 16);
      }
    for (int a = armed_v - 1; a <= armed_v; ++a)
      if (a >= 0) mbar_wait(&sh->v_full[a % C::kStages], ((uint32_t)a / C::kStages) & 1u, 1u << 16);
  }
  __syncthreads();
  if (warp == 13) tmem_dealloc(tmem, kTmemCols);
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
