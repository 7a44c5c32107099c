// Masked attention of Section 3.2 for bf16 tensors on the tcgen05 tensor cores.
//
// Persistent kernel, one CTA per SM.  A work item is one (b, h, query tile of 128 rows); items
// are handed out in pairs (a late and an early query tile of the same head), CTA c taking pairs
// c, c + gridDim.x, ...  The CTA follows the schedule stored
// with the tile list: the ROUNDS of the item's (h, qt) list row.  A round holds up to eight
// non-empty groups of 16 key columns (slots), taken in list order from one or several key tiles,
// together with the bitmap of exactly those columns; groups without a kept entry never appear, so
// leaving them out is exact.  Per round:
//   S  = Q K_round^T         tcgen05.mma, N = 16 * slots, fp32 accumulator in TMEM
//   P  = exp2(c*S - c*m)     one thread per query row reads its S row from TMEM, replaces pruned
//                            entries by -inf (the round's bitmap decides, exactly), keeps the
//                            running reference m and sum l of an online softmax, rescales O when m
//                            moved, and writes P as bf16 over S in TMEM
//   O += P V_round           tcgen05.mma, A = P from TMEM, B = V (MN-major), one K step of 16 keys
//                            per slot
// and at the item's last round O / l is written (zeros for rows that never saw a kept entry).
//
// Everything a round needs arrives through one ring of stages in shared memory, filled by the
// producer warp: the K and V rows of the round's slots (TMA boxes of 16..128 rows, slots whose key
// rows follow one another are copied as one box), the round's bitmap (one bulk copy) and a word
// that says how many slots there are and whether the round starts or ends an item.  The producer
// runs ahead across item boundaries, so an item's first loads are hidden behind the previous
// item's last rounds.  S is double-buffered in TMEM and the two kinds of MMA are issued by two
// warps, each held back only by what it really depends on: S(g) = Q K^T waits for K(g) and for
// O += P V of round g - 2 (the previous user of that S buffer), O += P(g) V for P(g) and V(g).
// So the softmax threads find the next S ready when they finish a round.
//
// A list row that carries GATHERED ROUNDS (the tile list's second schedule: the row's active key
// columns, those of whole 16-column groups first, 128 per round, with the bitmap re-packed per
// column) is followed through those instead, by the kernel's second instantiation: a slot of 16
// keys that follow one another is still one box; the rows of any other slot are copied one by one
// (see the producer).  Everything after the copies is the same: N = 16 * slots, the round's
// bitmap, the same softmax.
//
// The softmax is shared by two groups of four warps.  The 32-column chunks of a round alternate
// between them (chunk c belongs to group c & 1), and each group is an online softmax of its own:
// its own reference m and sum l per query row and its own output accumulator in TMEM (O += P V
// of a slot goes to the accumulator of the slot's group), so the groups never exchange anything
// inside a round.  The item's epilogue merges the two partial results
//   O = (a_0 O_0 + a_1 O_1) / (a_0 l_0 + a_1 l_1),   a_i = exp2(c (m_i - max(m_0, m_1))).
//
// Warp roles (480 threads): warps 0-3 softmax group 0, warps 4-7 group 1 (thread = query row =
// TMEM lane), warp 8 producer, warp 9 issuer of S = Q K^T and TMEM owner, warp 10 issuer of
// O += P V, warps 11-14 epilogue (the softmax groups hand (m, l) over and go on with the next
// item while the epilogue warps wait for the item's last O += P V, merge and write).  The softmax
// body of a round is straight-line code: both 32-column chunks of the group are always loaded, and
// the mask is applied by select (branches around the tensor-memory loads cost more than the loads).
// TMEM (512 columns): S[0] at column 0, S[1] at 128, O_0 at 256, O_1 at 384 (d = 128); at d = 64
// the pair (O_0, O_1) takes 128 columns and two items' pairs alternate at 256 and 384.  Every wait
// is bounded, with the poll limit a kernel argument; a wait that expires raises the device status
// word and the CTA winds down (the end of a CTA's work reaches the epilogue warps through a word of
// its own, not through the ring that hands (m, l) over).
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 480;
constexpr int kSoftmaxWarps = 8;       // two groups of four; barriers the softmax warps arrive on count warps
constexpr int kSubBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled sub-tile
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxStages = 4;

// per-stage word published by the producer
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
  static constexpr int kStages = D == 64 ? 4 : 2;     // ring depth
  static constexpr int kKOffset = 2 * kTileBytes;     // after the two Q buffers
  static constexpr int kVOffset = kKOffset + kStages * kTileBytes;
  static constexpr int kBarOffset = kVOffset + kStages * kTileBytes;
  static constexpr int kSmemBytes = kBarOffset + 18 * 1024 + 1024;  // + bitmaps/barriers + alignment slack
  static constexpr int kHalfStride = kSplit ? 1024 : kSubBytes;          // half 0 -> half 1 of the same rows
  static constexpr int kSbo = kSplit ? 2048 : 1024;                      // one group of 8 rows -> the next
  static constexpr int kSlotStride = 2 * kSbo;                           // 16 rows (one slot) -> the next
};

// Tensor maps of one launch: Q in whole-tile boxes; K and V in boxes of 16, 32, 64 and 128 rows.
struct FwdMaps {
  CUtensorMap q;
  CUtensorMap k[4];
  CUtensorMap v[4];
};

// The second schedule of a tile list, followed for the list rows that have gathered rounds.
struct Gathered {
  const int32_t *ptr;
  const int32_t *keys;
  const uint8_t *info;
  const uint32_t *bitmap;
  const uint16_t *K, *V;  // the tensors themselves: single key rows are fetched with plain asynchronous copies
  int Lk;
  int mode;
  const int32_t *unit_qt;  // [H][ceil(n_qt/2)][2]: the query tiles of each unit of work (kPairs)
};

struct Shared {
  alignas(16) uint32_t bitmap[kMaxStages][kTile][4];  // the round's bitmap, row r = words [r][0..3]
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[kMaxStages], v_full[kMaxStages];    // K / V rows of the stage have landed
  uint64_t b_full[kMaxStages];                        // info word and bitmap of the stage are valid
  uint64_t k_empty[kMaxStages], v_empty[kMaxStages];  // S = Q K^T / O += P V of the stage has completed
  uint64_t s_full[2], p_full[2];                      // per S buffer
  uint64_t pv_done[2];                                // O += P V of a round has completed, per S buffer
  uint64_t o_done[2], o_free[2];                      // per item: O complete / O read out by the epilogue
                                                      // (one pair per set of accumulators)
  uint64_t ml_ready[4];                               // per item: both groups have handed over (m, l)
  float2 ml[4][2][kTile];                             // [item % 4][group][row] = (m, l)
  int32_t ml_bh[4], ml_qt[4];                         // the item handed over (b * H + h, query tile); qt = -1: no more items
  alignas(16) int32_t keys[2][kTile];                 // producer's scratch: keys of a gathered round (two rounds in flight)
  uint32_t info[kMaxStages];
  int32_t item_bh[kMaxStages], item_qt[kMaxStages];   // the item a stage's round belongs to
  uint32_t tmem_base;
  uint32_t n_items;   // set when the CTA's last item has been handed to the epilogue: how many there were
  int abort_flag;
  uint32_t max_polls; // poll limit of every wait (directly behind abort_flag: wait_or_abort reads both)
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait that also gives up as soon as another thread of the CTA has.
__device__ __noinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag, unsigned *err,
                                           uint32_t max_polls) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 1024) __nanosleep(64);
  }
  *abort_flag = 1;
  atomicOr(err, kDevErrTimeout);
  return false;
}

// The same wait for a whole (converged) warp: one lane polls - 32 lanes polling one barrier would
// serialise - and the outcome is shared.
template <int kPollLane = 0>
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, int lane, volatile int *abort_flag,
                                          unsigned *err, uint32_t max_polls) {
  bool ok = true;
  if (lane == kPollLane && !mbar_try_wait(bar, parity)) ok = wait_or_abort(bar, parity, abort_flag, err, max_polls);
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

// kGath: the launch may follow gathered rounds (a second instantiation, so that the code for them
// costs lists without a gathered schedule nothing).  kPairs: the units of work are the pairs of query
// tiles the list's builder chose (balanced by their rounds) instead of (n_qt - 1 - j, j).
template <int D, bool kSplit, bool kF16, bool kGath, bool kPairs>
__global__ void __launch_bounds__(kThreads, 1)
fwd_tc_kernel(const __grid_constant__ FwdMaps maps, uint16_t *__restrict__ O,
              const int32_t *__restrict__ round_ptr, const int32_t *__restrict__ round_rows,
              const uint8_t *__restrict__ round_info, const uint32_t *__restrict__ round_bitmap,
              const Gathered gth, int B, int H, int Lq, int n_qt, float scale_log2, unsigned *err,
              uint32_t max_polls, int dbg_skip) {
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
      mbar_init(&sh->q_empty[i], 1);
      mbar_init(&sh->s_full[i], 1);
      mbar_init(&sh->p_full[i], kSoftmaxWarps);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&sh->k_full[s], 1);
      mbar_init(&sh->v_full[s], 1);
      mbar_init(&sh->k_empty[s], 1);
      mbar_init(&sh->v_empty[s], 1);
    }
    for (int s = 0; s < kMaxStages; ++s) mbar_init(&sh->b_full[s], 1);
    mbar_init(&sh->pv_done[0], 1);
    mbar_init(&sh->pv_done[1], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&sh->o_done[i], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&sh->o_free[i], 4);  // epilogue warps
    for (int i = 0; i < 4; ++i) mbar_init(&sh->ml_ready[i], kSoftmaxWarps);
    sh->abort_flag = 0;
    sh->max_polls = max_polls;
    sh->n_items = 0xffffffffu;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(&sh->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  // The two groups' accumulators of an item.  At d = 64 they take 128 columns together and TMEM has
  // room for two items' worth: items alternate between them, so that the next item's first
  // O += P V need not wait until the epilogue has read this item's result.
  constexpr uint32_t kOBufs = D == 64 ? 2u : 1u;
  constexpr uint32_t kOGroup = D == 64 ? 64u : 128u;  // columns from group 0's accumulator to group 1's
  const uint32_t tmem_o = tmem + 256;
  auto o_of_item = [&](uint32_t n) { return tmem_o + (kOBufs == 2u ? 128u * (n & 1u) : 0u); };
  volatile int *abort_flag = &sh->abort_flag;
  const int item_step = (int)gridDim.x;

  if (warp == 8) {
    // ------------------------------------------------------------ producer
    if (lane < 4) {
      prefetch_tensormap(&maps.k[lane]);
      prefetch_tensormap(&maps.v[lane]);
    }
    if (lane == 4) prefetch_tensormap(&maps.q);
    bool ok = true;
    uint32_t g = 0, n = 0;   // rounds / non-empty items so far
    int armed_q = -1;        // non-empty item whose Q copy was armed last
    // Work is handed out in units of two items of one (b, h): query tile n_qt - 1 - j and query
    // tile j.  Under a causal mask a late tile has a long list and an early one a short list, so
    // units weigh about the same; and because consecutive units belong to the same (b, h), the
    // CTAs running at any time share a few heads' K and V, which then stay in L2.  The t-th item
    // of this CTA is half t & 1 of unit blockIdx.x + (t >> 1) * gridDim.x.
    const int n_half = (n_qt + 1) / 2, n_units = B * H * n_half;
    struct ItemRef {
      int bh, qt, rho0, rho1;  // rounds [rho0, rho1): loaded here, first read when the item begins
      int gr0, gr1;            // the list row's gathered rounds (equal: none)
      bool in_range, exists;   // !exists: no such item (the unit's halves coincide)
    };
    // (called for t = 0, 1, 2, ... in turn: the unit's (j, bh, h = bh % H) are stepped from one unit
    // of this CTA to the next instead of divided out of the unit number every time; this warp's
    // instruction stream is what short items wait for)
    int cur_u = (int)blockIdx.x, cur_j = cur_u % n_half, cur_bh = cur_u / n_half, cur_h = cur_bh % H;
    const int step_j = item_step % n_half, step_bh = item_step / n_half, step_h = step_bh % H;
    auto next_unit = [&](int &u, int &j, int &bh, int &h) {
      u += item_step;
      j += step_j;
      bh += step_bh;
      h += step_h;
      if (j >= n_half) {
        j -= n_half;
        ++bh;
        ++h;
      }
      if (h >= H) h -= H;
    };
    // kPairs: a unit's two query tiles come from the list's table, fetched one unit ahead of their use
    // (the address of the rounds' offsets depends on them)
    uint2 cur_pair = make_uint2(0u, 0u), ahead_pair = make_uint2(0u, 0u);
    auto fetch_pair_after = [&]() {  // the pair of the unit after the current one
      int u = cur_u, j = cur_j, bh = cur_bh, h = cur_h;
      next_unit(u, j, bh, h);
      if (u < n_units) ahead_pair = ldg_now_v2(gth.unit_qt + ((size_t)h * n_half + j) * 2);
    };
    if constexpr (kPairs) {
      if (cur_u < n_units) cur_pair = ldg_now_v2(gth.unit_qt + ((size_t)cur_h * n_half + cur_j) * 2);
      fetch_pair_after();
    }
    auto item_ref = [&](int t) {
      ItemRef it;
      if (t >= 2 && !(t & 1)) {  // the next unit
        next_unit(cur_u, cur_j, cur_bh, cur_h);
        if constexpr (kPairs) {
          cur_pair = ahead_pair;
          fetch_pair_after();
        }
      }
      const int u = cur_u;
      it.in_range = u < n_units;
      it.bh = 0, it.qt = 0, it.rho0 = 0, it.rho1 = 0, it.gr0 = 0, it.gr1 = 0, it.exists = false;
      if (it.in_range) {
        const int j = cur_j;
        it.bh = cur_bh;
        bool there = !(t & 1) || j != n_qt - 1 - j;
        if constexpr (kPairs) {
          it.qt = (t & 1) ? (int)cur_pair.y : (int)cur_pair.x;
          there = it.qt >= 0;
          if (!there) it.qt = 0;
        } else {
          it.qt = (t & 1) ? j : n_qt - 1 - j;
        }
        if (there) {
          const int lr = cur_h * n_qt + it.qt;
          it.rho0 = (int)ldg_now_u32(round_ptr + lr);
          it.rho1 = (int)ldg_now_u32(round_ptr + lr + 1);
          if constexpr (kGath) {
            it.gr0 = (int)ldg_now_u32(gth.ptr + lr);
            it.gr1 = (int)ldg_now_u32(gth.ptr + lr + 1);
          }
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
    // slot g % kMaxStages.  K may be overwritten once S = Q K^T of round g - kStages has completed
    // (k_empty), V once O += P V of that round has (v_empty).  The info slot last served round
    // g - kMaxStages, whose softmax must be over: with kStages == kMaxStages that is what v_empty
    // says; with a ring of two, S of round g - 2 could only be computed after O += P V of round
    // g - 4 was issued, i.e. after that round's softmax, so k_empty implies it.
    static_assert(C::kStages == kMaxStages || C::kStages == 2, "ring discipline");
    auto wait_free = [&](uint64_t *bar, uint32_t ph) {
      if (lane == 0) ok = wait_or_abort(bar, ph ^ 1u, abort_flag, err, max_polls);
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
    // Gathered round: lane l holds the keys k4 of the stage's rows 4l .. 4l+3, lanes 4q .. 4q+3 those of
    // slot q.  A slot whose 16 keys follow one another from a multiple of 8 on is one box (most slots of
    // a gathered schedule are of that kind); the other slots' rows are fetched one by one.  The copy
    // engine spends some 60 cycles on every copy whatever its size, so a row-by-row slot would cost it
    // sixteen times a box with four-row gathers; instead the whole warp copies such a slot in 16-byte
    // pieces (cp.async) to where the 128-byte swizzle puts them, and ties those copies to the stage's
    // barrier before that barrier gets the producer's own arrival.
    auto box_slots = [&](int4 k4, int ng) {  // bit q: slot q is a box
      const int before = __shfl_up_sync(0xffffffffu, k4.w, 1);
      const bool chained = k4.y == k4.x + 1 && k4.z == k4.x + 2 && k4.w == k4.x + 3 &&
                           ((lane & 3) == 0 ? (k4.x & 7) == 0 : k4.x == before + 1);
      uint32_t chain = __ballot_sync(0xffffffffu, chained);
      chain &= chain >> 1;
      chain &= chain >> 2;  // bit 4q: lanes 4q .. 4q+3 all chained
      uint32_t boxes = 0u;
#pragma unroll
      for (int q = 0; q < 8; ++q) boxes |= ((chain >> (4 * q)) & 1u) << q;
      return boxes & ((1u << ng) - 1u);
    };
    // keys of the gathered round being copied and of the one before (whose V copies come a round later)
    auto load_scattered = [&](unsigned char *stage, const uint16_t *src, uint64_t *bar, const int32_t *keys_s,
                              uint32_t slots, int bh) {
      constexpr int kChunks = D / 8;             // 16-byte pieces per key row
      constexpr int kRowsPerStep = 32 / kChunks; // rows the warp covers per step: lane -> (row, piece)
      const uint16_t *rows = src + (size_t)bh * gth.Lk * D;
      const int c = lane % kChunks, r0 = lane / kChunks, half = c >> 3;
      unsigned char *dst_lane = stage + half * C::kHalfStride;
      while (slots) {
        const int q = __ffs((int)slots) - 1;
        slots &= slots - 1u;
#pragma unroll
        for (int i = 0; i < 16 / kRowsPerStep; ++i) {
          const int R = 16 * q + r0 + kRowsPerStep * i;
          const int key = keys_s[R];
          unsigned char *dst = dst_lane + (kSplit ? (R >> 3) * 2048 + (R & 7) * 128 : R * 128) + (((c ^ R) & 7) << 4);
          cp_async16(dst, rows + (size_t)key * D + 8 * c);
        }
      }
      cp_async_arrive_on(bar);
    };
    // The box slots of a gathered round, runs of them that continue one another as one copy.
    auto load_boxes = [&](unsigned char *stage, const CUtensorMap *m4, uint64_t *bar, int4 k4, uint32_t boxes,
                          int bh) {
      const int row_q = __shfl_sync(0xffffffffu, k4.x, (lane & 7) * 4);  // lanes 0..7: first key of slot `lane`
      const int row_before = __shfl_up_sync(0xffffffffu, row_q, 1);
      const bool is_box = lane < 8 && ((boxes >> lane) & 1u);
      const bool after_box = lane > 0 && ((boxes >> (lane - 1)) & 1u);
      const bool head = is_box && (!after_box || row_q != row_before + 16);
      const uint32_t heads = __ballot_sync(0xffffffffu, head);
      const uint32_t stop = ((heads | ~boxes) >> (lane + 1)) & 0x7fu;
      const int run = head ? (stop ? __ffs((int)stop) : 8 - lane) : 0;
      load_run(stage, m4, bar, row_q, run, bh);
    };
    // which schedule an item follows
    auto use_gathered = [&](const ItemRef &it) {
      if constexpr (!kGath) return false;
      return it.gr1 > it.gr0;  // the list's builder decided where they pay
    };
    // V of a round is copied one round later than its K: K only needs S = Q K^T of the round that
    // used the stage before to be over, V needs that round's O += P V, which comes much later;
    // issued in round order, the V copy would hold back the next round's K.
    bool pv_valid = false, pv_gathered = false;
    uint32_t pv_boxes = 0u;
    int pv_kb = 0;
    int pv_st = 0, pv_ng = 0, pv_row = 0, pv_run = 0, pv_bh = 0;
    int4 pv_keys = make_int4(0, 0, 0, 0);
    uint32_t pv_ph = 0;
    auto issue_v = [&]() {
      if (C::kStages != kMaxStages) wait_free(&sh->v_empty[pv_st], pv_ph);
      if (!ok) return;
      if constexpr (kGath) {
        const uint32_t scattered = pv_gathered ? ((1u << pv_ng) - 1u) & ~pv_boxes : 0u;
        if (scattered)
          load_scattered(v_s + pv_st * C::kTileBytes, gth.V, &sh->v_full[pv_st], sh->keys[pv_kb], scattered, pv_bh);
        __syncwarp();
      }
      if (lane == 0)
        mbar_arrive_expect_tx(&sh->v_full[pv_st],
                              (uint32_t)(kGath && pv_gathered ? __popc(pv_boxes) : pv_ng) * 16u * D * 2u);
      __syncwarp();
      if (kGath && pv_gathered) {
        load_boxes(v_s + pv_st * C::kTileBytes, maps.v, &sh->v_full[pv_st], pv_keys, pv_boxes, pv_bh);
      } else {
        load_run(v_s + pv_st * C::kTileBytes, maps.v, &sh->v_full[pv_st], pv_row, pv_run, pv_bh);
      }
      pv_valid = false;
    };
    // the rounds of an item are looked up two items ahead: the loads of item t + 2 are issued when
    // item t begins and their results first touched when item t + 1 does
    ItemRef next = item_ref(0);
    ItemRef next2 = item_ref(1);
    // ... and the slot rows and info byte of its first round while the current item is under way
    int pf_t = -1, pf_row = -1;
    int4 pf_keys = make_int4(0, 0, 0, 0);
    uint32_t pf_info = 0u;
    // slot rows (lanes 0..7) or, for a gathered round, this lane's four keys, and the info byte
    auto fetch_round = [&](bool gathered, int rho, int &row, int4 &keys, uint32_t &info) {
      if (kGath && gathered) {
        const uint4 k = ldg_now_v4(gth.keys + (size_t)rho * kTile + 4 * lane);
        keys = make_int4((int)k.x, (int)k.y, (int)k.z, (int)k.w);
        info = ldg_now_u8(gth.info + rho);
      } else {
        row = lane < 8 ? (int)ldg_now_u32(round_rows + (size_t)rho * 8 + lane) : -1;
        info = ldg_now_u8(round_info + rho);
      }
    };
    for (int t = 0; next.in_range && ok; ++t) {
      const ItemRef cur = next;
      next = next2;
      next2 = item_ref(t + 2);
      if (!cur.exists) continue;
      const bool gathered = use_gathered(cur);
      const int bh = cur.bh, qt = cur.qt, rho0 = gathered ? cur.gr0 : cur.rho0;
      const int n_rounds = gathered ? cur.gr1 - cur.gr0 : cur.rho1 - cur.rho0;
      const uint32_t *bitmaps = gathered ? gth.bitmap : round_bitmap;
      if (n_rounds == 0) {
        // nothing kept in this query tile: its output rows are zero (nobody else sees the item)
        const int rows = min(kTile, Lq - qt * kTile);
        uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + (size_t)qt * kTile) * D);
        for (int x = lane; x < rows * (D / 8); x += 32) dst[x] = make_uint4(0u, 0u, 0u, 0u);
        continue;
      }
      // Q of this item into its buffer (free once the last S = Q K^T of item n - 2 has completed)
      const int qb = (int)(n & 1u);
      if (lane == 0) {
        ok = wait_or_abort(&sh->q_empty[qb], ((n >> 1) & 1u) ^ 1u, abort_flag, err, max_polls);
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
      // a round's rows or keys and its info byte are fetched one round ahead
      int next_row = pf_row;
      int4 next_keys = pf_keys;
      uint32_t next_info = pf_info;
      if (pf_t != t) fetch_round(gathered, rho0, next_row, next_keys, next_info);
      for (int v = 0; v < n_rounds && ok; ++v, ++g) {
        const int row = next_row;
        const int4 keys = next_keys;
        const uint32_t rinfo = next_info;
        if (v + 1 < n_rounds) {
          fetch_round(gathered, rho0 + v + 1, next_row, next_keys, next_info);
        } else if (next.exists && next.rho1 > next.rho0) {
          pf_t = t + 1;
          const bool g_next = use_gathered(next);
          fetch_round(g_next, g_next ? next.gr0 : next.rho0, pf_row, pf_keys, pf_info);
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
        const int si = (int)(g % kMaxStages);
        wait_free(&sh->k_empty[st], ph);
        if (ok && C::kStages == kMaxStages) wait_free(&sh->v_empty[st], ph);
        if (!ok) break;
        const bool skip = dbg_skip != 0 && g == 0;   // (test hook: this round's copies and arrivals are left out)
        uint32_t boxes = 0u;
        uint32_t bytes = (uint32_t)ng * 16u * D * 2u;
        const int kb = (int)(g & 1u);
        if constexpr (kGath) {
          if (gathered) {
            boxes = box_slots(keys, ng);
            bytes = (uint32_t)__popc(boxes) * 16u * D * 2u;
            const uint32_t scattered = ((1u << ng) - 1u) & ~boxes;
            if (scattered && !skip) {
              // (V of the round before last, which used this buffer, was issued a round ago)
              *reinterpret_cast<int4 *>(&sh->keys[kb][4 * lane]) = keys;
              __syncwarp();
              load_scattered(k_s + st * C::kTileBytes, gth.K, &sh->k_full[st], sh->keys[kb], scattered, bh);
            }
            __syncwarp();
          }
        }
        if (lane == 0 && !skip) {
          sh->info[si] = (uint32_t)ng | (v == 0 ? kInfoFirst : 0u) | (v + 1 == n_rounds ? kInfoLast : 0u) |
                         (full ? kInfoFull : 0u);
          sh->item_bh[si] = bh;
          sh->item_qt[si] = qt;
          mbar_arrive_expect_tx(&sh->k_full[st], bytes);
          if (full) {
            mbar_arrive(&sh->b_full[si]);
          } else {
            mbar_arrive_expect_tx(&sh->b_full[si], kBitmapWords * 4);
            bulk_load(&sh->bitmap[si][0][0], bitmaps + (size_t)(rho0 + v) * kBitmapWords, kBitmapWords * 4,
                      &sh->b_full[si]);
          }
        }
        __syncwarp();
        if (!skip) {
          if (kGath && gathered) {
            load_boxes(k_s + st * C::kTileBytes, maps.k, &sh->k_full[st], keys, boxes, bh);
          } else {
            load_run(k_s + st * C::kTileBytes, maps.k, &sh->k_full[st], row, run, bh);
          }
        }
        if (pv_valid) issue_v();
        if (!ok) break;
        pv_valid = !skip;
        pv_gathered = gathered;
        pv_st = st, pv_ph = ph, pv_ng = ng, pv_row = row, pv_run = run, pv_bh = bh, pv_keys = keys, pv_boxes = boxes;
        pv_kb = kb;
      }
      ++n;
    }
    if (ok && pv_valid) issue_v();
    // no more work: one more stage carries the stop word
    if (ok) {
      const int st = (int)(g % C::kStages);
      const uint32_t ph = (g / C::kStages) & 1u;
      wait_free(&sh->k_empty[st], ph);
      if (ok && C::kStages == kMaxStages) wait_free(&sh->v_empty[st], ph);
      if (ok && lane == 0) {
        sh->info[g % kMaxStages] = kInfoStop;
        mbar_arrive(&sh->k_full[st]);
        mbar_arrive(&sh->b_full[g % kMaxStages]);
      }
    }
    if (lane == 0 && *abort_flag) {
      // winding down: wait (bounded) for the copies armed most recently
      if (armed_q >= 0) mbar_wait(&sh->q_full[armed_q & 1], ((uint32_t)armed_q >> 1) & 1u, 1u << 16);
      for (uint32_t a = g > (uint32_t)C::kStages ? g - C::kStages : 0; a <= g; ++a) {
        if (dbg_skip != 0 && a == 0) continue;  // never armed
        mbar_wait(&sh->k_full[a % C::kStages], (a / C::kStages) & 1u, 1u << 16);
        mbar_wait(&sh->v_full[a % C::kStages], (a / C::kStages) & 1u, 1u << 16);
        mbar_wait(&sh->b_full[a % kMaxStages], (a / kMaxStages) & 1u, 1u << 16);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ issuer of S = Q K^T
    // The whole warp walks the rounds in lockstep (one lane polls the barriers, another, elected
    // one issues the tcgen05 instructions; the state is warp-uniform).
    const uint32_t q_addr = smem_u32(q_s), k_addr = smem_u32(k_s);
    bool ok = true;
    uint32_t n = 0;  // non-empty items started so far
    for (uint32_t g = 0; ok; ++g) {
      const int st = (int)(g % C::kStages);
      const uint32_t sb = g & 1u;
      ok = warp_wait<31>(&sh->k_full[st], (g / C::kStages) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      const uint32_t info = sh->info[g % kMaxStages];
      if (info & kInfoStop) break;
      const int ng = (int)(info & kInfoSlots);
      const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
      const int qb = (int)(n & 1u);
      if (first) ok = warp_wait<31>(&sh->q_full[qb], (n >> 1) & 1u, lane, abort_flag, err, max_polls);
      // S[sb] still holds P of round g - 2 until that round's O += P V (issued by another warp) has
      // completed
      if (ok && g >= 2) ok = warp_wait<31>(&sh->pv_done[sb], ((g >> 1) - 1u) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (kGath) fence_proxy_async_smem();  // rows of a gathered round may come from plain asynchronous copies
      // N = 16 ng, D/16 steps of K = 16 (32 bytes inside the swizzled rows)
      if (elect_one()) {
        const uint32_t idesc_qk = idesc_bf16_f32(128, 16 * ng, false, false, kF16);
        const uint32_t q_buf = q_addr + qb * C::kTileBytes, k_stage = k_addr + st * C::kTileBytes;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int sub = ks / 4, off = (ks % 4) * 32;
          mma_ss(tmem + 128u * sb, smem_desc_sw128(q_buf + sub * kSubBytes + off, 16, 1024),
                 smem_desc_sw128(k_stage + sub * C::kHalfStride + off, 16, C::kSbo), idesc_qk, ks > 0);
        }
        mma_commit(&sh->k_empty[st]);
        if (last) mma_commit(&sh->q_empty[qb]);
        mma_commit(&sh->s_full[sb]);
      }
      __syncwarp();
      if (last) ++n;
    }
  } else if (warp == 10) {
    // ------------------------------------------------------------ issuer of O += P V
    constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true, kF16);
    const uint32_t v_addr = smem_u32(v_s);
    bool ok = true;
    uint32_t n = 0;                          // non-empty items started so far
    uint32_t started0 = 0u, started1 = 0u;  // the item's O_0 / O_1 holds a partial result already
    for (uint32_t g = 0; ok; ++g) {
      const int st = (int)(g % C::kStages);
      const uint32_t sb = g & 1u;
      ok = warp_wait<31>(&sh->b_full[g % kMaxStages], (g / kMaxStages) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      const uint32_t info = sh->info[g % kMaxStages];
      if (info & kInfoStop) break;
      const int ng = (int)(info & kInfoSlots);
      const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
      // (what is ready early first; P, which the softmax has just finished, last)
      ok = warp_wait<31>(&sh->v_full[st], (g / C::kStages) & 1u, lane, abort_flag, err, max_polls);
      // the first round of an item overwrites O: the epilogue of the previous item must have read it
      if (ok && first && n >= kOBufs)
        ok = warp_wait<31>(&sh->o_free[kOBufs == 2u ? (n & 1u) : 0u], ((n / kOBufs) - 1u) & 1u, lane, abort_flag, err, max_polls);
      if (ok) ok = warp_wait<31>(&sh->p_full[sb], (g >> 1) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (kGath) fence_proxy_async_smem();  // rows of a gathered round may come from plain asynchronous copies
      // One K step of 16 keys per slot.  P (bf16) of a 32-column chunk is written over the first
      // 16 columns of that chunk of S (each group stays inside its own chunks), so slot q's
      // eight columns of P start at column 32 (q / 2) + 8 (q % 2).
      // Slots 0, 1, 4, 5 (chunks 0 and 2) belong to softmax group 0 and add to O_0, the others to
      // O_1; a group's first step of an item overwrites its accumulator.
      if (first) started0 = started1 = 0u;
      if (elect_one()) {
        const uint32_t v_stage = v_addr + st * C::kTileBytes;
        const uint32_t p_base = tmem + 128u * sb;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          if (ks < ng) {
            const int grp = (ks >> 1) & 1;
            const uint32_t acc = ks == 0 ? started0 : ks == 2 ? started1 : 1u;  // slots 0 / 2 open their group
            mma_ts(o_of_item(n) + kOGroup * grp, p_base + 32 * (ks >> 1) + 8 * (ks & 1),
                   smem_desc_sw128(v_stage + ks * C::kSlotStride, C::kHalfStride, C::kSbo), idesc_pv, acc);
          }
        }
        mma_commit(&sh->v_empty[st]);
        mma_commit(&sh->pv_done[sb]);
        if (last) mma_commit(&sh->o_done[kOBufs == 2u ? (n & 1u) : 0u]);
      }
      __syncwarp();
      started0 = 1u;
      if (ng > 2) started1 = 1u;
      if (last) ++n;
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------ softmax
    const int grp = warp >> 2;               // softmax group: chunks grp and grp + 2 of every round
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    uint32_t tmem_og = tmem_o + kOGroup * grp;  // this group's output accumulator (of the current item)
    const float ref_slack = 8.f / scale_log2;
    bool ok = true;
    uint32_t n = 0;
    float m = -CUDART_INF_F, l = 0.f;       // this group's exponent reference and running sum of weights
    bool o_started = false;                  // an earlier round of the item added to this group's accumulator
    int cur_bh = 0, cur_qt = 0;
    for (uint32_t g = 0; ok; ++g) {
      const int st = (int)(g % kMaxStages);  // info / bitmap slot of the round
      const uint32_t sb = g & 1u;
      const uint32_t tmem_s = tmem + 128u * sb;
      ok = warp_wait(&sh->b_full[st], (g / kMaxStages) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      const uint32_t info = sh->info[st];
      if (info & kInfoStop) break;
      const int ng = (int)(info & kInfoSlots);
      const bool first = (info & kInfoFirst) != 0u, last = (info & kInfoLast) != 0u;
      const bool tile_full = (info & kInfoFull) != 0u;
      if (first) {
        cur_bh = sh->item_bh[st];
        cur_qt = sh->item_qt[st];
        m = -CUDART_INF_F;
        l = 0.f;
        o_started = false;
        tmem_og = o_of_item(n) + kOGroup * grp;
      }
      // this group's 32-column chunks of the round: grp and grp + 2, as far as the round reaches
      const int n_mine = ((ng + 1) >> 1) > grp + 2 ? 2 : ((ng + 1) >> 1) > grp ? 1 : 0;
      float alpha = 1.f;
      if (n_mine > 0) {
      uint32_t w0 = 0xffffffffu, w1 = 0xffffffffu;   // bitmap words of chunks grp and grp + 2
      if (!tile_full) {
        const uint32_t *brow = &sh->bitmap[st][r][0];
        w0 = brow[grp];
        w1 = brow[grp + 2];
      }
      ok = warp_wait(&sh->s_full[sb], (g >> 1) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      tc_fence_after_sync();
      // straight-line: both chunks always (a chunk the round does not reach holds stale scores whose
      // bitmap bits are zero), masked or not
      uint32_t xs[64];
      tmem_ld32(tmem_s + lane_addr + 32 * grp, &xs[0]);
      tmem_ld32(tmem_s + lane_addr + 32 * (grp + 2), &xs[32]);
      tmem_wait_ld();
      if (!tile_full) {
#pragma unroll
        for (int e = 0; e < 32; ++e) xs[e] = ((w0 >> e) & 1u) ? xs[e] : 0xff800000u;
#pragma unroll
        for (int e = 0; e < 32; ++e) xs[32 + e] = ((w1 >> e) & 1u) ? xs[32 + e] : 0xff800000u;
      }
      float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F, mx2 = -CUDART_INF_F, mx3 = -CUDART_INF_F;
#pragma unroll
      for (int e = 0; e < 64; e += 8) {
        mx0 = fmax3(mx0, __uint_as_float(xs[e]), __uint_as_float(xs[e + 1]));
        mx1 = fmax3(mx1, __uint_as_float(xs[e + 2]), __uint_as_float(xs[e + 3]));
        mx2 = fmax3(mx2, __uint_as_float(xs[e + 4]), __uint_as_float(xs[e + 5]));
        mx3 = fmax3(mx3, __uint_as_float(xs[e + 6]), __uint_as_float(xs[e + 7]));
      }
      const float tile_max = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      // The exponent's reference m follows the running maximum lazily: it moves only when
      // the maximum outgrows it by more than 2^8 in the exp2 domain (weights stay <= 256,
      // well inside bf16 and fp32 range), which saves most rescales of O.  O / l does not
      // depend on the reference.
      const bool move = tile_max > m + ref_slack;   // also true for the first kept entry (m = -inf)
      const float m_new = move ? tile_max : m;
      const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
      alpha = move ? ex2_approx((m - m_safe) * scale_log2) : 1.f;  // 0 when m was -inf
      const float neg_mc = -m_safe * scale_log2;
      m = m_new;
      // Rescale the group's running output where the reference moved.  O += P V of the previous
      // round may still be running (this round's S was computed ahead of it): wait for it first.
      if (o_started && __any_sync(0xffffffffu, alpha != 1.f)) {
        ok = warp_wait(&sh->pv_done[(g - 1u) & 1u], ((g - 1u) >> 1) & 1u, lane, abort_flag, err, max_polls);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tmem_og + lane_addr + 32 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st32(tmem_og + lane_addr + 32 * c, o);
        }
      }
      // pass 2: P = exp2(c*S - c*m); pruned entries are -inf by now and give exactly 0; bf16 P over
      // the first half of the chunk's columns of S
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float p0 = ex2_approx(fmaf(__uint_as_float(xs[32 * c + 2 * e]), scale_log2, neg_mc));
          const float p1 = ex2_approx(fmaf(__uint_as_float(xs[32 * c + 2 * e + 1]), scale_log2, neg_mc));
          pk[e] = pack16x2<kF16>(p0, p1);
          const float2 pr = unpack16x2<kF16>(pk[e]);
          sum0 += pr.x;
          sum1 += pr.y;
        }
        tmem_st16(tmem_s + lane_addr + 32 * (grp + 2 * c), pk);
      }
      l = l * alpha + (sum0 + sum1);
      o_started = true;
      tmem_wait_st();
      }  // n_mine > 0
      // one arrival per warp (32 lanes arriving one by one would take hundreds of cycles)
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->p_full[sb]);
      if (!last) continue;
      // The item's rounds are over for this group: it hands (m, l) to the epilogue warps and goes on
      // with the next item; the slot of the hand-over ring was read by the epilogue of item n - 4,
      // which is over (this item's S needed O += P V of item n - 2, that the epilogue of item n - 3).
      sh->ml[n & 3u][grp][r] = make_float2(m, l);
      if (threadIdx.x == 0) {
        sh->ml_bh[n & 3u] = cur_bh;
        sh->ml_qt[n & 3u] = cur_qt;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ml_ready[n & 3u]);
      ++n;
    }
    // No more items: tell the epilogue warps.  The end is signalled outside the hand-over ring (a
    // word of its own says how many items there were; the barrier of the slot the next item would
    // have used only wakes the epilogue warps up), so that no slot is written that an epilogue warp
    // may still be reading: with short items and two sets of accumulators the slot's previous owner,
    // item n - 4, need not have been read by now.
    if (ok) {
      if (threadIdx.x == 0) sh->n_items = n;
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->ml_ready[n & 3u]);
    }
  } else if (warp >= 11) {
    // ------------------------------------------------------------ epilogue
    // Per item: merge the two groups' accumulators and write O / l, rounded once to bf16.
    const int r = (warp & 3) * 32 + lane;    // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    bool ok = true;
    for (uint32_t n = 0; ok; ++n) {
      ok = warp_wait(&sh->ml_ready[n & 3u], (n >> 2) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      if (n >= *reinterpret_cast<volatile uint32_t *>(&sh->n_items)) break;
      const int item_qt = sh->ml_qt[n & 3u], item_bh = sh->ml_bh[n & 3u];
      const float2 g0 = sh->ml[n & 3u][0][r], g1 = sh->ml[n & 3u][1][r];
      const int i = item_qt * kTile + r;
      uint16_t *orow = O + ((size_t)item_bh * Lq + i) * D;
      const float m_tot = fmaxf(g0.x, g1.x);
      // weight of a partial result; 0 for a group that saw no kept entry of this row (m = -inf),
      // whose accumulator is then never read into the sum (it may hold a previous item's data)
      const float a0 = g0.x == -CUDART_INF_F ? 0.f : ex2_approx((g0.x - m_tot) * scale_log2);
      const float a1 = g1.x == -CUDART_INF_F ? 0.f : ex2_approx((g1.x - m_tot) * scale_log2);
      const float l_tot = g0.y * a0 + g1.y * a1;
      const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
      const float f0 = a0 * inv, f1 = a1 * inv;
      ok = warp_wait(&sh->o_done[kOBufs == 2u ? (n & 1u) : 0u], (n / kOBufs) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) break;
      tc_fence_after_sync();
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o0[32], o1[32];
        tmem_ld32(o_of_item(n) + lane_addr + 32 * c, o0);
        tmem_ld32(o_of_item(n) + kOGroup + lane_addr + 32 * c, o1);
        tmem_wait_ld();
        if (c == D / 32 - 1) {  // this thread's rows of O are in registers: the next item may overwrite them
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh->o_free[kOBufs == 2u ? (n & 1u) : 0u]);
        }
        if (i < Lq) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // a row without kept entries has l = 0 and P = 0 throughout: write exact zeros
              const int j = 8 * q + 2 * e;
              const float x0 = (f0 > 0.f ? __uint_as_float(o0[j]) * f0 : 0.f) + (f1 > 0.f ? __uint_as_float(o1[j]) * f1 : 0.f);
              const float x1 = (f0 > 0.f ? __uint_as_float(o0[j + 1]) * f0 : 0.f) +
                               (f1 > 0.f ? __uint_as_float(o1[j + 1]) * f1 : 0.f);
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
  if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

template <int D, bool kSplit, bool kF16, bool kGath, bool kPairs>
cudaError_t launch_kernel(const FwdMaps &maps, const void *K, const void *V, void *O, const ap_tiles &t, int B, int H,
                          int Lq, int Lk, const DebugKnobs &dbg, float scale, unsigned *err, cudaStream_t s) {
  using C = Cfg<D, kSplit>;
  static_assert(sizeof(Shared) <= 18 * 1024, "shared bookkeeping outgrew its reservation");
  static_assert(C::kStages <= kMaxStages, "ring deeper than its barriers");
  static_assert(C::kSmemBytes > 114 * 1024 && C::kSmemBytes <= 227 * 1024, "one CTA per SM, within the limit");
  auto kern = fwd_tc_kernel<D, kSplit, kF16, kGath, kPairs>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int n_units = B * H * ((t.n_qt + 1) / 2);  // pairs of query tiles, see the producer
  const float scale_log2 = scale * 1.4426950408889634f;
  Gathered gth = {nullptr, nullptr, nullptr, nullptr, static_cast<const uint16_t *>(K), static_cast<const uint16_t *>(V),
                  Lk, dbg.schedule, kPairs ? t.unit_qt : nullptr};
  if (kGath) gth.ptr = t.ground_ptr, gth.keys = t.ground_keys, gth.info = t.ground_info, gth.bitmap = t.ground_bitmap;
  // the test hook runs on one CTA only (a tiny grid is all it is meant for)
  kern<<<dbg.skip_arrive ? 1 : (n_units < sms ? n_units : sms), kThreads, C::kSmemBytes, s>>>(
      maps, static_cast<uint16_t *>(O), t.round_ptr, t.round_rows, t.round_info, t.round_bitmap, gth, B, H, Lq,
      t.n_qt, scale_log2, err, dbg.max_polls, dbg.skip_arrive);
  count_launches(1);
  return cudaGetLastError();
}

// Lists that carry a gathered schedule get the instantiation that can follow it.
template <int D, bool kSplit, bool kF16>
cudaError_t launch(const FwdMaps &maps, const void *K, const void *V, void *O, const ap_tiles &t, int B, int H, int Lq,
                   int Lk, bool, float scale, unsigned *err, cudaStream_t s) {
  const DebugKnobs dbg = debug_knobs();
  if (t.ground_ptr != nullptr && dbg.schedule != 1)
    return launch_kernel<D, kSplit, kF16, true, false>(maps, K, V, O, t, B, H, Lq, Lk, dbg, scale, err, s);
  if (t.unit_qt != nullptr && !dbg.skip_arrive)
    return launch_kernel<D, kSplit, kF16, false, true>(maps, K, V, O, t, B, H, Lq, Lk, dbg, scale, err, s);
  return launch_kernel<D, kSplit, kF16, false, false>(maps, K, V, O, t, B, H, Lq, Lk, dbg, scale, err, s);
}

}  // namespace

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
  const bool gm = t.ground_ptr != nullptr;
  if (f16) {
    if (d == 64) return launch<64, false, true>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s);
    return split ? launch<128, true, true>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s)
                 : launch<128, false, true>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s);
  }
  if (d == 64) return launch<64, false, false>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s);
  return split ? launch<128, true, false>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s)
               : launch<128, false, false>(maps, K, V, O, t, B, H, Lq, Lk, gm, scale, err, s);
}

}  // namespace ap
