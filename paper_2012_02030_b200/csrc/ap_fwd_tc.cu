// Masked attention of Section 3.2 for bf16 tensors on the tcgen05 tensor cores.
//
// Persistent kernel, one CTA per SM.  A work item is one (b, h, query tile of 128 rows); CTA c
// takes items c, c + gridDim.x, ... (heavy items first).  The CTA walks the tile list of the
// item's (h, qt) row in ROUNDS.  A round is either one stored key tile, or - when the list is long
// and its tiles are mostly empty - one PACKED tile: each stored tile's bitmap is cut into eight
// groups of 16 key columns, the tile list's group summary says which groups hold a kept entry,
// and up to eight such groups, taken in list order from one or several key tiles, form a round of
// 16..128 key columns.  A skipped group holds no kept entry, so leaving it out is exact.
//   S  = Q K_round^T         tcgen05.mma, N = 16 * groups, fp32 accumulator in TMEM
//   P  = exp2(c*S - c*m)     one thread per query row reads its S row from TMEM, replaces pruned
//                            entries by -inf (the bitmap decides, exactly), keeps the running
//                            reference m and sum l of an online softmax, rescales O when m moved,
//                            and writes P as bf16 over S in TMEM
//   O += P V_round           tcgen05.mma, A = P from TMEM, B = V (MN-major), one K step of 16 keys
//                            per group
// and finally O / l is written (zeros for rows that never saw a kept entry).
//
// Pipeline.  S is double-buffered in TMEM and the MMA thread issues S(g+1) = Q K^T before
// O += P(g) V, so the softmax threads find the next S ready when they finish a round and the
// tensor pipe works on one round while the CUDA cores work on another.  The producer warp runs
// ahead: it plans the next item (prefix sum over the list's group summaries), loads its Q into
// the second Q buffer and keeps the K/V ring full across item boundaries, which hides the
// latency of an item's first loads behind the previous item's last rounds.
//
// Warp roles (192 threads): warps 0-3 softmax + epilogue (thread = query row = TMEM lane),
// warp 4 producer (plan, TMA), warp 5 MMA issuer and TMEM owner.  TMEM (512 columns): S[0] at
// column 0, S[1] at 128, O at 256.  Every wait is bounded; a wait that expires raises the
// device status word and the CTA winds down.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 192;
constexpr int kSubBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled sub-tile
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kMaxPlanTiles = 128;    // longest list whose groups are packed (longer ones go tile by tile)
constexpr int kMaxSlots = 8 * kMaxPlanTiles;
constexpr int kMinTilesToPack = 3;    // shorter lists are processed tile by tile
constexpr int kReadersPerItem = 5;    // threads/warps that read an item's plan: MMA thread + 4 softmax warps

// Shared-memory layout of a K or V stage.  Rows are the round's keys, a row's d elements are cut
// into halves of 64 (128 bytes, the swizzle span).
//   kSplit = false: [half][row / 8][8 rows][128 B]   one TMA box per half (3-D tensor map)
//   kSplit = true:  [row / 8][half][8 rows][128 B]   d = 128 only: one box brings both halves (5-D map)
template <int D, bool kSplit>
struct Cfg {
  static_assert(!kSplit || D == 128, "the split layout is for d = 128");
  static constexpr int kSub = D / 64;                 // halves per row
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kStages = D == 64 ? 4 : 2;     // K and V ring depth
  static constexpr int kKOffset = 2 * kTileBytes;     // after the two Q buffers
  static constexpr int kVOffset = kKOffset + kStages * kTileBytes;
  static constexpr int kBarOffset = kVOffset + kStages * kTileBytes;
  static constexpr int kSmemBytes = kBarOffset + 14 * 1024 + 1024;  // + barriers/plans + alignment slack
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

// What the producer publishes per item.  In a packed item slot s (s = 0, 1, ... in list order) is
// one non-empty group of 16 key columns and round v consists of slots [8v, 8v + 8).
struct ItemPlan {
  int32_t t_begin, n_tiles;         // the item's part of the tile list (n_tiles == 0: nothing kept)
  uint32_t packing;                 // 1: rounds are packed tiles, 0: rounds are list tiles
  uint32_t n_slots;
  uint8_t partial[kMaxPlanTiles];   // round v holds a slot of a tile that is not fully kept
  alignas(16) uint16_t tg[kMaxSlots];   // bit 15: tile flagged fully kept; bits 3..14: list index relative
                                        // to t_begin; bits 0..2: group
  alignas(16) int32_t row[kMaxSlots];   // first key row of the slot
};

struct Shared {
  uint64_t item_ready[2];            // producer -> MMA thread and softmax: plan[i] is valid
  uint64_t q_full[2], q_empty[2];
  uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
  uint64_t s_full[2], p_full[2];     // per S buffer
  uint64_t pv_done;                  // O += P V of a round has completed
  uint64_t o_done, o_free;           // per item: O complete / O read out by the epilogue
  uint32_t tmem_base;
  int abort_flag;
  int readers_done;                  // counts kReadersPerItem per item once its plan is no longer read
  int pad;
  ItemPlan plan[2];
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait that also gives up as soon as another thread of the CTA has.
__device__ __noinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                              unsigned *err) {
  for (uint32_t i = 0; i < kMaxPolls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 64) __nanosleep(64);
  }
  *abort_flag = 1;
  atomicOr(err, kDevErrTimeout);
  return false;
}

// Bounded wait until a shared counter reaches `target`.
__device__ __noinline__ bool wait_count_or_abort(volatile int *counter, int target, volatile int *abort_flag,
                                                    unsigned *err) {
  for (uint32_t i = 0; i < kMaxPolls; ++i) {
    if (*counter >= target) {
      __threadfence_block();
      return true;
    }
    if (*abort_flag) return false;
    if (i > 16) __nanosleep(64);
  }
  *abort_flag = 1;
  atomicOr(err, kDevErrTimeout);
  return false;
}

// kCanPack = false compiles the tile-by-tile rounds only (no list of the launch is long enough to pack).
template <int D, bool kCanPack, bool kSplit>
__global__ void __launch_bounds__(kThreads, 1)
fwd_tc_kernel(const __grid_constant__ FwdMaps maps, __nv_bfloat16 *__restrict__ O,
              const int32_t *__restrict__ row_ptr, const int32_t *__restrict__ col_idx,
              const uint8_t *__restrict__ flags, const uint32_t *__restrict__ bitmap,
              const uint8_t *__restrict__ groups, int B, int H, int Lq, int n_qt, int n_items,
              float scale_log2, unsigned *err) {
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
      mbar_init(&sh->item_ready[i], 1);
      mbar_init(&sh->q_full[i], 1);
      mbar_init(&sh->q_empty[i], 1);
      mbar_init(&sh->s_full[i], 1);
      mbar_init(&sh->p_full[i], 128);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&sh->k_full[s], 1);
      mbar_init(&sh->k_empty[s], 1);
      mbar_init(&sh->v_full[s], 1);
      mbar_init(&sh->v_empty[s], 1);
    }
    mbar_init(&sh->pv_done, 1);
    mbar_init(&sh->o_done, 1);
    mbar_init(&sh->o_free, 128);
    sh->abort_flag = 0;
    sh->readers_done = 0;
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(&sh->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sh->tmem_base;
  const uint32_t tmem_o = tmem + 256;
  volatile int *abort_flag = &sh->abort_flag;
  const int item_step = (int)gridDim.x;

  // Items are numbered so that heavy (late, under a causal mask) query tiles come first and b runs
  // fastest, so that CTAs working at the same time share tile lists and bitmaps in L2.
  auto list_row_of = [&](int item) { return ((item / B) % H) * n_qt + (n_qt - 1 - item / (B * H)); };

  if (warp == 4) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&maps.q);
      prefetch_tensormap(&maps.k[3]);
      prefetch_tensormap(&maps.v[3]);
    }
    if (kCanPack && lane < 3) {
      prefetch_tensormap(&maps.k[lane]);
      prefetch_tensormap(&maps.v[lane]);
    }
    bool ok = true;
    uint32_t g = 0, n = 0;   // rounds / non-empty items so far
    int armed_q = -1;        // non-empty item whose Q copy was armed last
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
    // the list row of an item is fetched one item ahead
    int nb = 0, ne = 0;
    if ((int)blockIdx.x < n_items) {
      const int lr = list_row_of((int)blockIdx.x);
      nb = row_ptr[lr];
      ne = row_ptr[lr + 1];
    }
    int seq = 0;
    for (int item = (int)blockIdx.x; item < n_items && ok; item += item_step, ++seq) {
      const int bh = (item % B) * H + (item / B) % H;
      const int qt = n_qt - 1 - item / (B * H);
      const int t_begin = nb, n_tiles = ne - nb;
      if (item + item_step < n_items) {
        const int lr = list_row_of(item + item_step);
        nb = row_ptr[lr];
        ne = row_ptr[lr + 1];
      }
      ItemPlan *pl = &sh->plan[seq & 1];
      // the plan buffer is free once everybody has finished reading the plan of item seq - 2
      if (seq >= 2) {
        if (lane == 0) ok = wait_count_or_abort(&sh->readers_done, kReadersPerItem * (seq - 1), abort_flag, err);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
      // The plan: every lane takes one list tile per pass, reads its group summary, and a prefix
      // sum over the lanes gives each tile's first slot.  Packing pays when it saves enough
      // rounds over going tile by tile.
      bool packing = false;
      uint32_t n_slots = 0;
      if (kCanPack && n_tiles >= kMinTilesToPack && n_tiles <= kMaxPlanTiles) {
        reinterpret_cast<uint32_t *>(pl->partial)[lane] = 0u;
        static_assert(kMaxPlanTiles == 128, "one 32-bit word of `partial` per lane");
        __syncwarp();
        int carry = 0;
        for (int base = 0; base < n_tiles; base += 32) {
          const int t = base + lane;
          uint32_t gm = 0u;
          int kt = 0;
          bool full = false;
          if (t < n_tiles) {
            full = flags[t_begin + t] & 1;
            gm = groups[t_begin + t];
            kt = col_idx[t_begin + t];
            if (full) gm = 0xffu;
          }
          const int cnt = __popc(gm);
          int incl = cnt;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
          }
          int s = carry + incl - cnt;
          while (gm) {
            const int grp = __ffs((int)gm) - 1;
            gm &= gm - 1u;
            pl->tg[s] = (uint16_t)((full ? 0x8000u : 0u) | ((uint32_t)t << 3) | (uint32_t)grp);
            pl->row[s] = kt * kTile + 16 * grp;
            if (!full) pl->partial[s >> 3] = 1;
            ++s;
          }
          carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        n_slots = (uint32_t)carry;
        const uint32_t n_packed = (n_slots + 7u) / 8u;
        packing = n_slots > 0u && 4u * n_packed <= 3u * (uint32_t)n_tiles;
      }
      __syncwarp();
      if (lane == 0) {
        pl->t_begin = t_begin;
        pl->n_tiles = n_tiles;
        pl->packing = packing ? 1u : 0u;
        pl->n_slots = n_slots;
        mbar_arrive(&sh->item_ready[seq & 1]);
      }
      if (n_tiles <= 0) continue;
      // Q of this item into its buffer (free once the last S = Q K^T of item n - 2 has completed)
      const int qb = (int)(n & 1u);
      if (lane == 0) {
        ok = wait_or_abort(&sh->q_empty[qb], ((n >> 1) & 1u) ^ 1u, abort_flag, err);
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
      const uint32_t n_rounds = packing ? (n_slots + 7u) / 8u : (uint32_t)n_tiles;
      int kt_next = packing ? 0 : col_idx[t_begin];
      for (uint32_t v = 0; v < n_rounds && ok; ++v, ++g) {
        const int st = (int)(g % C::kStages);
        const uint32_t ph = (g / C::kStages) & 1u;
        unsigned char *kd = k_s + st * C::kTileBytes, *vd = v_s + st * C::kTileBytes;
        if (!packing) {
          // one list tile: whole-tile boxes, one lane
          const int kt = kt_next;
          if ((int)v + 1 < n_tiles) kt_next = col_idx[t_begin + v + 1];
          if (lane == 0) {
            ok = wait_or_abort(&sh->k_empty[st], ph ^ 1u, abort_flag, err);
            if (ok) {
              mbar_arrive_expect_tx(&sh->k_full[st], C::kTileBytes);
              load_piece(kd, &maps.k[3], &sh->k_full[st], 0, kt * kTile, bh);
              ok = wait_or_abort(&sh->v_empty[st], ph ^ 1u, abort_flag, err);
            }
            if (ok) {
              mbar_arrive_expect_tx(&sh->v_full[st], C::kTileBytes);
              load_piece(vd, &maps.v[3], &sh->v_full[st], 0, kt * kTile, bh);
            }
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          continue;
        }
        // packed round: slots whose key rows follow one another form a run; the lane of a run's
        // first slot copies it (K, then V) in pieces of 8, 4, 2 or 1 slots
        const int ng = min(8, (int)(n_slots - 8u * v));
        const int row = lane < ng ? pl->row[8u * v + lane] : 0;
        const int row_before = __shfl_up_sync(0xffffffffu, row, 1);
        const bool head = lane < ng && (lane == 0 || row != row_before + 16);
        const uint32_t heads = __ballot_sync(0xffffffffu, head);
        const uint32_t later = lane < 31 ? heads >> (lane + 1) : 0u;
        const int run = head ? (later ? __ffs((int)later) : ng - lane) : 0;  // slots in this lane's run
        auto load_run = [&](unsigned char *stage, const CUtensorMap *m4, uint64_t *bar) {
          int q = lane, r = row, left = run;
          while (left > 0) {
            const int lg = left >= 8 ? 3 : left >= 4 ? 2 : left >= 2 ? 1 : 0;
            load_piece(stage, m4 + lg, bar, q, r, bh);
            q += 1 << lg;
            r += 16 << lg;
            left -= 1 << lg;
          }
        };
        const uint32_t bytes = (uint32_t)ng * 16u * D * 2u;
        if (lane == 0) {
          ok = wait_or_abort(&sh->k_empty[st], ph ^ 1u, abort_flag, err);
          if (ok) mbar_arrive_expect_tx(&sh->k_full[st], bytes);
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        load_run(kd, maps.k, &sh->k_full[st]);
        if (lane == 0) {
          ok = wait_or_abort(&sh->v_empty[st], ph ^ 1u, abort_flag, err);
          if (ok) mbar_arrive_expect_tx(&sh->v_full[st], bytes);
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        load_run(vd, maps.v, &sh->v_full[st]);
      }
      ++n;
    }
    if (lane == 0 && *abort_flag) {
      // winding down: wait (bounded) for the copies armed most recently.  A barrier whose copy was
      // armed but not waited for by anybody completes its phase; one that was not armed fails the
      // bounded wait quickly enough (the polls are not slept through).
      if (armed_q >= 0) mbar_wait(&sh->q_full[armed_q & 1], ((uint32_t)armed_q >> 1) & 1u, 1u << 16);
      for (uint32_t a = g > (uint32_t)C::kStages ? g - C::kStages : 0; a < g; ++a) {
        mbar_wait(&sh->k_full[a % C::kStages], (a / C::kStages) & 1u, 1u << 16);
        mbar_wait(&sh->v_full[a % C::kStages], (a / C::kStages) & 1u, 1u << 16);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
      bool ok = true;
      uint32_t g = 0, n = 0;
      // O += P V of the round before the current one is issued after the current S = Q K^T
      bool pending = false;
      uint32_t pend_g = 0, pend_n = 0;
      int pend_ng = 0;
      bool pend_first = false, pend_last = false;
      auto issue_pv = [&]() {
        const uint32_t sb = pend_g & 1u;
        const int st = (int)(pend_g % C::kStages);
        ok = wait_or_abort(&sh->p_full[sb], (pend_g >> 1) & 1u, abort_flag, err);
        if (ok) ok = wait_or_abort(&sh->v_full[st], (pend_g / C::kStages) & 1u, abort_flag, err);
        // the first round of an item overwrites O: the epilogue of the previous item must have read it
        if (ok && pend_first && pend_n > 0) ok = wait_or_abort(&sh->o_free, (pend_n - 1u) & 1u, abort_flag, err);
        if (!ok) return;
        tc_fence_after_sync();
        // one K step of 16 keys per group; P (bf16) of group q sits in columns [8q, 8q + 8) of S
#pragma unroll 1
        for (int ks = 0; ks < pend_ng; ++ks) {
          const uint64_t db =
              smem_desc_sw128(smem_u32(v_s + st * C::kTileBytes + ks * C::kSlotStride), C::kHalfStride, C::kSbo);
          mma_ts(tmem_o, tmem + 128u * sb + 8 * ks, db, idesc_pv, (!pend_first || ks > 0) ? 1u : 0u);
        }
        mma_commit(&sh->v_empty[st]);
        mma_commit(&sh->pv_done);
        if (pend_last) mma_commit(&sh->o_done);
        pending = false;
      };
      int seq = 0;
      for (int item = (int)blockIdx.x; item < n_items && ok; item += item_step, ++seq) {
        const ItemPlan *pl = &sh->plan[seq & 1];
        ok = wait_or_abort(&sh->item_ready[seq & 1], (uint32_t)(seq >> 1) & 1u, abort_flag, err);
        if (!ok) break;
        const int n_tiles = pl->n_tiles;
        const bool packing = kCanPack && pl->packing != 0u;
        const uint32_t n_slots = pl->n_slots;
        __threadfence_block();
        atomicAdd(&sh->readers_done, 1);
        if (n_tiles <= 0) continue;
        // the previous item's last O += P V goes first: its epilogue should not wait for this
        // item's first loads
        if (pending) issue_pv();
        if (!ok) break;
        const int qb = (int)(n & 1u);
        ok = wait_or_abort(&sh->q_full[qb], (n >> 1) & 1u, abort_flag, err);
        if (!ok) break;
        const uint32_t n_rounds = packing ? (n_slots + 7u) / 8u : (uint32_t)n_tiles;
        for (uint32_t v = 0; v < n_rounds && ok; ++v, ++g) {
          const int st = (int)(g % C::kStages);
          const uint32_t sb = g & 1u;
          const int ng = packing ? min(8, (int)(n_slots - 8u * v)) : 8;
          ok = wait_or_abort(&sh->k_full[st], (g / C::kStages) & 1u, abort_flag, err);
          if (!ok) break;
          tc_fence_after_sync();
          // S[sb] = Q K_round^T: N = 16 ng, D/16 steps of K = 16 (32 bytes inside the swizzled rows).
          // S[sb] last held P of round g - 2, whose O += P V was issued before this.
          const uint32_t idesc_qk = idesc_bf16_f32(128, 16 * ng, false, false);
#pragma unroll 1
          for (int ks = 0; ks < D / 16; ++ks) {
            const int sub = ks / 4, off = (ks % 4) * 32;
            const uint64_t da = smem_desc_sw128(smem_u32(q_s + qb * C::kTileBytes + sub * kSubBytes + off), 16, 1024);
            const uint64_t db =
                smem_desc_sw128(smem_u32(k_s + st * C::kTileBytes + sub * C::kHalfStride + off), 16, C::kSbo);
            mma_ss(tmem + 128u * sb, da, db, idesc_qk, ks > 0);
          }
          mma_commit(&sh->k_empty[st]);
          if (v + 1 == n_rounds) mma_commit(&sh->q_empty[qb]);
          mma_commit(&sh->s_full[sb]);
          if (pending) issue_pv();
          if (!ok) break;
          pending = true;
          pend_g = g;
          pend_n = n;
          pend_ng = ng;
          pend_first = v == 0;
          pend_last = v + 1 == n_rounds;
        }
        ++n;
      }
      if (ok && pending) issue_pv();
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int r = warp * 32 + lane;          // row of the query tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    const float ref_slack = 8.f / scale_log2;
    bool ok = true;
    uint32_t g = 0, n = 0;
    int seq = 0;
    for (int item = (int)blockIdx.x; item < n_items && ok; item += item_step, ++seq) {
      const int bh = (item % B) * H + (item / B) % H;
      const int qt = n_qt - 1 - item / (B * H);
      const int i = qt * kTile + r;
      const ItemPlan *pl = &sh->plan[seq & 1];
      ok = wait_or_abort(&sh->item_ready[seq & 1], (uint32_t)(seq >> 1) & 1u, abort_flag, err);
      if (!ok) break;
      const int t_begin = pl->t_begin, n_tiles = pl->n_tiles;
      const bool packing = kCanPack && pl->packing != 0u;
      const uint32_t n_slots = pl->n_slots;
      auto plan_read_done = [&]() {
        __syncwarp();
        if (lane == 0) {
          __threadfence_block();
          atomicAdd(&sh->readers_done, 1);
        }
      };
      if (n_tiles <= 0) {  // no stored tile: every row of this query tile is fully pruned
        plan_read_done();
        if (i < Lq) {
          uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + i) * D);
#pragma unroll
          for (int c = 0; c < D / 8; ++c) dst[c] = make_uint4(0u, 0u, 0u, 0u);
        }
        continue;
      }
      const uint32_t n_rounds = packing ? (n_slots + 7u) / 8u : (uint32_t)n_tiles;
      float m = -CUDART_INF_F, l = 0.f;       // exponent reference and running sum of weights
      // Bitmap words of the round after the current one, requested one round ahead.
      // Tile by tile: this thread's row of the next tile (bw) and that tile's flag.
      // Packed: for each of the eight slots the word of this thread's row that holds the slot's
      // 16 columns (raw[q]), the slots' plan entries (tg) and whether any slot is partial.
      uint4 bw = make_uint4(0u, 0u, 0u, 0u);
      bool full = false;
      uint32_t raw[8];
      uint4 tg = make_uint4(0u, 0u, 0u, 0u);
      bool next_partial = false;
      auto fetch_packed = [&](uint32_t v) {
        tg = *reinterpret_cast<const uint4 *>(&pl->tg[8u * v]);
        const int ng = min(8, (int)(n_slots - 8u * v));
        next_partial = pl->partial[v] != 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const uint32_t pair = q < 2 ? tg.x : q < 4 ? tg.y : q < 6 ? tg.z : tg.w;
          const uint32_t e = (q & 1) ? pair >> 16 : pair & 0xffffu;
          raw[q] = q < ng ? 0xffffffffu : 0u;
          if (next_partial && q < ng && !(e & 0x8000u))
            raw[q] = ldg_now_u32(bitmap + (size_t)(t_begin + (int)((e >> 3) & 0xfffu)) * kBitmapWords + r * 4 +
                                 ((e & 7u) >> 1));
        }
      };
      if (!packing) {
        bw = ldg_now_v4(bitmap + (size_t)t_begin * kBitmapWords + r * 4);
        full = ldg_now_u8(flags + t_begin) & 1u;
      } else {
        fetch_packed(0);
      }
      for (uint32_t v = 0; v < n_rounds && ok; ++v, ++g) {
        const uint32_t sb = g & 1u;
        const uint32_t tmem_s = tmem + 128u * sb;
        const bool last = v + 1 == n_rounds;
        int n_chunks = 4;            // 32-column chunks the round spans
        bool tile_full = full;
        uint4 cur = bw;
        if (packing) {
          const int ng = min(8, (int)(n_slots - 8u * v));
          n_chunks = (ng + 1) >> 1;
          tile_full = ng == 8 && !next_partial;
          // this thread's packed bitmap row: slot q's 16 bits at [16q, 16q + 16)
          uint32_t f[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const uint32_t pair = q < 2 ? tg.x : q < 4 ? tg.y : q < 6 ? tg.z : tg.w;
            const uint32_t e = (q & 1) ? pair >> 16 : pair & 0xffffu;
            f[q] = (raw[q] >> (16u * (e & 1u))) & 0xffffu;
          }
          cur = make_uint4(f[0] | (f[1] << 16), f[2] | (f[3] << 16), f[4] | (f[5] << 16), f[6] | (f[7] << 16));
          if (!last) fetch_packed(v + 1);
        } else if (!last) {  // next tile's bitmap row while this one computes
          bw = ldg_now_v4(bitmap + (size_t)(t_begin + v + 1) * kBitmapWords + r * 4);
          full = ldg_now_u8(flags + t_begin + v + 1) & 1u;
        }
        if (last) plan_read_done();  // nothing of the plan is read after this point
        // 32-column chunks in which none of this warp's 32 rows keeps anything are skipped
        // (their P is written as zeros without reading S); a fully kept tile needs no bitmap
        const uint32_t w0 = tile_full ? 0xffffffffu : cur.x, w1 = tile_full ? 0xffffffffu : cur.y,
                       w2 = tile_full ? 0xffffffffu : cur.z, w3 = tile_full ? 0xffffffffu : cur.w;
        const uint32_t active = (__any_sync(0xffffffffu, w0 != 0u) ? 1u : 0u) | (__any_sync(0xffffffffu, w1 != 0u) ? 2u : 0u) |
                                (__any_sync(0xffffffffu, w2 != 0u) ? 4u : 0u) | (__any_sync(0xffffffffu, w3 != 0u) ? 8u : 0u);
        ok = wait_or_abort(&sh->s_full[sb], (g >> 1) & 1u, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        // pass 1: row maximum over kept entries (four independent chains).  In a partially filled
        // tile the pruned entries are replaced by -inf and the chunk is written back to TMEM, so
        // that pass 2 needs no bitmap: exp2 of -inf is exactly 0.
        float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F, mx2 = -CUDART_INF_F, mx3 = -CUDART_INF_F;
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
          if (!((active >> c) & 1u)) continue;
          uint32_t x[32];
          tmem_ld32(tmem_s + lane_addr + 32 * c, x);
          tmem_wait_ld();
          if (!tile_full) {
            const uint32_t w = c == 0 ? w0 : c == 1 ? w1 : c == 2 ? w2 : w3;
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (!((w >> e) & 1u)) x[e] = 0xff800000u;  // -inf
            tmem_st32(tmem_s + lane_addr + 32 * c, x);
          }
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            mx0 = fmaxf(mx0, __uint_as_float(x[e]));
            mx1 = fmaxf(mx1, __uint_as_float(x[e + 1]));
            mx2 = fmaxf(mx2, __uint_as_float(x[e + 2]));
            mx3 = fmaxf(mx3, __uint_as_float(x[e + 3]));
          }
        }
        const float tile_max = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        if (!tile_full) tmem_wait_st();  // the masked chunks are re-read below
        // The exponent's reference m follows the running maximum lazily: it moves only when
        // the maximum outgrows it by more than 2^8 in the exp2 domain (weights stay <= 256,
        // well inside bf16 and fp32 range), which saves most rescales of O.  O / l does not
        // depend on the reference.
        const bool move = tile_max > m + ref_slack;   // also true for the first kept entry (m = -inf)
        const float m_new = move ? tile_max : m;
        const float m_safe = m_new == -CUDART_INF_F ? 0.f : m_new;
        const float alpha = move ? ex2_approx((m - m_safe) * scale_log2) : 1.f;  // 0 when m was -inf
        const float neg_mc = -m_safe * scale_log2;
        m = m_new;
        // Rescale the running output where the reference moved.  O += P V of the previous round may
        // still be running (this round's S was computed ahead of it): wait for it first.
        if (v > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
          ok = wait_or_abort(&sh->pv_done, (g - 1u) & 1u, abort_flag, err);
          if (!ok) break;
          tc_fence_after_sync();
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_addr + 32 * c, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_o + lane_addr + 32 * c, o);
          }
        }
        // pass 2: P = exp2(c*S - c*m); pruned entries are -inf by now and give exactly 0; bf16 P over S
        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll 1
        for (int c = 0; c < n_chunks; ++c) {
          uint32_t pk[16];
          if (!((active >> c) & 1u)) {
#pragma unroll
            for (int e = 0; e < 16; ++e) pk[e] = 0u;
            tmem_st16(tmem_s + lane_addr + 16 * c, pk);
            continue;
          }
          uint32_t x[32];
          tmem_ld32(tmem_s + lane_addr + 32 * c, x);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = ex2_approx(fmaf(__uint_as_float(x[2 * e]), scale_log2, neg_mc));
            const float p1 = ex2_approx(fmaf(__uint_as_float(x[2 * e + 1]), scale_log2, neg_mc));
            __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<uint32_t *>(&hh);
            // the row sum is taken over the bf16-rounded weights the MMA will use, so that
            // O / l is an exact convex combination of V rows whatever the rounding of P
            sum0 += __uint_as_float(pk[e] << 16);
            sum1 += __uint_as_float(pk[e] & 0xffff0000u);
          }
          tmem_st16(tmem_s + lane_addr + 16 * c, pk);
        }
        l = l * alpha + (sum0 + sum1);
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&sh->p_full[sb]);
      }
      if (!ok) break;
      // epilogue: O / l, rounded once to bf16
      ok = wait_or_abort(&sh->o_done, n & 1u, abort_flag, err);
      if (!ok) break;
      tc_fence_after_sync();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16 *orow = O + ((size_t)bh * Lq + i) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_addr + 32 * c, o);
        tmem_wait_ld();
        if (c == D / 32 - 1) {  // O is in registers: the next item may overwrite it
          tc_fence_before_sync();
          mbar_arrive(&sh->o_free);
        }
        if (i < Lq) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // a row without kept entries has l = 0 and P = 0 throughout: write exact zeros
              const float a = l > 0.f ? __uint_as_float(o[8 * q + 2 * e]) * inv : 0.f;
              const float bb = l > 0.f ? __uint_as_float(o[8 * q + 2 * e + 1]) * inv : 0.f;
              __nv_bfloat162 hh = __floats2bfloat162_rn(a, bb);
              pk[e] = *reinterpret_cast<uint32_t *>(&hh);
            }
            *reinterpret_cast<uint4 *>(orow + 32 * c + 8 * q) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      ++n;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, kTmemCols);
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

template <int D, bool kCanPack, bool kSplit>
cudaError_t launch(const FwdMaps &maps, void *O, const ap_tiles &t, int B, int H, int Lq, float scale,
                   unsigned *err, cudaStream_t s) {
  using C = Cfg<D, kSplit>;
  static_assert(sizeof(Shared) <= 14 * 1024, "shared bookkeeping outgrew its reservation");
  static_assert(C::kSmemBytes > 114 * 1024 && C::kSmemBytes <= 227 * 1024, "one CTA per SM, within the limit");
  auto kern = fwd_tc_kernel<D, kCanPack, kSplit>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int n_items = B * H * t.n_qt;
  const float scale_log2 = scale * 1.4426950408889634f;
  kern<<<n_items < sms ? n_items : sms, kThreads, C::kSmemBytes, s>>>(
      maps, static_cast<__nv_bfloat16 *>(O), t.row_ptr, t.col_idx, t.flags, t.bitmap, t.groups, B, H, Lq, t.n_qt,
      n_items, scale_log2, err);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                          int Lq, int Lk, int d, float scale, cudaStream_t s) {
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
  // lists are at most n_kt tiles long: below the packing threshold the smaller kernel does
  const bool can_pack = t.n_kt >= kMinTilesToPack;
  if (d == 64)
    return can_pack ? launch<64, true, false>(maps, O, t, B, H, Lq, scale, err, s)
                    : launch<64, false, false>(maps, O, t, B, H, Lq, scale, err, s);
  if (split)
    return can_pack ? launch<128, true, true>(maps, O, t, B, H, Lq, scale, err, s)
                    : launch<128, false, true>(maps, O, t, B, H, Lq, scale, err, s);
  return can_pack ? launch<128, true, false>(maps, O, t, B, H, Lq, scale, err, s)
                  : launch<128, false, false>(maps, O, t, B, H, Lq, scale, err, s);
}

}  // namespace ap
