// Masked attention of Section 3.2 for bf16 tensors on the tcgen05 tensor cores.
//
// One CTA per (b, h, query tile of 128 rows).  It walks the tile list of its
// (h, qt) row and, for every stored key tile:
//   S  = Q_tile K_tile^T            tcgen05.mma, both operands in shared memory
//                                   (TMA, 128-byte swizzle), fp32 accumulator in TMEM
//   P  = exp2(c*S - c*m) on kept    one thread per query row reads its S row from
//        entries, 0 on pruned ones  TMEM, applies the tile's bitmap row exactly,
//                                   keeps the running row maximum m and sum l
//                                   (online softmax), rescales O when m moved,
//                                   and writes P as bf16 over S in TMEM
//   O += P V_tile                   tcgen05.mma with A = P from TMEM and
//                                   B = V (MN-major) from shared memory
// and finally writes O / l (zeros for rows that never saw a kept entry).
//
// Warp roles (192 threads): warps 0-3 softmax + epilogue (thread = query row),
// warp 4 TMA producer, warp 5 MMA issuer and TMEM owner.  TMEM: columns
// [0,128) S / P, [128,128+D) O; 256 columns per CTA so two CTAs share an SM and
// one CTA's softmax overlaps the other's MMAs.  Every mbarrier wait is bounded;
// a wait that expires raises the device status word and the CTA winds down.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 192;
constexpr int kSubBytes = 128 * 128;  // one [128 rows][64 bf16] swizzled sub-tile
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kMaxPolls = 1u << 22;

template <int D>
struct Cfg {
  static constexpr int kSub = D / 64;                 // sub-tiles per operand tile
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kStages = D == 64 ? 2 : 1;     // K and V ring depth
  static constexpr int kBarOffset = (1 + 2 * kStages) * kTileBytes;
  static constexpr int kSmemBytes = kBarOffset + 256 + 1024;  // + barriers + alignment slack
};

struct Barriers {
  uint64_t q_full, s_full, p_full, o_done;
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait that also gives up as soon as another thread of the CTA has.
__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
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

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
fwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
              const __grid_constant__ CUtensorMap map_v, __nv_bfloat16 *__restrict__ O,
              const int32_t *__restrict__ row_ptr, const int32_t *__restrict__ col_idx,
              const uint8_t *__restrict__ flags, const uint32_t *__restrict__ bitmap, int B, int H, int Lq,
              int n_qt, float scale_log2, unsigned *err) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *q_s = smem;
  unsigned char *k_s = smem + C::kTileBytes;
  unsigned char *v_s = smem + (1 + C::kStages) * C::kTileBytes;
  Barriers *bars = reinterpret_cast<Barriers *>(smem + C::kBarOffset);

  // work item: heavy (late, under a causal mask) query tiles first; b fastest so
  // that neighbouring CTAs share one tile list and its bitmaps in L2
  const int item = blockIdx.x;
  const int b = item % B;
  const int h = (item / B) % H;
  const int qt = n_qt - 1 - item / (B * H);
  const int bh = b * H + h;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t_begin = row_ptr[h * n_qt + qt], t_end = row_ptr[h * n_qt + qt + 1];
  const int n_tiles = t_end - t_begin;

  if (n_tiles <= 0) {  // no stored tile: every row of this query tile is fully pruned
    if (warp < 4) {
      const int i = qt * kTile + warp * 32 + lane;
      if (i < Lq) {
        uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + i) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) dst[c] = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    return;
  }

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->s_full, 1);
    mbar_init(&bars->p_full, 128);
    mbar_init(&bars->o_done, 1);
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  const uint32_t tmem_s = tmem, tmem_o = tmem + 128;
  volatile int *abort_flag = &bars->abort_flag;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      prefetch_tensormap(&map_v);
      mbar_arrive_expect_tx(&bars->q_full, C::kTileBytes);
#pragma unroll
      for (int s = 0; s < C::kSub; ++s) tma_load_3d(q_s + s * kSubBytes, &map_q, &bars->q_full, 64 * s, qt * kTile, bh);
      int it = 0;
      bool ok = true;
      for (; it < n_tiles && ok; ++it) {
        const int st = it % C::kStages;
        const uint32_t ph = (uint32_t)(it / C::kStages) & 1u;
        const int kt = col_idx[t_begin + it];
        ok = wait_or_abort(&bars->k_empty[st], ph ^ 1u, abort_flag, err);
        if (!ok) break;
        mbar_arrive_expect_tx(&bars->k_full[st], C::kTileBytes);
#pragma unroll
        for (int s = 0; s < C::kSub; ++s)
          tma_load_3d(k_s + st * C::kTileBytes + s * kSubBytes, &map_k, &bars->k_full[st], 64 * s, kt * kTile, bh);
        ok = wait_or_abort(&bars->v_empty[st], ph ^ 1u, abort_flag, err);
        if (!ok) {
          // the K copy just armed is still in flight: let it land before leaving
          mbar_wait(&bars->k_full[st], ph, kMaxPolls);
          break;
        }
        mbar_arrive_expect_tx(&bars->v_full[st], C::kTileBytes);
#pragma unroll
        for (int s = 0; s < C::kSub; ++s)
          tma_load_3d(v_s + st * C::kTileBytes + s * kSubBytes, &map_v, &bars->v_full[st], 64 * s, kt * kTile, bh);
      }
      if (*abort_flag) {
        // winding down: wait (bounded) for every copy this thread armed and nobody consumed
        mbar_wait(&bars->q_full, 0, kMaxPolls);
        for (int j = max(0, it - C::kStages); j < it; ++j) {
          const int st = j % C::kStages;
          const uint32_t ph = (uint32_t)(j / C::kStages) & 1u;
          mbar_wait(&bars->k_full[st], ph, kMaxPolls);
          mbar_wait(&bars->v_full[st], ph, kMaxPolls);
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
      bool ok = wait_or_abort(&bars->q_full, 0, abort_flag, err);
      for (int it = 0; it < n_tiles && ok; ++it) {
        const int st = it % C::kStages;
        const uint32_t ph = (uint32_t)(it / C::kStages) & 1u;
        ok = wait_or_abort(&bars->k_full[st], ph, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        // S = Q K^T: D/16 steps of K = 16 (32 bytes inside the 128-byte swizzled rows)
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int sub = ks / 4, off = (ks % 4) * 32;
          const uint64_t da = smem_desc_sw128(smem_u32(q_s + sub * kSubBytes + off), 16, 1024);
          const uint64_t db = smem_desc_sw128(smem_u32(k_s + st * C::kTileBytes + sub * kSubBytes + off), 16, 1024);
          mma_ss(tmem_s, da, db, idesc_qk, ks > 0);
        }
        mma_commit(&bars->k_empty[st]);
        mma_commit(&bars->s_full);
        ok = wait_or_abort(&bars->p_full, (uint32_t)it & 1u, abort_flag, err);
        if (!ok) break;
        ok = wait_or_abort(&bars->v_full[st], ph, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        // O += P V: 8 steps of 16 keys; P (bf16) sits in the first 64 columns of S
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t db = smem_desc_sw128(smem_u32(v_s + st * C::kTileBytes + ks * 2048), kSubBytes, 1024);
          mma_ts(tmem_o, tmem_s + 8 * ks, db, idesc_pv, (it > 0 || ks > 0) ? 1u : 0u);
        }
        mma_commit(&bars->v_empty[st]);
        if (it == n_tiles - 1) mma_commit(&bars->o_done);
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int r = warp * 32 + lane;          // row of the query tile == TMEM lane
    const int i = qt * kTile + r;
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    float m = -CUDART_INF_F, l = 0.f;       // exponent reference and running sum of weights
    const float ref_slack = 8.f / scale_log2;
    bool ok = true;
    uint4 bw = *reinterpret_cast<const uint4 *>(bitmap + (size_t)t_begin * kBitmapWords + r * 4);
    bool full = flags[t_begin] & 1;
    for (int it = 0; it < n_tiles; ++it) {
      const uint4 cur = bw;
      const bool tile_full = full;
      if (it + 1 < n_tiles) {  // next tile's bitmap row while this one computes
        bw = *reinterpret_cast<const uint4 *>(bitmap + (size_t)(t_begin + it + 1) * kBitmapWords + r * 4);
        full = flags[t_begin + it + 1] & 1;
      }
      ok = wait_or_abort(&bars->s_full, (uint32_t)it & 1u, abort_flag, err);
      if (!ok) break;
      tc_fence_after_sync();
      // 32-column chunks in which none of this warp's 32 rows keeps anything are skipped
      // (their P is written as zeros without reading S)
      const uint32_t w0 = tile_full ? 0xffffffffu : cur.x, w1 = tile_full ? 0xffffffffu : cur.y,
                     w2 = tile_full ? 0xffffffffu : cur.z, w3 = tile_full ? 0xffffffffu : cur.w;
      const uint32_t active = (__any_sync(0xffffffffu, w0 != 0u) ? 1u : 0u) | (__any_sync(0xffffffffu, w1 != 0u) ? 2u : 0u) |
                              (__any_sync(0xffffffffu, w2 != 0u) ? 4u : 0u) | (__any_sync(0xffffffffu, w3 != 0u) ? 8u : 0u);
      // pass 1: row maximum over kept entries (four independent chains).  In a partially filled
      // tile the pruned entries are replaced by -inf and the chunk is written back to TMEM, so
      // that pass 2 needs no bitmap: exp2 of -inf is exactly 0.
      float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F, mx2 = -CUDART_INF_F, mx3 = -CUDART_INF_F;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
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
      // rescale the running output where the reference moved (O of step it-1 is complete:
      // the MMA thread committed s_full after it)
      if (it > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
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
      for (int c = 0; c < 4; ++c) {
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
      mbar_arrive(&bars->p_full);
    }
    // epilogue: O / l, rounded once to bf16
    if (ok) ok = wait_or_abort(&bars->o_done, 0, abort_flag, err);
    if (ok) {
      tc_fence_after_sync();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      __nv_bfloat16 *orow = O + ((size_t)bh * Lq + i) * D;
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_o + lane_addr + 32 * c, o);
        tmem_wait_ld();
        if (i < Lq) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // a row without kept entries has l = 0 and P = 0 throughout: write exact zeros
              const float a = l > 0.f ? __uint_as_float(o[8 * g + 2 * e]) * inv : 0.f;
              const float bb = l > 0.f ? __uint_as_float(o[8 * g + 2 * e + 1]) * inv : 0.f;
              __nv_bfloat162 hh = __floats2bfloat162_rn(a, bb);
              pk[e] = *reinterpret_cast<uint32_t *>(&hh);
            }
            *reinterpret_cast<uint4 *>(orow + 32 * c + 8 * g) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
cudaError_t launch(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, void *O, const ap_tiles &t,
                   int B, int H, int Lq, float scale, unsigned *err, cudaStream_t s) {
  auto kern = fwd_tc_kernel<D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  const float scale_log2 = scale * 1.4426950408889634f;
  kern<<<B * H * t.n_qt, kThreads, Cfg<D>::kSmemBytes, s>>>(mq, mk, mv, static_cast<__nv_bfloat16 *>(O), t.row_ptr,
                                                          t.col_idx, t.flags, t.bitmap, B, H, Lq, t.n_qt,
                                                          scale_log2, err);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                          int Lq, int Lk, int d, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  CUtensorMap mq, mk, mv;
  if (!make_tile_map_bf16(&mq, Q, B * H, Lq, d) || !make_tile_map_bf16(&mk, K, B * H, Lk, d) ||
      !make_tile_map_bf16(&mv, V, B * H, Lk, d))
    return cudaErrorUnknown;
  return d == 64 ? launch<64>(mq, mk, mv, O, t, B, H, Lq, scale, err, s)
                 : launch<128>(mq, mk, mv, O, t, B, H, Lq, scale, err, s);
}

}  // namespace ap
