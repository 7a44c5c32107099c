// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ap.h"

namespace ap {

constexpr int kTile = AP_TILE;
constexpr int kBitmapWords = kTile * 4;  // 32-bit words of one tile bitmap

// Bits of the sticky device status word.
constexpr unsigned kDevErrCapacity = 1u;
constexpr unsigned kDevErrTimeout = 2u;

// Address of the device status word of the current device (NULL on failure).
unsigned *device_error_word();

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// The checks every entry point that fills or reads a tile list applies to the descriptor before
// anything is enqueued: all arrays present, the arrays that kernels access with 16-byte vectors
// (bitmap, round_bitmap, round_rows) 16-byte aligned, the 32-bit arrays 4-byte aligned, a capacity
// of at least one tile, and (for readers) the recorded shape equal to the call's.
inline ap_status check_tiles(const ap_tiles *t, int H, int Lq, int Lk, bool shape_must_match) {
  auto misaligned = [](const void *p, uintptr_t mask) { return (reinterpret_cast<uintptr_t>(p) & mask) != 0; };
  if (!t) return AP_ERR_INVALID_ARG;
  if (!t->row_ptr || !t->col_idx || !t->flags || !t->bitmap || !t->groups || !t->round_ptr || !t->round_rows ||
      !t->round_info || !t->round_bitmap)
    return AP_ERR_INVALID_ARG;
  if (misaligned(t->bitmap, 15u) || misaligned(t->round_bitmap, 15u) || misaligned(t->round_rows, 15u) ||
      misaligned(t->row_ptr, 3u) || misaligned(t->col_idx, 3u) || misaligned(t->round_ptr, 3u))
    return AP_ERR_INVALID_ARG;
  // the gathered rounds are optional: all four arrays or none
  const int n_g = (t->ground_ptr != nullptr) + (t->ground_keys != nullptr) + (t->ground_info != nullptr) +
                  (t->ground_bitmap != nullptr);
  if (n_g != 0 && n_g != 4) return AP_ERR_INVALID_ARG;
  if (n_g == 4 && (misaligned(t->ground_bitmap, 15u) || misaligned(t->ground_keys, 15u) || misaligned(t->ground_ptr, 3u)))
    return AP_ERR_INVALID_ARG;
  if (t->unit_qt && misaligned(t->unit_qt, 7u)) return AP_ERR_INVALID_ARG;
  if (t->cap < 1) return AP_ERR_WORKSPACE;
  if (shape_must_match) {
    if (t->H != H || t->Lq != Lq || t->Lk != Lk || t->n_qt != ceil_div(Lq, kTile) ||
        t->n_kt != ceil_div(Lk, kTile))
      return AP_ERR_INVALID_ARG;
  }
  return AP_OK;
}

// Poll limit of the kernels' bounded waits and the test hook that makes one wait run out (see
// ap_debug_expire_waits in ap.h): skip_arrive != 0 asks the next launches' producers to leave out
// one arrival on a single-CTA grid.
struct DebugKnobs {
  uint32_t max_polls;
  int skip_arrive;
  int schedule;  // ap_debug_schedule: 0 = gathered rounds where they pay, 1 = never followed, 2 = built for every list row
};
DebugKnobs debug_knobs();

// SMs of the current device (0 if it cannot be queried).
int sm_count();

// Kernels launched by this library in this process (see ap_launch_count in ap.h).
void count_launches(int n);

// Host: entries kept per head (see ap_build_mask in ap.h).
int64_t keep_count(int64_t n_valid, int64_t n_forced, double keep_frac);
int64_t domain_size(int Lq, int Lk, int causal);

// Tiles of the full domain in the list rows 0..qt-1 of a head.  Causal: row i sees the keys
// j <= i + (Lk - Lq), so query tile q holds the key tiles 0 .. min(n_kt, q + 1 + c) - 1 with
// c = ceil((Lk - Lq) / 128).
__host__ __device__ inline int dense_row_tiles(int qt, int n_kt, int Lq, int Lk, int causal) {
  if (!causal) return n_kt;
  const int c = (Lk - Lq + kTile - 1) / kTile;
  return qt + 1 + c < n_kt ? qt + 1 + c : n_kt;
}
__host__ __device__ inline int64_t dense_row_start(int qt, int n_kt, int Lq, int Lk, int causal) {
  if (!causal) return (int64_t)qt * n_kt;
  const int c = (Lk - Lq + kTile - 1) / kTile;
  int a = n_kt - 1 - c;  // query tiles below this one hold fewer than n_kt key tiles
  if (a < 0) a = 0;
  if (a > qt) a = qt;
  return (int64_t)a * (a + 1) / 2 + (int64_t)a * c + (int64_t)(qt - a) * n_kt;
}

// ---- launchers (each returns the cudaError_t of its launches) -------------------------------

// Per-tile bitmaps + popcounts of an element mask into a dense staging area
// stage_bitmap[H*n_qt*n_kt][128][4], stage_count[H*n_qt*n_kt].
cudaError_t launch_stage_from_mask(const uint8_t *mask, int H, int Lq, int Lk, uint32_t *stage_bitmap,
                                   int32_t *stage_count, cudaStream_t s);
// Staging area -> compacted tile list.
cudaError_t launch_compact_tiles(const uint32_t *stage_bitmap, const int32_t *stage_count,
                                 const ap_tiles &t, cudaStream_t s);
cudaError_t launch_dense_tiles(const ap_tiles &t, int causal, cudaStream_t s);

size_t stage_bytes(int H, int Lq, int Lk);

struct BuildMaskArgs {
  const float *acc;
  int H, Lq, Lk, causal, keep_diag;
  int per_layer;   // one selection over all heads instead of one per head
  int keep_ties;   // every entry equal to the threshold is kept (the kept count may exceed k)
  int64_t k_rest;  // entries to select among the non-forced entries of the selection's population
  int64_t k;       // entries kept per selection (per head, or in the whole layer)
  uint8_t *mask;   // may be NULL
  int64_t *nnz;    // may be NULL
  uint32_t *stage_bitmap;  // may be NULL (no tile list wanted)
  int32_t *stage_count;
  void *scratch;  // select scratch
};
size_t select_scratch_bytes(int H, int Lq, int Lk);
cudaError_t launch_build_mask(const BuildMaskArgs &a, cudaStream_t s);

// (entmax: the 1.5-entmax normaliser instead of the softmax; fp32 tensors)
cudaError_t launch_accumulate_simt(float *acc, const void *Q, const void *K, const float *bias, int B,
                                   int H, int Lq, int Lk, int d, ap_dtype dt, int causal, float scale,
                                   cudaStream_t s, int entmax = 0);

// fp32 tensors: CUDA-core kernel
cudaError_t launch_fwd_simt(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O,
                            int B, int H, int Lq, int Lk, int d, float scale, cudaStream_t s);
cudaError_t launch_fwd_entmax_simt(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O,
                                   int B, int H, int Lq, int Lk, int d, float scale, cudaStream_t s);
cudaError_t launch_accumulate_tc(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                 int Lq, int Lk, int d, int causal, int f16, float scale, cudaStream_t s);

// the same sum with 1.5-entmax as the normaliser
cudaError_t launch_accumulate_entmax_tc(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                        int Lq, int Lk, int d, int causal, int f16, float scale, cudaStream_t s);

cudaError_t launch_fwd_entmax_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                                 int Lq, int Lk, int d, int f16, float scale, cudaStream_t s);

// Tensor map of a [B*H, L, d] tensor of 16-bit elements (bf16 or fp16: the copy engine moves them
// unchanged and fills out-of-range elements with zero bits) for box_rows-row x 64-element swizzled boxes.
bool make_tile_map_bf16(CUtensorMap *m, const void *base, int BH, int L, int d, int box_rows = 128);
bool make_split_map_bf16_d128(CUtensorMap *m, const void *base, int BH, int L, int box_rows);
// Tensor map of an [H, Lq, Lk] fp32 tensor for box_rows x 32-column swizzled boxes (Lk % 4 == 0,
// base 16-byte aligned).
bool make_tile_map_f32(CUtensorMap *m, const void *base, int H, int Lq, int Lk, int box_rows = 128);

// bf16 tensors: tcgen05 tensor-core kernel
cudaError_t launch_pool_scores(const float *acc, int H, int Lq, int Lk, int bs, int causal, float *pooled,
                               cudaStream_t s);
cudaError_t launch_expand_block_mask(const uint8_t *block_mask, int H, int Lq, int Lk, int bs, int causal,
                                     uint8_t *mask, cudaStream_t s);
size_t bwd_workspace_bytes(int B, int H, int Lq, int Lk);
cudaError_t launch_bwd_tc(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                          const ap_tiles &t, void *dQ, void *dK, void *dV, void *workspace, int B, int H, int Lq,
                          int Lk, int d, int f16, float scale, cudaStream_t s);
cudaError_t launch_random_scores(float *out, int64_t count, uint64_t seed, cudaStream_t s);
cudaError_t launch_fwd_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O,
                          int B, int H, int Lq, int Lk, int d, int f16, float scale, cudaStream_t s);

}  // namespace ap
