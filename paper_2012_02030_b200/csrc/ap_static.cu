// ap_mask_to_tiles_static: the tile-list builder for callers that cannot allocate.
//
// Some hosts of this library may not call cudaMalloc at the point where they
// need a tile list: a plugin running inside another framework's memory pool, a
// real-time loop that must not touch the allocator, or code running while the
// device allocator is locked by someone else.  For them the staging area that
// ap_mask_to_tiles takes as a caller-provided workspace lives here instead, in
// a fixed array in device global memory that belongs to the library image.
// Every GPU that loads the library carries the array until the process exits.
#include "ap_common.cuh"

namespace ap {

namespace {

constexpr int kStaticMaxTiles = AP_STATIC_MAX_TILES;
// bitmaps + popcounts + list positions of kStaticMaxTiles tiles, same layout as stage_bytes()
constexpr size_t kStaticBytes =
    (size_t)kStaticMaxTiles * kBitmapWords * sizeof(uint32_t) +
    2 * (((size_t)kStaticMaxTiles * sizeof(int32_t) + 255) / 256 * 256);

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a
// device address and must never be handed to a kernel directly.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
void *g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device; resolved once per device.
void *static_scratch() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  if (!g_scratch_ptr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return nullptr;
    g_scratch_ptr[dev] = p;
  }
  return g_scratch_ptr[dev];
}

}  // namespace
}  // namespace ap

using namespace ap;

extern "C" ap_status ap_mask_to_tiles_static(const uint8_t *mask, int H, int Lq, int Lk, ap_tiles *tiles,
                                             void *stream) {
  if (!mask || H < 1 || Lq < 1 || Lk < 1) return AP_ERR_INVALID_ARG;
  const ap_status st = check_tiles(tiles, H, Lq, Lk, false);
  if (st != AP_OK) return st;
  const int64_t n_tiles = (int64_t)H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
  if (n_tiles > kStaticMaxTiles) return AP_ERR_WORKSPACE;  // beyond the built-in scratch
  if (stage_bytes(H, Lq, Lk) > kStaticBytes) return AP_ERR_WORKSPACE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return AP_ERR_CUDA;
  char *ws = static_cast<char *>(static_scratch());
  if (!ws || !device_error_word()) return AP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t *stage_bitmap = reinterpret_cast<uint32_t *>(ws);
  int32_t *stage_count = reinterpret_cast<int32_t *>(ws + (size_t)n_tiles * kBitmapWords * sizeof(uint32_t));
  // Every staged byte that is read later is written first by the staging
  // kernel (all bitmaps, all popcounts, all positions), so nothing left over
  // from the previous call can leak into this one and nothing needs clearing.
  if (launch_stage_from_mask(mask, H, Lq, Lk, stage_bitmap, stage_count, s) != cudaSuccess) return AP_ERR_CUDA;
  tiles->H = H;
  tiles->Lq = Lq;
  tiles->Lk = Lk;
  tiles->n_qt = ceil_div(Lq, kTile);
  tiles->n_kt = ceil_div(Lk, kTile);
  if (launch_compact_tiles(stage_bitmap, stage_count, *tiles, s) != cudaSuccess) return AP_ERR_CUDA;
  return AP_OK;
}
