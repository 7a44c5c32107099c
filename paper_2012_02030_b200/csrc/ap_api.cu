// The C ABI declared in ap.h: argument validation, workspace carving, dispatch.
// Nothing is enqueued before every argument has been checked.
#include <math.h>

#include <atomic>
#include <mutex>

#include "ap_common.cuh"

namespace ap {

namespace {

__device__ unsigned g_error_word = 0u;  // sticky device status, one per device

std::atomic<unsigned long long> g_launches{0};

constexpr int kMaxDevices = 64;
unsigned *g_error_ptr[kMaxDevices] = {nullptr};

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool shape_ok(int H, int Lq, int Lk) {
  if (H < 1 || Lq < 1 || Lk < 1) return false;
  if ((int64_t)Lq * Lk > (int64_t)1 << 31) return false;                  // 32-bit tie ranks / indices
  if ((int64_t)H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile) > (1 << 24)) return false;
  if ((int64_t)H * Lq * ceil_div(Lk, kTile) > (int64_t)1 << 31) return false;
  return true;
}

void fill_tiles_shape(ap_tiles *t, int H, int Lq, int Lk) {
  t->H = H;
  t->Lq = Lq;
  t->Lk = Lk;
  t->n_qt = ceil_div(Lq, kTile);
  t->n_kt = ceil_div(Lk, kTile);
}

bool have_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev >= 0;
}

}  // namespace

std::atomic<int> g_expire_waits{0};
std::atomic<int> g_schedule{0};

DebugKnobs debug_knobs() {
  const int on = g_expire_waits.load(std::memory_order_relaxed);
  return DebugKnobs{on ? (1u << 12) : (1u << 22), on, g_schedule.load(std::memory_order_relaxed)};
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

void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

unsigned *device_error_word() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  if (!g_error_ptr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_error_word) != cudaSuccess) return nullptr;
    g_error_ptr[dev] = static_cast<unsigned *>(p);
  }
  return g_error_ptr[dev];
}

int64_t domain_size(int Lq, int Lk, int causal) {
  if (!causal) return (int64_t)Lq * Lk;
  // row i sees the keys j <= i + (Lk - Lq), Lk >= Lq
  return (int64_t)Lq * (Lq + 1) / 2 + (int64_t)Lq * (Lk - Lq);
}

int64_t keep_count(int64_t n_valid, int64_t n_forced, double keep_frac) {
  int64_t k = (int64_t)floor(keep_frac * (double)n_valid + 0.5);
  if (k > n_valid) k = n_valid;
  if (k < n_forced) k = n_forced;
  return k;
}

}  // namespace ap

using namespace ap;

extern "C" {

int ap_version(void) { return 200; }

void ap_debug_expire_waits(int on) { ap::g_expire_waits.store(on ? 1 : 0, std::memory_order_relaxed); }

void ap_debug_schedule(int mode) {
  ap::g_schedule.store(mode == 1 || mode == 2 ? mode : 0, std::memory_order_relaxed);
}

uint64_t ap_launch_count(void) { return (uint64_t)g_launches.load(std::memory_order_relaxed); }

const char *ap_status_string(ap_status s) {
  switch (s) {
    case AP_OK: return "ok";
    case AP_ERR_INVALID_ARG: return "invalid argument";
    case AP_ERR_UNSUPPORTED: return "unsupported head dimension or dtype";
    case AP_ERR_WORKSPACE: return "workspace or tile capacity too small";
    case AP_ERR_CUDA: return "CUDA runtime error";
    case AP_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int64_t ap_tiles_capacity(int H, int Lq, int Lk) {
  if (H < 1 || Lq < 1 || Lk < 1) return 0;
  return (int64_t)H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
}

size_t ap_mask_to_tiles_workspace_bytes(int H, int Lq, int Lk) {
  if (!shape_ok(H, Lq, Lk)) return 0;
  return stage_bytes(H, Lq, Lk);
}

size_t ap_build_mask_workspace_bytes(int H, int Lq, int Lk) {
  if (!shape_ok(H, Lq, Lk)) return 0;
  return stage_bytes(H, Lq, Lk) + select_scratch_bytes(H, Lq, Lk);
}

ap_status ap_accumulate_attention(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                  int Lq, int Lk, int d, ap_dtype dt, int causal, float scale, void *stream) {
  if (!acc || !Q || !K || !aligned16(acc) || !aligned16(Q) || !aligned16(K) || (bias && !aligned16(bias)))
    return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || (causal && Lk < Lq) || !(scale >= 0.f) || isinf(scale))
    return AP_ERR_INVALID_ARG;
  if ((d != 64 && d != 128) || (dt != AP_F32 && dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  const float sc = scale == 0.f ? (float)(1.0 / sqrt((double)d)) : scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt != AP_F32 && !device_error_word()) return AP_ERR_CUDA;
  cudaError_t e = dt == AP_F32 ? launch_accumulate_simt(acc, Q, K, bias, B, H, Lq, Lk, d, dt, causal ? 1 : 0, sc, s)
                               : launch_accumulate_tc(acc, Q, K, bias, B, H, Lq, Lk, d, causal ? 1 : 0,
                                                      dt == AP_F16 ? 1 : 0, sc, s);
  if (e == cudaErrorInvalidValue) return AP_ERR_UNSUPPORTED;  // key length beyond the shared-memory budget
  return e == cudaSuccess ? AP_OK : AP_ERR_CUDA;
}

ap_status ap_accumulate_attention_entmax15(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                           int Lq, int Lk, int d, ap_dtype dt, int causal, float scale,
                                           void *stream) {
  if (!acc || !Q || !K || !aligned16(acc) || !aligned16(Q) || !aligned16(K) || (bias && !aligned16(bias)))
    return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || (causal && Lk < Lq) || !(scale >= 0.f) || isinf(scale))
    return AP_ERR_INVALID_ARG;
  if ((d != 64 && d != 128) || (dt != AP_F32 && dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (!have_device() || !device_error_word()) return AP_ERR_CUDA;
  const float sc = scale == 0.f ? (float)(1.0 / sqrt((double)d)) : scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = dt == AP_F32
                      ? launch_accumulate_simt(acc, Q, K, bias, B, H, Lq, Lk, d, dt, causal ? 1 : 0, sc, s, 1)
                      : launch_accumulate_entmax_tc(acc, Q, K, bias, B, H, Lq, Lk, d, causal ? 1 : 0,
                                                    dt == AP_F16 ? 1 : 0, sc, s);
  if (e == cudaErrorInvalidValue) return AP_ERR_UNSUPPORTED;  // key length beyond the shared-memory budget
  return e == cudaSuccess ? AP_OK : AP_ERR_CUDA;
}

namespace {
ap_status build_mask_impl(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal, int keep_diag,
                          uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head, void *workspace,
                          size_t workspace_bytes, void *stream, int per_layer, int keep_ties = 0) {
  if (!acc || !aligned16(acc) || !shape_ok(H, Lq, Lk) || (causal && Lk < Lq)) return AP_ERR_INVALID_ARG;
  if (!(keep_frac > 0.0) || !(keep_frac <= 1.0)) return AP_ERR_INVALID_ARG;
  if (mask && !aligned16(mask)) return AP_ERR_INVALID_ARG;
  if (nnz_per_head && (reinterpret_cast<uintptr_t>(nnz_per_head) & 7u)) return AP_ERR_INVALID_ARG;
  if (tiles) {
    ap_status st = check_tiles(tiles, H, Lq, Lk, false);
    if (st != AP_OK) return st;
  }
  if (!workspace || !aligned16(workspace)) return AP_ERR_INVALID_ARG;
  if (workspace_bytes < ap_build_mask_workspace_bytes(H, Lq, Lk)) return AP_ERR_WORKSPACE;
  // the selection over a whole layer ranks ties by a 32-bit global index (h*Lq + i)*Lk + j
  if (per_layer && (int64_t)H * Lq * Lk > (int64_t)0xffffffffLL) return AP_ERR_UNSUPPORTED;
  // one selection per head is one grid row per head (65 535 grid rows at most)
  if (!per_layer && H > 65535) return AP_ERR_UNSUPPORTED;
  if (!have_device() || !device_error_word()) return AP_ERR_CUDA;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int n_tiles = H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
  char *ws = static_cast<char *>(workspace);
  const size_t stage = stage_bytes(H, Lq, Lk);
  BuildMaskArgs a;
  a.acc = acc;
  a.H = H; a.Lq = Lq; a.Lk = Lk;
  a.causal = causal ? 1 : 0;
  a.keep_diag = keep_diag ? 1 : 0;
  a.per_layer = per_layer;
  a.keep_ties = keep_ties;
  // population of one selection: a head's domain, or the union of the heads' domains
  const int64_t heads = per_layer ? H : 1;
  const int64_t n_valid = domain_size(Lq, Lk, a.causal) * heads;
  const int64_t n_forced = ((a.keep_diag && (Lq == Lk || a.causal)) ? Lq : 0) * heads;
  a.k = keep_count(n_valid, n_forced, keep_frac);
  a.k_rest = a.k - n_forced;
  a.mask = mask;
  a.nnz = nnz_per_head;
  a.stage_bitmap = tiles ? reinterpret_cast<uint32_t *>(ws) : nullptr;
  a.stage_count = tiles ? reinterpret_cast<int32_t *>(ws + (size_t)n_tiles * kBitmapWords * sizeof(uint32_t)) : nullptr;
  a.scratch = ws + stage;
  if (launch_build_mask(a, s) != cudaSuccess) return AP_ERR_CUDA;
  if (tiles) {
    fill_tiles_shape(tiles, H, Lq, Lk);
    if (launch_compact_tiles(a.stage_bitmap, a.stage_count, *tiles, s) != cudaSuccess) return AP_ERR_CUDA;
  }
  return AP_OK;
}
}  // namespace

ap_status ap_build_mask(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal, int keep_diag,
                        uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head, void *workspace,
                        size_t workspace_bytes, void *stream) {
  return build_mask_impl(acc, H, Lq, Lk, keep_frac, causal, keep_diag, mask, tiles, nnz_per_head, workspace,
                         workspace_bytes, stream, 0);
}

ap_status ap_build_mask_layer(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal, int keep_diag,
                              uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head, void *workspace,
                              size_t workspace_bytes, void *stream) {
  return build_mask_impl(acc, H, Lq, Lk, keep_frac, causal, keep_diag, mask, tiles, nnz_per_head, workspace,
                         workspace_bytes, stream, 1);
}

ap_status ap_build_mask_ex(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal, int keep_diag,
                           int flags, uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head, void *workspace,
                           size_t workspace_bytes, void *stream) {
  if (flags & ~(AP_MASK_PER_LAYER | AP_MASK_KEEP_TIES)) return AP_ERR_INVALID_ARG;
  return build_mask_impl(acc, H, Lq, Lk, keep_frac, causal, keep_diag, mask, tiles, nnz_per_head, workspace,
                         workspace_bytes, stream, (flags & AP_MASK_PER_LAYER) ? 1 : 0,
                         (flags & AP_MASK_KEEP_TIES) ? 1 : 0);
}

namespace {
bool block_ok(int Lq, int Lk, int block) {
  return (block == 16 || block == 32 || block == 64 || block == 128) && Lq % block == 0 && Lk % block == 0;
}
}  // namespace

ap_status ap_pool_scores(const float *acc, int H, int Lq, int Lk, int block, int causal, float *pooled,
                         void *stream) {
  if (!acc || !pooled || !aligned16(acc) || !aligned16(pooled) || !shape_ok(H, Lq, Lk) || (causal && Lk < Lq))
    return AP_ERR_INVALID_ARG;
  if (!block_ok(Lq, Lk, block)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  return launch_pool_scores(acc, H, Lq, Lk, block, causal ? 1 : 0, pooled, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess
             ? AP_OK
             : AP_ERR_CUDA;
}

ap_status ap_expand_block_mask(const uint8_t *block_mask, int H, int Lq, int Lk, int block, int causal,
                               uint8_t *mask, void *stream) {
  if (!block_mask || !mask || !aligned16(mask) || !shape_ok(H, Lq, Lk) || (causal && Lk < Lq))
    return AP_ERR_INVALID_ARG;
  if (!block_ok(Lq, Lk, block)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  return launch_expand_block_mask(block_mask, H, Lq, Lk, block, causal ? 1 : 0, mask,
                                  static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? AP_OK
             : AP_ERR_CUDA;
}

ap_status ap_random_scores(float *scores, int H, int Lq, int Lk, uint64_t seed, void *stream) {
  if (!scores || !aligned16(scores) || !shape_ok(H, Lq, Lk)) return AP_ERR_INVALID_ARG;
  if (!have_device()) return AP_ERR_CUDA;
  return launch_random_scores(scores, (int64_t)H * Lq * Lk, seed, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? AP_OK
             : AP_ERR_CUDA;
}

ap_status ap_mask_to_tiles(const uint8_t *mask, int H, int Lq, int Lk, ap_tiles *tiles, void *workspace,
                           size_t workspace_bytes, void *stream) {
  if (!mask || !shape_ok(H, Lq, Lk)) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, false);
  if (st != AP_OK) return st;
  if (!workspace || !aligned16(workspace)) return AP_ERR_INVALID_ARG;
  if (workspace_bytes < ap_mask_to_tiles_workspace_bytes(H, Lq, Lk)) return AP_ERR_WORKSPACE;
  if (!have_device() || !device_error_word()) return AP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int n_tiles = H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
  char *ws = static_cast<char *>(workspace);
  uint32_t *stage_bitmap = reinterpret_cast<uint32_t *>(ws);
  int32_t *stage_count = reinterpret_cast<int32_t *>(ws + (size_t)n_tiles * kBitmapWords * sizeof(uint32_t));
  if (launch_stage_from_mask(mask, H, Lq, Lk, stage_bitmap, stage_count, s) != cudaSuccess) return AP_ERR_CUDA;
  fill_tiles_shape(tiles, H, Lq, Lk);
  if (launch_compact_tiles(stage_bitmap, stage_count, *tiles, s) != cudaSuccess) return AP_ERR_CUDA;
  return AP_OK;
}

ap_status ap_dense_tiles(int H, int Lq, int Lk, int causal, ap_tiles *tiles, void *stream) {
  if (!shape_ok(H, Lq, Lk) || (causal && Lk < Lq)) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, false);
  if (st != AP_OK) return st;
  const int n_qt = ceil_div(Lq, kTile), n_kt = ceil_div(Lk, kTile);
  const int64_t need = (int64_t)H * dense_row_start(n_qt, n_kt, Lq, Lk, causal ? 1 : 0);
  if (tiles->cap < need) return AP_ERR_WORKSPACE;
  if (!have_device() || !device_error_word()) return AP_ERR_CUDA;
  fill_tiles_shape(tiles, H, Lq, Lk);
  return launch_dense_tiles(*tiles, causal ? 1 : 0, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? AP_OK
             : AP_ERR_CUDA;
}

ap_status ap_sparse_attention_fwd(const void *Q, const void *K, const void *V, const ap_tiles *tiles, void *O,
                                  int B, int H, int Lq, int Lk, int d, ap_dtype dt, float scale, void *stream) {
  if (!Q || !K || !V || !O || !aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O))
    return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || !(scale >= 0.f) || isinf(scale)) return AP_ERR_INVALID_ARG;
  if ((int64_t)B * H * ceil_div(Lq, kTile) > (int64_t)0x7fffffff) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, true);
  if (st != AP_OK) return st;
  if ((d != 64 && d != 128) || (dt != AP_F32 && dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  const float sc = scale == 0.f ? (float)(1.0 / sqrt((double)d)) : scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = dt == AP_F32 ? launch_fwd_simt(Q, K, V, *tiles, O, B, H, Lq, Lk, d, sc, s)
                               : launch_fwd_tc(Q, K, V, *tiles, O, B, H, Lq, Lk, d, dt == AP_F16 ? 1 : 0, sc, s);
  return e == cudaSuccess ? AP_OK : AP_ERR_CUDA;
}

ap_status ap_sparse_attention_entmax15_fwd(const void *Q, const void *K, const void *V, const ap_tiles *tiles,
                                           void *O, int B, int H, int Lq, int Lk, int d, ap_dtype dt, float scale,
                                           void *stream) {
  if (!Q || !K || !V || !O || !aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O))
    return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || !(scale >= 0.f) || isinf(scale)) return AP_ERR_INVALID_ARG;
  if ((int64_t)B * H * ceil_div(Lq, kTile) > (int64_t)0x7fffffff) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, true);
  if (st != AP_OK) return st;
  if ((d != 64 && d != 128) || (dt != AP_F32 && dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  const float sc = scale == 0.f ? (float)(1.0 / sqrt((double)d)) : scale;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = dt == AP_F32 ? launch_fwd_entmax_simt(Q, K, V, *tiles, O, B, H, Lq, Lk, d, sc, s)
                               : launch_fwd_entmax_tc(Q, K, V, *tiles, O, B, H, Lq, Lk, d, dt == AP_F16 ? 1 : 0, sc, s);
  return e == cudaSuccess ? AP_OK : AP_ERR_CUDA;
}

size_t ap_sparse_attention_bwd_workspace_bytes(int B, int H, int Lq, int Lk) {
  if (B < 1 || !shape_ok(H, Lq, Lk)) return 0;
  return bwd_workspace_bytes(B, H, Lq, Lk);
}

ap_status ap_sparse_attention_bwd(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                                  const ap_tiles *tiles, void *dQ, void *dK, void *dV, int B, int H, int Lq,
                                  int Lk, int d, ap_dtype dt, float scale, void *workspace,
                                  size_t workspace_bytes, void *stream) {
  const void *ptrs[] = {Q, K, V, O, dO, dQ, dK, dV, workspace};
  for (const void *p : ptrs)
    if (!p || !aligned16(p)) return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || !(scale >= 0.f) || isinf(scale)) return AP_ERR_INVALID_ARG;
  if ((int64_t)B * H * ceil_div(Lq > Lk ? Lq : Lk, kTile) > (int64_t)0x7fffffff) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, true);
  if (st != AP_OK) return st;
  if ((d != 64 && d != 128) || (dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (workspace_bytes < bwd_workspace_bytes(B, H, Lq, Lk)) return AP_ERR_WORKSPACE;
  if (!have_device()) return AP_ERR_CUDA;
  const float sc = scale == 0.f ? (float)(1.0 / sqrt((double)d)) : scale;
  return launch_bwd_tc(Q, K, V, O, dO, *tiles, dQ, dK, dV, workspace, B, H, Lq, Lk, d, dt == AP_F16 ? 1 : 0, sc,
                       static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? AP_OK
             : AP_ERR_CUDA;
}

namespace {
// Streams and events of ap_sparse_attention_fwd_host, one set per device, created on first use and
// kept for the life of the process: an input-copy stream, an output-copy stream and one event pair
// per chunk of batch elements.
constexpr int kMaxChunks = 8;
struct HostPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, out_done = nullptr;
  cudaEvent_t in_done[kMaxChunks] = {}, fwd_done[kMaxChunks] = {};
};
HostPipe g_pipe[kMaxDevices];
std::mutex g_pipe_mutex;

HostPipe *host_pipe() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe &p = g_pipe[dev];
  if (!p.ready) {
    bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&p.out_done, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; ok && c < kMaxChunks; ++c)
      ok = cudaEventCreateWithFlags(&p.in_done[c], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&p.fwd_done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;
    p.ready = true;
  }
  return &p;
}
}  // namespace

ap_status ap_sparse_attention_fwd_host(const void *hQ, const void *hK, const void *hV, const ap_tiles *tiles,
                                       void *hO, void *dQ, void *dK, void *dV, void *dO, int B, int H, int Lq,
                                       int Lk, int d, ap_dtype dt, float scale, void *stream) {
  if (!hQ || !hK || !hV || !hO) return AP_ERR_INVALID_ARG;
  if (!dQ || !dK || !dV || !dO || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV) || !aligned16(dO))
    return AP_ERR_INVALID_ARG;
  if (B < 1 || !shape_ok(H, Lq, Lk) || !(scale >= 0.f) || isinf(scale)) return AP_ERR_INVALID_ARG;
  ap_status st = check_tiles(tiles, H, Lq, Lk, true);
  if (st != AP_OK) return st;
  if ((d != 64 && d != 128) || (dt != AP_F32 && dt != AP_BF16 && dt != AP_F16)) return AP_ERR_UNSUPPORTED;
  if (!have_device()) return AP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t elem = dt == AP_F32 ? 4 : 2;
  // The batch is cut into chunks of batch elements (the masks are per head, so any subset of the
  // batch is a valid call): chunk c + 1 is copied in while chunk c is computed and chunk c - 1 is
  // copied out, so the two directions of the host link work at the same time.
  HostPipe *pipe = host_pipe();
  if (!pipe) return AP_ERR_CUDA;
  const int per_chunk = ceil_div(B, kMaxChunks), n_chunks = ceil_div(B, per_chunk);
  const size_t q_one = elem * H * (size_t)Lq * d, k_one = elem * H * (size_t)Lk * d;  // bytes of one batch element
  bool ok = cudaEventRecord(pipe->start, s) == cudaSuccess &&  // the staging buffers are free once s gets here
            cudaStreamWaitEvent(pipe->in, pipe->start, 0) == cudaSuccess;
  for (int c = 0; ok && c < n_chunks; ++c) {
    const int b0 = c * per_chunk, nb = B - b0 < per_chunk ? B - b0 : per_chunk;
    const size_t qo = q_one * b0, ko = k_one * b0;
    const char *hq = static_cast<const char *>(hQ) + qo, *hk = static_cast<const char *>(hK) + ko,
               *hv = static_cast<const char *>(hV) + ko;
    char *q = static_cast<char *>(dQ) + qo, *k = static_cast<char *>(dK) + ko, *v = static_cast<char *>(dV) + ko,
         *o = static_cast<char *>(dO) + qo;
    ok = cudaMemcpyAsync(q, hq, q_one * nb, cudaMemcpyHostToDevice, pipe->in) == cudaSuccess &&
         cudaMemcpyAsync(k, hk, k_one * nb, cudaMemcpyHostToDevice, pipe->in) == cudaSuccess &&
         cudaMemcpyAsync(v, hv, k_one * nb, cudaMemcpyHostToDevice, pipe->in) == cudaSuccess &&
         cudaEventRecord(pipe->in_done[c], pipe->in) == cudaSuccess &&
         cudaStreamWaitEvent(s, pipe->in_done[c], 0) == cudaSuccess;
    if (!ok) break;
    st = ap_sparse_attention_fwd(q, k, v, tiles, o, nb, H, Lq, Lk, d, dt, scale, stream);
    if (st != AP_OK) break;
    ok = cudaEventRecord(pipe->fwd_done[c], s) == cudaSuccess &&
         cudaStreamWaitEvent(pipe->out, pipe->fwd_done[c], 0) == cudaSuccess &&
         cudaMemcpyAsync(static_cast<char *>(hO) + qo, o, q_one * nb, cudaMemcpyDeviceToHost, pipe->out) == cudaSuccess;
  }
  // whatever happened, s rejoins the output stream: the caller synchronises s only
  // (s has already waited for every input copy issued above)
  const bool joined = cudaEventRecord(pipe->out_done, pipe->out) == cudaSuccess &&
                      cudaStreamWaitEvent(s, pipe->out_done, 0) == cudaSuccess;
  if (st != AP_OK) return st;
  return ok && joined ? AP_OK : AP_ERR_CUDA;
}

ap_status ap_device_status(void *stream) {
  if (!have_device()) return AP_ERR_CUDA;
  unsigned *word = device_error_word();
  if (!word) return AP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned host = 0u;
  if (cudaMemcpyAsync(&host, word, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess) return AP_ERR_CUDA;
  if (cudaMemsetAsync(word, 0, sizeof(host), s) != cudaSuccess) return AP_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return AP_ERR_CUDA;
  if (host & kDevErrTimeout) return AP_ERR_TIMEOUT;
  if (host & kDevErrCapacity) return AP_ERR_WORKSPACE;
  return AP_OK;
}

}  // extern "C"
