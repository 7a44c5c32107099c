// Block-structured pruning: scores of bs x bs blocks (the mean of the accumulator over the
// block's entries inside the domain) and the expansion of a block mask to an element mask.
// Eq. 2's selection runs in between on the pooled array (the mask builder), so a kept block
// keeps all of its entries inside the domain; with bs = 128 every stored tile of the forward's
// list is fully kept.  Both kernels stream the [H,Lq,Lk] array once with 16-byte accesses.
#include "ap_common.cuh"

namespace ap {

namespace {

constexpr int kThreads = 256;

// One CTA per (block row I, head): the bs rows of the block row are read with float4 loads,
// thread t taking columns 4t .. 4t+3 (+ 1024 per pass) of every row; the bs/4 threads of a block
// then add their sums with shuffles (bs/4 <= 32 consecutive lanes), in a fixed order.
__global__ void __launch_bounds__(kThreads) pool_scores_kernel(const float *__restrict__ acc, int Lq, int Lk, int bs,
                                                               int causal, float *__restrict__ pooled) {
  const int I = blockIdx.x, h = blockIdx.y;
  const int nI = Lq / bs, nJ = Lk / bs;
  const int off = causal ? Lk - Lq : 0;
  const int lanes_per_block = bs / 4;  // 4, 8, 16 or 32
  for (int base = 0; base < Lk; base += 4 * kThreads) {  // warp-uniform trip count: all lanes reach the shuffles
    const int j0 = base + 4 * (int)threadIdx.x;
    float sum = 0.f;
    for (int r = 0; r < bs; ++r) {
      const int i = I * bs + r;
      const int jend = causal ? min(Lk, i + 1 + off) : Lk;
      if (j0 < jend) {
        const float4 v = *reinterpret_cast<const float4 *>(acc + ((size_t)h * Lq + i) * Lk + j0);
        sum += v.x;
        if (j0 + 1 < jend) sum += v.y;
        if (j0 + 2 < jend) sum += v.z;
        if (j0 + 3 < jend) sum += v.w;
      }
    }
    for (int o = lanes_per_block >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((threadIdx.x & (lanes_per_block - 1)) == 0 && j0 < Lk) {
      const int J = j0 / bs;
      // entries of the block inside the domain: row i holds min(bs, max(0, jend - J*bs)) of them
      long long count = 0;
      for (int r = 0; r < bs; ++r) {
        const int i = I * bs + r;
        const int jend = causal ? min(Lk, i + 1 + off) : Lk;
        count += max(0, min(bs, jend - J * bs));
      }
      pooled[((size_t)h * nI + I) * nJ + J] = count ? sum / (float)count : 0.f;
    }
  }
}

// One thread per four consecutive mask bytes.
__global__ void __launch_bounds__(kThreads) expand_block_mask_kernel(const uint8_t *__restrict__ block_mask, int H,
                                                                     int Lq, int Lk, int bs, int causal,
                                                                     uint8_t *__restrict__ mask) {
  const int nI = Lq / bs, nJ = Lk / bs;
  const int off = causal ? Lk - Lq : 0;
  const long long quads = (long long)H * Lq * (Lk / 4);
  for (long long q = (long long)blockIdx.x * kThreads + threadIdx.x; q < quads; q += (long long)gridDim.x * kThreads) {
    const int j0 = (int)(q % (Lk / 4)) * 4;
    const long long row = q / (Lk / 4);
    const int i = (int)(row % Lq), h = (int)(row / Lq);
    const int jend = causal ? min(Lk, i + 1 + off) : Lk;
    const uint8_t keep = block_mask[((size_t)h * nI + i / bs) * nJ + j0 / bs];  // bs % 4 == 0: one block
    uchar4 out;
    out.x = (keep && j0 < jend) ? 1 : 0;
    out.y = (keep && j0 + 1 < jend) ? 1 : 0;
    out.z = (keep && j0 + 2 < jend) ? 1 : 0;
    out.w = (keep && j0 + 3 < jend) ? 1 : 0;
    *reinterpret_cast<uchar4 *>(mask + (size_t)row * Lk + j0) = out;
  }
}

}  // namespace

cudaError_t launch_pool_scores(const float *acc, int H, int Lq, int Lk, int bs, int causal, float *pooled,
                               cudaStream_t s) {
  pool_scores_kernel<<<dim3(Lq / bs, H), kThreads, 0, s>>>(acc, Lq, Lk, bs, causal, pooled);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_expand_block_mask(const uint8_t *block_mask, int H, int Lq, int Lk, int bs, int causal,
                                     uint8_t *mask, cudaStream_t s) {
  const long long quads = (long long)H * Lq * (Lk / 4);
  long long blocks = (quads + kThreads - 1) / kThreads;
  if (blocks > 148ll * 32) blocks = 148ll * 32;
  expand_block_mask_kernel<<<(unsigned)blocks, kThreads, 0, s>>>(block_mask, H, Lq, Lk, bs, causal, mask);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace ap
