// Scores for the random-pruning control: entry n of the tensor is the top 24 bits of the
// (n+1)-th output of the SplitMix64 generator seeded with `seed`, scaled to [0, 1).  Output n+1
// is a function of seed and n alone (the state advances by a constant), so every thread computes
// its own entries; the mask builder then turns the scores into a random mask of exact count.
// Pure integer work up to the final conversion, which is exact (24 bits fit a float).
#include "ap_common.cuh"

namespace ap {

namespace {

__device__ __forceinline__ float score_of(unsigned long long seed, unsigned long long n) {
  unsigned long long z = seed + (n + 1ull) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z ^= z >> 31;
  return (float)(unsigned)(z >> 40) * (1.0f / 16777216.0f);
}

// A thread writes four consecutive entries at a time (one 16-byte store).
__global__ void __launch_bounds__(256) random_scores_kernel(float *__restrict__ out, unsigned long long count,
                                                            unsigned long long seed) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x * 4ull;
  for (unsigned long long n0 = ((unsigned long long)blockIdx.x * blockDim.x + threadIdx.x) * 4ull; n0 < count;
       n0 += stride) {
    if (n0 + 4ull <= count) {
      *reinterpret_cast<float4 *>(out + n0) =
          make_float4(score_of(seed, n0), score_of(seed, n0 + 1), score_of(seed, n0 + 2), score_of(seed, n0 + 3));
    } else {
      for (unsigned long long n = n0; n < count; ++n) out[n] = score_of(seed, n);
    }
  }
}

}  // namespace

cudaError_t launch_random_scores(float *out, int64_t count, uint64_t seed, cudaStream_t s) {
  const long long quads = (count + 3) / 4;
  long long blocks = (quads + 255) / 256;
  if (blocks > 148ll * 16) blocks = 148ll * 16;  // grid-stride beyond that
  random_scores_kernel<<<(unsigned)blocks, 256, 0, s>>>(out, (unsigned long long)count, (unsigned long long)seed);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace ap
