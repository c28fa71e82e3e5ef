// CUDA side of the seeded synthetic input generator (the stand-in for back-propagation).  Produces
// the same bits as the numpy generator in synth.py; holds none of the method's arithmetic.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

typedef unsigned long long u64;

__host__ __device__ inline u64 mix64(u64 z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void k_fill(float* out, long long d, int rows, int T, const long long* __restrict__ ends,
                       const float* __restrict__ scales, u64 seed_mixed, u64 t, unsigned outlier_thresh,
                       float outlier_mult, float post_mult) {
  const long long total = d * rows;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < total;
       q += (long long)gridDim.x * blockDim.x) {
    const long long k = q / d, i = q - k * d;
    const u64 key = mix64(seed_mixed + t * 0xD1342543DE82EF95ull + (u64)k * 0xA0761D6478BD642Full);
    int total16 = 0;
    u64 h = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      h = mix64(key + ((u64)i * 4ull + (u64)r) * 0x9E3779B97F4A7C15ull);
      if (r < 3) total16 += (int)(h & 0xFFFF) + (int)((h >> 16) & 0xFFFF) + (int)((h >> 32) & 0xFFFF) + (int)(h >> 48);
    }
    const unsigned lane12 = (unsigned)(h & 0xFFFF);
    const float z = __fmul_rn((float)(total16 - 393210), 1.0f / 65536.0f);
    int lo = 0, hi = T - 1;                 // first tensor whose end exceeds i
    while (lo < hi) { int mid = (lo + hi) >> 1; if (ends[mid] > i) hi = mid; else lo = mid + 1; }
    float g = __fmul_rn(scales[lo], z);
    if (lane12 < outlier_thresh) g = __fmul_rn(g, outlier_mult);
    if (post_mult != 1.0f) g = __fmul_rn(post_mult, g);
    out[q] = g;
  }
}

}  // namespace

// out: device [rows][d]; ends: device [T] cumulative tensor ends; scales: device [T].
// Returns 0 or the cudaError_t of the launch.
extern "C" int sae_synth_fill(float* out, long long d, int rows, int T, const long long* ends, const float* scales,
                              unsigned long long seed_mixed, unsigned long long t, unsigned outlier_thresh,
                              float outlier_mult, float post_mult, void* stream) {
  const long long total = d * rows;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  if (blocks < 1) blocks = 1;
  k_fill<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(out, d, rows, T, ends, scales, seed_mixed, t,
                                                            outlier_thresh, outlier_mult, post_mult);
  return (int)cudaGetLastError();
}
