// sae_sign_compress_noalloc: the scaled-sign compressor (exact L1 + sign bit-pack) of one tensor for
// callers that must not allocate.  Declaration and contract: include/sae.h.
//
// The worker pass of the library accumulates its L1 partial sums in global scratch that sae_init
// allocates.  This variant keeps the scratch in a file-scope device array instead, so the call needs
// no cudaMalloc at all: one (lo, hi) partial per tile plus an arrival counter and a range flag.
#include "../../include/sae.h"
#include "sae_device.cuh"

#include <mutex>

using namespace sae;

#define SAE_NOALLOC_MAX_TILES 8192   // x TILE (4096) elements = 33 554 432 elements per call
#define SAE_NOALLOC_MAX_DEVICES 64

namespace {

constexpr int NA_COUNTER = 2 * SAE_NOALLOC_MAX_TILES;      // index of the arrival counter
constexpr int NA_FLAG = NA_COUNTER + 1;                    // index of the range flag
constexpr int NA_WORDS = NA_COUNTER + 32;                  // 128 KiB + 256 B, held by every GPU that loads the library

static __device__ __align__(256) unsigned long long g_noalloc_scratch[NA_WORDS];

// In host code `g_noalloc_scratch` is only a stand-in for the symbol; the device address is looked up
// once per device and cached here.
std::mutex g_mutex;
unsigned long long* g_scratch_addr[SAE_NOALLOC_MAX_DEVICES] = {nullptr};

__global__ void __launch_bounds__(THREADS) k_sign_compress_noalloc(const float* __restrict__ v, long long n, int ntiles,
                                                                   u32* __restrict__ words, float* scale,
                                                                   int* range_flag, u64* scratch) {
  __shared__ u64 sh_red[3 * (THREADS / 32)];
  __shared__ int sh_last;
  const int tile = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long t0 = (long long)tile * TILE;
  const int cnt = (int)min((long long)TILE, n - t0);
  const float* vp = v + t0;
  u32* wp = words + (t0 >> 5);
  Acc128 acc; acc_init(acc);
  if (cnt == TILE && (reinterpret_cast<uintptr_t>(vp) & 15) == 0) {
#pragma unroll
    for (int it = 0; it < VEC_ITERS; ++it) {
      const int i = it * (THREADS * 4) + tid * 4;
      const float4 d = ld4_stream(vp + i);
      acc_add(acc, d.x); acc_add(acc, d.y); acc_add(acc, d.z); acc_add(acc, d.w);
      const u32 w = pack_row4(d.x >= 0.0f, d.y >= 0.0f, d.z >= 0.0f, d.w >= 0.0f);
      if ((lane & 7) == 0) wp[i >> 5] = w;
    }
  } else {
    for (int r = 0; r < ROWS; ++r) {
      const int i = r * THREADS + tid;
      const bool valid = i < cnt;
      float d = 0.0f;
      if (valid) { d = vp[i]; acc_add(acc, d); }
      const u32 w = __ballot_sync(0xffffffffu, valid && d >= 0.0f);
      if (lane == 0 && (r * THREADS + warp * 32) < cnt) wp[(r * THREADS + warp * 32) >> 5] = w;
    }
  }
  acc_block_reduce(acc, sh_red);
  if (tid == 0) {
    scratch[2 * tile] = acc.lo;
    scratch[2 * tile + 1] = acc.hi;
    if (acc.bad) atomicOr((unsigned int*)(scratch + NA_FLAG), 1u);
    __threadfence();
    const u32 ticket = atomicAdd((unsigned int*)(scratch + NA_COUNTER), 1u);
    sh_last = (ticket == (u32)ntiles - 1u);
  }
  __syncthreads();
  if (!sh_last) return;
  // The block that arrived last adds every tile's partial (integers: any order gives the same sum).
  __threadfence();
  Acc128 tot; acc_init(tot);
  for (int t = tid; t < ntiles; t += THREADS) acc_add_u(tot, __ldcg(scratch + 2 * t), __ldcg(scratch + 2 * t + 1));
  __syncthreads();                    // sh_red is reused
  acc_block_reduce(tot, sh_red);
  if (tid == 0) {
    const u64 l0 = tot.lo & M43;
    const u64 l1 = ((tot.lo >> 43) | (tot.hi << 21)) & M43;
    const u64 l2 = tot.hi >> 22;
    *scale = scale_from_limbs(l0, l1, l2, (int)n);
    if (range_flag) *range_flag = (int)atomicExch((unsigned int*)(scratch + NA_FLAG), 0u);
    else atomicExch((unsigned int*)(scratch + NA_FLAG), 0u);
    atomicExch((unsigned int*)(scratch + NA_COUNTER), 0u);     // ready for the next call
  }
}

}  // namespace

extern "C" {

int64_t sae_noalloc_max_elements(void) { return (int64_t)SAE_NOALLOC_MAX_TILES * TILE; }

int sae_sign_compress_noalloc(const float* v, int64_t n, uint32_t* words, float* scale, int32_t* range_flag,
                              void* stream) {
  if (!v || !words || !scale || n < 1) return SAE_ERR_INVALID_ARG;
  if (n > sae_noalloc_max_elements()) return SAE_ERR_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= SAE_NOALLOC_MAX_DEVICES) { cudaGetLastError(); return SAE_ERR_CUDA; }
  unsigned long long* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
      // Set-up, once per device, with that device current: resolve the symbol to its device address.
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return SAE_ERR_CUDA; }
      g_scratch_addr[dev] = (unsigned long long*)p;
    }
    scratch = g_scratch_addr[dev];
  }
  cudaStream_t st = (cudaStream_t)stream;
  // The counter and the flag must start at zero even if an earlier call was cut short.
  if (cudaMemsetAsync(scratch + NA_COUNTER, 0, 2 * sizeof(unsigned long long), st) != cudaSuccess) {
    cudaGetLastError();
    return SAE_ERR_CUDA;
  }
  const int ntiles = (int)((n + TILE - 1) / TILE);
  k_sign_compress_noalloc<<<ntiles, THREADS, 0, st>>>(v, n, ntiles, words, scale, range_flag, scratch);
  if (cudaGetLastError() != cudaSuccess) return SAE_ERR_CUDA;
  return SAE_OK;
}

}  // extern "C"
