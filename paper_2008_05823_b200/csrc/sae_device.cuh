// Device-side helpers shared by the kernels of libsae: tile plan, pinned fp32 arithmetic, the exact
// fixed-point L1 accumulator of the scaled-sign compressor (Eq. 2) and Top-K magnitude keys.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sae {

typedef unsigned long long u64;
typedef unsigned int u32;

#ifndef SAE_TILE
#define SAE_TILE 4096
#endif
#ifndef SAE_WORKER_MINBLOCKS
#define SAE_WORKER_MINBLOCKS 4
#endif
constexpr int TILE = SAE_TILE;   // elements of one tensor handled by one thread block
constexpr int THREADS = 256;     // threads per block: 8 warps
constexpr int VEC_ITERS = TILE / (THREADS * 4);   // float4 iterations per thread (4)
constexpr int ROWS = TILE / THREADS;              // scalar elements per thread (16)
constexpr int MAX_WORKERS = 1024;

constexpr u32 STATUS_RANGE = 1u;  // a model difference was non-finite or >= 2^32 in magnitude

// Segment / tile tables (device memory), passed to kernels by value.
// Internal ("padded") layout: tensor j starts at poff[j], a multiple of 32 elements, so that every
// tensor start is 128-byte aligned and owns whole bit words; padding elements stay zero.
struct Plan {
  int K, T;
  int k_pow2;            // K is a power of two: dividing by K is the exact multiplication by inv_k (same bits)
  float inv_k;           // 1 / K (exact when k_pow2)
  int ntiles;            // tiles over all tensors
  long long d;           // sum n_j (caller layout length)
  long long dpad;        // padded length, multiple of 32
  long long nwords;      // dpad / 32 = sum ceil(n_j/32)
  const int* tile_tensor;     // [ntiles] tensor of each tile
  const int* first_tile;      // [T] first tile of each tensor
  const int* n;               // [T] tensor sizes
  const long long* off;       // [T] caller-layout offsets
  const long long* poff;      // [T] padded offsets
};

struct TileInfo {
  int j;            // tensor
  int t0;           // first element of the tile inside the tensor
  int n;            // tensor size
  int cnt;          // valid elements in this tile (1..TILE)
  int tiles_j;      // number of tiles of this tensor
  long long off, poff;
};

__device__ __forceinline__ TileInfo tile_info(const Plan& P, int tile) {
  TileInfo ti;
  ti.j = P.tile_tensor[tile];
  ti.n = P.n[ti.j];
  ti.t0 = (tile - P.first_tile[ti.j]) * TILE;
  ti.cnt = min(TILE, ti.n - ti.t0);
  ti.tiles_j = (ti.n + TILE - 1) / TILE;
  ti.off = P.off[ti.j];
  ti.poff = P.poff[ti.j];
  return ti;
}

// acc / (float)K, one correctly rounded operation.  For a power-of-two K the product with 2^-log2(K) is the
// same real number as the quotient, so the cheaper multiply gives identical bits (denormals included).
__device__ __forceinline__ float div_by_k(const Plan& P, float a) {
  return P.k_pow2 ? __fmul_rn(a, P.inv_k) : __fdiv_rn(a, (float)P.K);
}

// ---- streaming loads/stores ------------------------------------------------------------------------
__device__ __forceinline__ float4 ld4_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

// ---- the scaled-sign code of one element -------------------------------------------------------------
__device__ __forceinline__ float sign_code(float v, float s) { return (v >= 0.0f) ? s : -s; }

// ---- Top-K ---------------------------------------------------------------------------------------
__device__ __forceinline__ u32 mag_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }
__device__ __forceinline__ bool topk_selected(float v, u32 tau) {
  u32 key = mag_key(v);
  return key >= tau && key != 0u;
}

// ---- exact L1: S = sum floor(|v| 2^64) as a 128-bit integer ----------------------------------------
struct Acc128 {
  u64 lo, hi;
  u32 bad;
};

__device__ __forceinline__ void acc_init(Acc128& a) { a.lo = 0; a.hi = 0; a.bad = 0; }

__device__ __forceinline__ void acc_add_u(Acc128& a, u64 lo, u64 hi) {
  a.lo += lo;
  a.hi += hi + (a.lo < lo ? 1ull : 0ull);
}

// |v| < 1: |v| * 2^64 is exact in fp32 (a power-of-two scaling that can neither overflow nor lose
// bits; denormals become normal) and the round-down conversion is the floor.  1 <= |v| < 2^32: integer
// part and fraction are split exactly first.  Anything else (including NaN/Inf) flags RANGE.
__device__ __forceinline__ void acc_add(Acc128& a, float v) {
  float m = fabsf(v);
  if (m < 1.0f) {
    u64 f = __float2ull_rd(__fmul_rn(m, 18446744073709551616.0f));
    a.lo += f;
    a.hi += (a.lo < f ? 1ull : 0ull);
  } else if (m < 4294967296.0f) {
    float ip = floorf(m);
    float fr = __fsub_rn(m, ip);
    acc_add_u(a, __float2ull_rd(__fmul_rn(fr, 18446744073709551616.0f)), __float2ull_rd(ip));
  } else {
    a.bad = 1u;
  }
}

__device__ __forceinline__ void acc_warp_reduce(Acc128& a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    u64 lo = __shfl_xor_sync(0xffffffffu, a.lo, o);
    u64 hi = __shfl_xor_sync(0xffffffffu, a.hi, o);
    u32 bad = __shfl_xor_sync(0xffffffffu, a.bad, o);
    acc_add_u(a, lo, hi);
    a.bad |= bad;
  }
}

// Block reduction; the result is valid in thread 0.  `sh` must hold 3 * (THREADS/32) u64.
__device__ __forceinline__ void acc_block_reduce(Acc128& a, u64* sh) {
  acc_warp_reduce(a);
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int NW = THREADS / 32;
  if (lane == 0) { sh[warp] = a.lo; sh[NW + warp] = a.hi; sh[2 * NW + warp] = a.bad; }
  __syncthreads();
  if (threadIdx.x == 0) {
    Acc128 r; acc_init(r);
    for (int w = 0; w < NW; ++w) { acc_add_u(r, sh[w], sh[NW + w]); r.bad |= (u32)sh[2 * NW + w]; }
    a = r;
  }
}

// Per-lane L1 accumulator of the streaming passes: a 96-bit sum (lo0, lo1, carry) fed by a three-instruction
// carry chain, plus a 64-bit word for the integer parts of the rare values >= 1.
struct LaneAcc {
  u32 lo0, lo1, carry;
  u64 hi;
  u32 bad;
};

__device__ __forceinline__ void lane_acc_init(LaneAcc& a) { a.lo0 = 0; a.lo1 = 0; a.carry = 0; a.hi = 0; a.bad = 0; }

// += floor(m 2^64) for 0 <= m < 1 (exact: power-of-two scaling, then a round-down conversion)
__device__ __forceinline__ void lane_add_small(LaneAcc& a, float m) {
  const u64 f = __float2ull_rd(__fmul_rn(m, 18446744073709551616.0f));
  const u32 f0 = (u32)f, f1 = (u32)(f >> 32);
  asm("add.cc.u32 %0, %0, %3;\n\taddc.cc.u32 %1, %1, %4;\n\taddc.u32 %2, %2, 0;"
      : "+r"(a.lo0), "+r"(a.lo1), "+r"(a.carry)
      : "r"(f0), "r"(f1));
}

// any magnitude: the general (rare) path splits off the integer part, non-finite / >= 2^32 flags RANGE
__device__ __forceinline__ void lane_add(LaneAcc& a, float v) {
  const float m = fabsf(v);
  if (m < 1.0f) {
    lane_add_small(a, m);
  } else if (m < 4294967296.0f) {
    const float ip = floorf(m);
    lane_add_small(a, __fsub_rn(m, ip));
    a.hi += __float2ull_rd(ip);
  } else {
    a.bad = 1u;
  }
}

// Four values at once: one test decides whether all of them are below 1 (the bit pattern of |v| orders
// magnitudes and puts NaN / Inf above every finite value), so the common case has no per-element branch.
__device__ __forceinline__ void lane_add4(LaneAcc& a, float4 v) {
  const u32 k0 = __float_as_uint(v.x) & 0x7fffffffu, k1 = __float_as_uint(v.y) & 0x7fffffffu;
  const u32 k2 = __float_as_uint(v.z) & 0x7fffffffu, k3 = __float_as_uint(v.w) & 0x7fffffffu;
  if (max(max(k0, k1), max(k2, k3)) < 0x3f800000u) {
    lane_add_small(a, __uint_as_float(k0)); lane_add_small(a, __uint_as_float(k1));
    lane_add_small(a, __uint_as_float(k2)); lane_add_small(a, __uint_as_float(k3));
  } else {
    lane_add(a, v.x); lane_add(a, v.y); lane_add(a, v.z); lane_add(a, v.w);
  }
}

// the lane's sum as a 128-bit value
__device__ __forceinline__ Acc128 lane_acc_total(const LaneAcc& a) {
  Acc128 r;
  r.lo = ((u64)a.lo1 << 32) | a.lo0;
  r.hi = a.hi + a.carry;
  r.bad = a.bad;
  return r;
}

// The per-(row, tensor) accumulator in global memory: three 43-bit limbs in 64-bit words (21 bits of
// headroom each, so integer atomicAdd from up to 2^21 tiles cannot overflow and the total does not
// depend on the order of arrival).  A later kernel turns the finished sum into the scale and clears
// the record for the next step.
struct L1Record {
  u64 limb[3];
  u64 pad;
};

constexpr u64 M43 = (1ull << 43) - 1;

// scale = (float)((double)(S truncated to its top 53 bits) / n * 2^-64)
__device__ __forceinline__ float scale_from_limbs(u64 l0, u64 l1, u64 l2, int n) {
  Acc128 s; acc_init(s);
  s.lo = l0;
  acc_add_u(s, l1 << 43, l1 >> 21);
  acc_add_u(s, 0ull, l2 << 22);
  if (s.lo == 0 && s.hi == 0) return 0.0f;
  int p = s.hi ? 127 - __clzll((long long)s.hi) : 63 - __clzll((long long)s.lo);
  u64 mant; int sh = 0;
  if (p > 52) {
    sh = p - 52;
    mant = (sh >= 64) ? (s.hi >> (sh - 64)) : ((s.lo >> sh) | (s.hi << (64 - sh)));   // sh in 1..75
  } else {
    mant = s.lo;
  }
  double Dd = ldexp((double)mant, sh);                  // exact: mant < 2^53
  double q = __ddiv_rn(Dd, (double)n);
  return __double2float_rn(q * 5.421010862427522e-20);  // 2^-64, exact scaling
}

// Adds one partial sum to a record: three fire-and-forget integer atomics (no ordering needed: the
// record is only read by a later kernel of the same stream).
__device__ __forceinline__ void l1_add_partial(const Acc128& a, L1Record* rec, u32* status) {
  if (a.bad) atomicOr(status, STATUS_RANGE);
  const u64 l0 = a.lo & M43;
  const u64 l1 = ((a.lo >> 43) | (a.hi << 21)) & M43;
  const u64 l2 = a.hi >> 22;
  if (l0) atomicAdd(&rec->limb[0], l0);
  if (l1) atomicAdd(&rec->limb[1], l1);
  if (l2) atomicAdd(&rec->limb[2], l2);
}

// Warp-level sum of the lanes' 128-bit partials, added by lane 0 to the (worker, tensor) record.
// The low 64 bits are split into 22-bit pieces so that a 32-lane sum fits a 32-bit redux add; the
// high word (almost always a small carry count) takes one more redux, or a shuffle tree if large.
__device__ __forceinline__ void warp_commit(const LaneAcc& a, L1Record* rec, u32* status) {
  const u32 full = 0xffffffffu;
  const u64 lo = ((u64)a.lo1 << 32) | a.lo0;
  const u32 r0 = __reduce_add_sync(full, (u32)(lo & 0x3fffffu));
  const u32 r1 = __reduce_add_sync(full, (u32)((lo >> 22) & 0x3fffffu));
  const u32 r2 = __reduce_add_sync(full, (u32)(lo >> 44));                   // 20 bits
  u64 hi = a.hi + a.carry;
  if (__any_sync(full, hi >> 24)) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) hi += __shfl_xor_sync(full, hi, o);
  } else {
    hi = __reduce_add_sync(full, (u32)hi);
  }
  const u32 bad = __any_sync(full, a.bad);
  if ((threadIdx.x & 31) == 0) {
    Acc128 s; acc_init(s);
    s.lo = r0;
    acc_add_u(s, (u64)r1 << 22, 0ull);
    acc_add_u(s, (u64)r2 << 44, hi + (u64)(r2 >> 20));
    s.bad = bad;
    l1_add_partial(s, rec, status);
  }
}

// ---- sign bits -----------------------------------------------------------------------------------
// Four consecutive elements per lane (lane l holds elements 4l..4l+3 of a 128-element row): the four
// words of the row are assembled by OR-ing nibbles across each group of 8 lanes.  Every lane of group
// g ends up holding word g.
__device__ __forceinline__ u32 pack_row4(bool p0, bool p1, bool p2, bool p3) {
  int lane = threadIdx.x & 31;
  u32 nib = (p0 ? 1u : 0u) | (p1 ? 2u : 0u) | (p2 ? 4u : 0u) | (p3 ? 8u : 0u);
  u32 w = nib << (4 * (lane & 7));
  w |= __shfl_xor_sync(0xffffffffu, w, 1);
  w |= __shfl_xor_sync(0xffffffffu, w, 2);
  w |= __shfl_xor_sync(0xffffffffu, w, 4);
  return w;
}

// ---- mbarrier / bulk-copy (TMA) primitives ----------------------------------------------------------
// Every wait on an mbarrier is bounded in time: a waiter that has polled for longer than the limit (the
// handle's, one second unless set otherwise) gives up, the caller raises STATUS_TIMEOUT in the handle's status
// word and the kernel returns; nothing traps and nothing spins without a limit.
constexpr u32 DEFAULT_WAIT_US = 1000000u;
constexpr u32 STATUS_TIMEOUT = 2u;

// How the kernels wait, passed by value with their arguments.
struct WaitCfg {
  u32 limit_us;       // 0 = DEFAULT_WAIT_US
  u32 drop_item;      // testing only: 1 + index of the work item whose copies the producer announces (expect_tx)
                      // but does not issue, so that the waits on it run out; 0 = none
};

__device__ __forceinline__ u32 smem_u32(const void* p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64* bar, u32 count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u64* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(u64* bar, u32 bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ u64 global_ns() {
  u64 t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// One poll: true when the phase with the given parity has completed.  (A poll that finds it incomplete suspends
// the thread for a hardware-defined time, a few microseconds on B200, or until the phase completes.)
__device__ __forceinline__ u32 mbar_try(u32 addr, u32 parity) {
  u32 done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(addr), "r"(parity)
      : "memory");
  return done;
}
// The path taken when the first poll came back empty-handed, kept out of line so that the kernels' hot loops
// carry a single poll instruction per wait (inlining the timed loop at every wait cost the three-array worker
// pass 16 %): polls on and gives up once the clock, read after every failed poll, shows the limit exceeded.
static __device__ __noinline__ bool mbar_wait_slow(u32 addr, u32 parity, u32 limit_us) {
  const u64 t0 = global_ns();
  const u64 limit_ns = (u64)(limit_us ? limit_us : DEFAULT_WAIT_US) * 1000ull;
  for (;;) {
    if (mbar_try(addr, parity)) return true;
    if (global_ns() - t0 > limit_ns) return false;
  }
}
// Bounded wait for the completion of the phase with the given parity; false = gave up.
__device__ __forceinline__ bool mbar_wait(u64* bar, u32 parity, const WaitCfg& wc) {
  const u32 addr = smem_u32(bar);
  if (mbar_try(addr, parity)) return true;
  return mbar_wait_slow(addr, parity, wc.limit_us);
}
// 1-D bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), completing on `bar`.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, u32 bytes, u64* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

}  // namespace sae
