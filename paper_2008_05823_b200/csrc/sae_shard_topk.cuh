// Sharded operation with the Top-K compressor (Section 3.1): the message of worker k for tensor j is the
// list of its selected entries, (index inside the tensor, value) pairs -- what Algorithm 1 sends to the
// server.  The owner compacts its workers' selections into such lists after the thresholds are known;
// every shard then adds the lists of ALL workers in k order, reading them in place from their owners.
//
// Why the sparse sum is exact: the worker-axis sum of Algorithm 1's server line runs k = 0..K-1 from +0 over
// C(Delta^(k))_i, and an unselected entry contributes an exact +0, which leaves a running fp32 sum unchanged;
// so the ordered sum over the workers that selected i is the full ordered sum, bit for bit.
#pragma once
#include "sae_topk.cuh"

namespace sae {

// ---- owner side: compact the selected entries of the local workers ---------------------------------
struct SparseMsgArgs {
  const float* D;               // [K_loc][dpad] stored model differences
  const u32* tau;               // [K_loc][T] this step's thresholds
  unsigned long long* entries;  // [K_loc][stride]: value bits << 32 | index inside the tensor
  const long long* off;         // [T] start of tensor j's region inside a row
  const int* cap;               // [T] capacity of that region
  long long stride;
  u32* count;                   // [K_loc][T] entries appended (may exceed cap: the list then counts as overflowed)
};

// One block per (tile, local worker): one atomic per block reserves the block's slots.
__global__ void __launch_bounds__(THREADS) k_topk_compact(Plan P, SparseMsgArgs A) {
  __shared__ u32 cnt_wr[ROWS][THREADS / 32];   // selected entries of warp w in row r
  __shared__ u32 pre_wr[ROWS][THREADS / 32];   // exclusive prefix in (r, w) order
  __shared__ u32 sh_base;
  const int tile = blockIdx.x / P.K, k = blockIdx.x - tile * P.K;
  const TileInfo ti = tile_info(P, tile);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 t = A.tau[(long long)k * P.T + ti.j];
  const float* __restrict__ dp = A.D + (long long)k * P.dpad + ti.poff + ti.t0;
  u32 mine = 0;                                 // bit r: my element of row r is selected
  for (int r = 0; r < ROWS; ++r) {
    const int i = r * THREADS + tid;
    const bool q = i < ti.cnt && topk_selected(dp[i], t);
    const u32 b = __ballot_sync(0xffffffffu, q);
    if (q) mine |= 1u << r;
    if (lane == 0) cnt_wr[r][warp] = (u32)__popc(b);
  }
  __syncthreads();
  if (warp == 0) {
    // exclusive prefix over the ROWS x 8 counts in (r, w) order: four consecutive counts per lane
    constexpr int NV = ROWS * (THREADS / 32);          // 128
    static_assert(NV == 128, "four counts per lane");
    u32* flat_c = &cnt_wr[0][0];
    u32* flat_p = &pre_wr[0][0];
    const u32 c0 = flat_c[4 * lane], c1 = flat_c[4 * lane + 1], c2 = flat_c[4 * lane + 2], c3 = flat_c[4 * lane + 3];
    const u32 sum = c0 + c1 + c2 + c3;
    u32 inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const u32 v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const u32 ex = inc - sum;
    flat_p[4 * lane] = ex; flat_p[4 * lane + 1] = ex + c0; flat_p[4 * lane + 2] = ex + c0 + c1;
    flat_p[4 * lane + 3] = ex + c0 + c1 + c2;
    const u32 total = __shfl_sync(0xffffffffu, inc, 31);
    if (lane == 0) sh_base = total ? atomicAdd(A.count + (long long)k * P.T + ti.j, total) : 0u;
  }
  __syncthreads();
  if (mine == 0u && __ballot_sync(0xffffffffu, mine != 0u) == 0u) return;   // (whole warp idle)
  const u32 base = sh_base, cap = (u32)A.cap[ti.j];
  unsigned long long* dst = A.entries + (long long)k * A.stride + A.off[ti.j];
  for (int r = 0; r < ROWS; ++r) {
    const bool q = (mine >> r) & 1u;
    const u32 b = __ballot_sync(0xffffffffu, q);
    if (q) {
      const u32 pos = base + pre_wr[r][warp] + (u32)__popc(b & ((1u << lane) - 1u));
      const int i = r * THREADS + tid;
      if (pos < cap)
        dst[pos] = ((unsigned long long)__float_as_uint(dp[i]) << 32) | (unsigned long long)(u32)(ti.t0 + i);
    }
  }
}

// ---- every shard: the ordered worker-axis sum from all owners' lists --------------------------------
struct SparseAggArgs {
  float* e_srv;                                   // [dpad] in: e, out: Delta = e + (1/K) sum_k C(Delta^(k))
  float* acc;                                     // [dpad] scratch, all zero on entry and on exit
  const unsigned long long* const* entry_rows;    // [K] -> worker k's [stride] entries (at its owner)
  const u32* const* count_rows;                   // [K] -> worker k's [T] counts
  const float* const* d_rows;                     // [K] -> worker k's [dpad] differences (overflowed lists only)
  const u32* const* tau_rows;                     // [K] -> worker k's [T] thresholds of this step (likewise)
  const long long* off;
  const int* cap;
};

constexpr int AGG_THREADS = 1024;
constexpr int AGG_TILES = 16;          // consecutive plan tiles (65 536 elements) owned by one block

// A block owns the elements of AGG_TILES consecutive tiles, tensor by tensor.  For k = 0..K-1 in turn (a
// block barrier between workers keeps the order per element) it scans worker k's list of the tensor and
// adds the entries that fall into its range into the scratch sum; a second sweep over the same entries
// turns every touched element into Delta = e + sum / K and returns the scratch to zero.  Every block of a
// large tensor scans that tensor's whole lists (they are short and stay in L2); ranges never overlap, so
// no two blocks touch the same element.  A list that overflowed its region is replaced by a pass over the
// range of that worker's stored row with its threshold.
__global__ void __launch_bounds__(AGG_THREADS) k_topk_sparse_aggregate(Plan P, SparseAggArgs A) {
  const int tid = threadIdx.x;
  const int tile0 = blockIdx.x * AGG_TILES;
  const int tile1 = min(P.ntiles, tile0 + AGG_TILES);
  int tile = tile0;
  while (tile < tile1) {
    // the run of this block's tiles that belong to one tensor: elements [lo, hi) of tensor j
    const TileInfo ti = tile_info(P, tile);
    const int j = ti.j;
    const int last = min(tile1, tile + (ti.tiles_j - (ti.t0 / TILE)));     // one past the run's last tile
    const u32 lo = (u32)ti.t0;
    const u32 hi = (u32)min((long long)ti.n, (long long)ti.t0 + (long long)(last - tile) * TILE);
    tile = last;
    float* acc = A.acc + ti.poff;
    float* es = A.e_srv + ti.poff;
    const u32 cap = (u32)A.cap[j];
    for (int pass = 0; pass < 2; ++pass) {
      for (int k = 0; k < P.K; ++k) {
        const u32 cnt = A.count_rows[k][j];
        if (cnt <= cap) {
          const unsigned long long* __restrict__ en = A.entry_rows[k] + A.off[j];
          for (u32 e = tid; e < cnt; e += AGG_THREADS) {
            const unsigned long long v = en[e];
            const u32 idx = (u32)v;
            if (idx < lo || idx >= hi) continue;
            if (pass == 0) {
              acc[idx] = __fadd_rn(acc[idx], __uint_as_float((u32)(v >> 32)));
            } else {
              const float s = acc[idx];
              if (s != 0.0f) { es[idx] = __fadd_rn(es[idx], div_by_k(P, s)); acc[idx] = 0.0f; }
            }
          }
        } else {
          const u32 t = A.tau_rows[k][j];
          const float* __restrict__ dp = A.d_rows[k] + ti.poff;
          for (u32 i = lo + tid; i < hi; i += AGG_THREADS) {
            const float v = dp[i];
            if (!topk_selected(v, t)) continue;
            if (pass == 0) {
              acc[i] = __fadd_rn(acc[i], v);
            } else {
              const float s = acc[i];
              if (s != 0.0f) { es[i] = __fadd_rn(es[i], div_by_k(P, s)); acc[i] = 0.0f; }
            }
          }
        }
        __syncthreads();
      }
    }
  }
}

// Double-way: the server's candidate keys of Delta (the dense server pass collects them on the way; here
// the sum was sparse, so the window scan is a pass of its own over the d-vector).
__global__ void __launch_bounds__(THREADS) k_server_candidates(Plan P, const float* __restrict__ delta, CandArgs C,
                                                               const u32* __restrict__ tau_srv_prev) {
  __shared__ u32 cstage[(THREADS / 32) * CAND_STAGE];
  const TileInfo ti = tile_info(P, blockIdx.x);
  const int tid = threadIdx.x;
  const u32 lo = window_lo(tau_srv_prev[ti.j], C.wlog2[ti.j]);
  if (lo == NO_GUESS) return;
  WarpStage stg; stg.buf = cstage + (tid >> 5) * CAND_STAGE; stg.n = 0;
  const float* __restrict__ dp = delta + ti.poff + ti.t0;
  for (int r = 0; r < ROWS; ++r) {
    const int i = r * THREADS + tid;
    const bool valid = i < ti.cnt;
    if (stg.n > CAND_STAGE - 32) stage_flush(stg, C, 0, ti.j);
    stage_row1(stg, lo, valid, valid ? mag_key(dp[i]) : 0u);
  }
  stage_flush(stg, C, 0, ti.j);
}

}  // namespace sae
