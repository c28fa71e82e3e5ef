// K1, the worker pass of Algorithm 1 (step-ahead point, local momentum, local model difference, exact
// L1 partials, sign bit-pack), as a persistent, warp-specialised kernel:
//
//   * grid = (#SMs x blocks per SM) persistent blocks; block b handles work items b, b+grid, ...
//     where item = (tile, worker) with the worker index fastest, so the K items that share one tile
//     of ebar / x run close together and share it through L2;
//   * one producer warp looks up the tile table for the items ahead and issues 1-D bulk asynchronous
//     copies (TMA, cp.async.bulk) of the gradient / momentum / error tiles into a ring of shared-memory
//     stages, each guarded by a "full" mbarrier (transaction bytes) and an "empty" mbarrier
//     (one arrival per consumer warp);
//   * consumer warps read their slice of a stage with 128-bit shared loads, compute, and store m / Delta
//     / sign words straight to global memory; each warp adds its own L1 partial to the (worker, tensor)
//     record (32-bit redux adds, then fire-and-forget integer atomics): no block-wide barrier, no
//     fence and no returned value anywhere in the loop.
//
// Ragged tails and gradient rows that are not 16-byte aligned cannot use bulk copies; for those items
// the producer only publishes the tile description and the consumers load from global memory.
//
// Every wait on an mbarrier is bounded: a waiter that has polled for longer than the handle's limit raises
// STATUS_TIMEOUT in the status word and leaves the loop; the producer, the last to leave, first waits (with the same
// bound) for the copies it still has in flight.
#pragma once
#include "sae_kernels.cuh"

namespace sae {

#ifndef SAE_WT_BLOCKS_PER_SM
#define SAE_WT_BLOCKS_PER_SM 1
#endif

#ifndef SAE_WT_CONSUMER_WARPS
#define SAE_WT_CONSUMER_WARPS 16
#endif
constexpr int WT_CONSUMER_WARPS = SAE_WT_CONSUMER_WARPS;
constexpr int WT_THREADS = WT_CONSUMER_WARPS * 32 + 32;     // + one producer warp
// Ring depth: three stages of 48 KB when the pass also writes the model differences (20 bytes per element:
// a fourth stage measured 1-2 % slower there), four when it moves 12 bytes per element (+2 %).
__host__ __device__ constexpr int wt_stages(bool write_d) { return write_d ? 3 : 4; }
constexpr int WT_SLICE = TILE / WT_CONSUMER_WARPS;          // elements of a tile owned by one consumer warp (256)
constexpr int WT_SLICE_ITERS = WT_SLICE / 128;              // float4 iterations per lane (2)
constexpr int WT_SLICE_ROWS = WT_SLICE / 32;                // scalar rows per warp (8)
static_assert(WT_SLICE % 128 == 0, "a consumer warp owns whole 128-element rows");

struct WtItem {          // description of one work item, written by the producer
  long long gofs;        // index of the tile's first gradient element in g
  long long pbase;       // index of the tile's first element in the [dpad] arrays
  long long wbase;       // ... in the [K][dpad] arrays
  int k, j, cnt, tiles_j, n, vec;
  float sprev;
  u32 tprev;
  u32 lo;               // Top-K: lower edge of the candidate window (NO_GUESS: collect nothing)
};

template <int STAGES>
struct WtSmemT {
  alignas(128) float buf[STAGES][3][TILE];   // [stage][g | m | e-source][element]
  alignas(8) u64 full[STAGES];
  alignas(8) u64 empty[STAGES];
  WtItem item[STAGES];
  u32 cstage[WT_CONSUMER_WARPS][CAND_STAGE];   // Top-K: per-warp staging of candidate keys
};

// Tile-table lookup of work item w (cnt = 0 marks "no such item").
template <int ESRC, bool TOPK>
__device__ __forceinline__ WtItem wt_lookup(const Plan& P, const WorkerArgs& A, long long w, long long nitems) {
  WtItem it;
  it.cnt = 0; it.vec = 0; it.gofs = 0; it.pbase = 0; it.wbase = 0; it.k = 0; it.j = 0; it.tiles_j = 0; it.n = 0;
  it.sprev = 0.0f; it.tprev = 0u; it.lo = NO_GUESS;
  if (w >= nitems) return it;
  const int tile = (int)(w / P.K);
  const int k = (int)(w - (long long)tile * P.K);
  const TileInfo ti = tile_info(P, tile);
  it.gofs = (long long)k * P.d + ti.off + ti.t0;
  it.pbase = ti.poff + ti.t0;
  it.wbase = (long long)k * P.dpad + it.pbase;
  it.k = k; it.j = ti.j; it.cnt = ti.cnt; it.tiles_j = ti.tiles_j; it.n = ti.n;
  if (ESRC == ESRC_LAZY_SIGN) it.sprev = A.scale_prev[(long long)k * P.T + ti.j];
  if (ESRC == ESRC_LAZY_TOPK || TOPK) it.tprev = A.tau_prev[(long long)k * P.T + ti.j];
  if (TOPK) it.lo = window_lo(it.tprev, A.cand.wlog2[ti.j]);
  it.vec = (ti.cnt == TILE) && ((reinterpret_cast<uintptr_t>(A.g + it.gofs) & 15) == 0);
  return it;
}

// MU0: momentum constant 0 (the SGD / SignSGD variants of Section 5): m^(k) is this step's gradient term and
// is not state, so the momentum rows are neither read nor written (12 instead of 20 bytes per element).
template <int ESRC, bool SIGN, bool WRITE_D, bool WD, bool TOPK, bool MU0 = false>
__global__ void __launch_bounds__(WT_THREADS, SAE_WT_BLOCKS_PER_SM) k_worker_tma(Plan P, StepParams sp, WorkerArgs A,
                                                                                  long long nitems) {
  extern __shared__ unsigned char smem_raw[];
  constexpr int WT_STAGES = wt_stages(WRITE_D);
  using WtSmem = WtSmemT<WT_STAGES>;
  WtSmem& S = *reinterpret_cast<WtSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < WT_STAGES; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], WT_CONSUMER_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == WT_CONSUMER_WARPS) {
    // ---------------- producer ----------------
    // The tile-table lookups cost a few dependent global loads, so the warp does them for 32 items at
    // a time (lane l looks up the l-th item of the batch, and the next batch is fetched while this
    // one is being issued); the lanes then take turns, in item order, to publish and issue.
    const long long G = gridDim.x;
    long long wb = blockIdx.x;                               // first item of the current batch
    WtItem nxt = wt_lookup<ESRC, TOPK>(P, A, wb + lane * G, nitems);
    for (int i0 = 0; wb < nitems; i0 += 32, wb += 32 * G) {
      const WtItem cur = nxt;
      nxt = wt_lookup<ESRC, TOPK>(P, A, wb + (32 + lane) * G, nitems);
      bool ok = true;
      for (int l = 0; l < 32; ++l) {
        if (lane == l && cur.cnt > 0) {
          const int i = i0 + l;
          const int s = i % WT_STAGES;
          if (i >= WT_STAGES && !mbar_wait(&S.empty[s], ((i / WT_STAGES) - 1) & 1, A.wc)) {
            atomicOr(A.status, STATUS_TIMEOUT);
            ok = false;
          } else {
            S.item[s] = cur;
            if (cur.vec) {
              constexpr u32 B = TILE * sizeof(float);
              mbar_arrive_expect_tx(&S.full[s], (MU0 ? 2 : 3) * B);
              if (A.wc.drop_item != (u32)(wb + l * G) + 1u) {
                bulk_load(S.buf[s][0], A.g + cur.gofs, B, &S.full[s]);
                if (!MU0) bulk_load(S.buf[s][1], A.m + cur.wbase, B, &S.full[s]);
                bulk_load(S.buf[s][2], (ESRC == ESRC_UNIFORM) ? (A.ebar + cur.pbase) : (A.D + cur.wbase), B,
                          &S.full[s]);
              }
            } else {
              mbar_arrive(&S.full[s]);
            }
          }
        }
        __syncwarp();
        if (!__all_sync(0xffffffffu, ok)) {
          // Gave up on item i0 + l.  The consumers never release a stage again; before this warp -- the last
          // one to leave -- returns, it waits (bounded) for the copies already on their way into each stage.
          if (lane < WT_STAGES) {
            const int last = i0 + l - 1;                           // last item issued
            const int j = last - ((last - lane) % WT_STAGES + WT_STAGES) % WT_STAGES;   // ... into stage `lane`
            if (last >= 0 && j >= 0) mbar_wait(&S.full[lane], (j / WT_STAGES) & 1, A.wc);
          }
          return;
        }
      }
    }
    return;
  }

  // ---------------- consumers ----------------
  // A warp keeps adding to its L1 partial while consecutive items belong to the same (worker, tensor)
  // -- with a grid that is a multiple of K every item of a block has the same worker -- and commits
  // when that changes: the commit (atomics plus a fence) is then off the per-item path.
  LaneAcc acc; lane_acc_init(acc);
  int acc_k = 0, acc_j = 0;
  u32 acc_items = 0;
  // Top-K: candidate keys are staged per warp and appended to the (worker, tensor) list in batches
  WarpStage stg; stg.buf = S.cstage[warp]; stg.n = 0;
  int stg_k = 0, stg_j = 0;
  long long w = blockIdx.x;
  for (int i = 0; w < nitems; ++i, w += gridDim.x) {
    const int s = i % WT_STAGES;
    if (!mbar_wait(&S.full[s], (i / WT_STAGES) & 1, A.wc)) {
      if (lane == 0) atomicOr(A.status, STATUS_TIMEOUT);
      return;
    }
    const WtItem it = S.item[s];
    float* __restrict__ mp = A.m + it.wbase;
    float* dp = A.D + it.wbase;
    u32* wp = A.words + (long long)it.k * P.nwords + (it.pbase >> 5);
    if (TOPK) {
      if (it.k != stg_k || it.j != stg_j) { stage_flush(stg, A.cand, stg_k, stg_j); stg_k = it.k; stg_j = it.j; }
    }
    if (SIGN) {
      if (acc_items && (it.k != acc_k || it.j != acc_j)) {
        warp_commit(acc, A.recs + (long long)acc_k * P.T + acc_j, A.status);
        lane_acc_init(acc); acc_items = 0;
      }
      acc_k = it.k; acc_j = it.j; acc_items += 1;
    }
    const int base = warp * WT_SLICE;
    if (it.vec) {
      const float* __restrict__ xp = A.x + it.pbase;
      const float* sg = S.buf[s][0];
      const float* sm = S.buf[s][1];
      const float* se = S.buf[s][2];
#pragma unroll
      for (int q = 0; q < WT_SLICE_ITERS; ++q) {
        const int e0 = base + q * 128 + lane * 4;
        const float4 G = *reinterpret_cast<const float4*>(sg + e0);
        float4 M = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!MU0) M = *reinterpret_cast<const float4*>(sm + e0);
        const float4 E = *reinterpret_cast<const float4*>(se + e0);
        float4 X = make_float4(0.f, 0.f, 0.f, 0.f);
        if (WD) X = ld4(xp + e0);
        float4 mn, dl;
        dl.x = worker_update<WD>(G.x, M.x, prev_error<ESRC>(E.x, it.sprev, it.tprev), X.x, sp, mn.x);
        dl.y = worker_update<WD>(G.y, M.y, prev_error<ESRC>(E.y, it.sprev, it.tprev), X.y, sp, mn.y);
        dl.z = worker_update<WD>(G.z, M.z, prev_error<ESRC>(E.z, it.sprev, it.tprev), X.z, sp, mn.z);
        dl.w = worker_update<WD>(G.w, M.w, prev_error<ESRC>(E.w, it.sprev, it.tprev), X.w, sp, mn.w);
        if (!MU0) st4(mp + e0, mn);
        if (WRITE_D) st4(dp + e0, dl);
        if (TOPK && it.lo != NO_GUESS) {
          if (stg.n > CAND_STAGE - 128) stage_flush(stg, A.cand, stg_k, stg_j);
          stage_row4(stg, it.lo, mag_key(dl.x), mag_key(dl.y), mag_key(dl.z), mag_key(dl.w));
        }
        if (SIGN) {
          lane_add4(acc, dl);
          const u32 wd = pack_row4(dl.x >= 0.0f, dl.y >= 0.0f, dl.z >= 0.0f, dl.w >= 0.0f);
          if ((lane & 7) == 0) wp[e0 >> 5] = wd;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&S.empty[s]);
    } else {
      // the stage carries no data for this item: release it at once, then work from global memory
      __syncwarp();
      if (lane == 0) mbar_arrive(&S.empty[s]);
      const float* __restrict__ gp = A.g + it.gofs;
      const float* __restrict__ ebp = A.ebar + it.pbase;
      const float* __restrict__ xp = A.x + it.pbase;
#pragma unroll 4
      for (int r = 0; r < WT_SLICE_ROWS; ++r) {
        const int e0 = base + r * 32 + lane;
        const bool valid = e0 < it.cnt;
        float dl = 0.0f;
        if (valid) {
          const float e = prev_error<ESRC>((ESRC == ESRC_UNIFORM) ? ebp[e0] : dp[e0], it.sprev, it.tprev);
          const float xv = WD ? xp[e0] : 0.0f;
          float mn;
          dl = worker_update<WD>(__ldcs(gp + e0), MU0 ? 0.0f : mp[e0], e, xv, sp, mn);
          if (!MU0) mp[e0] = mn;
          if (WRITE_D) dp[e0] = dl;
          if (SIGN) lane_add(acc, dl);
        }
        if (TOPK && it.lo != NO_GUESS) {
          if (stg.n > CAND_STAGE - 32) stage_flush(stg, A.cand, stg_k, stg_j);
          stage_row1(stg, it.lo, valid, mag_key(dl));
        }
        if (SIGN) {
          const u32 wd = __ballot_sync(0xffffffffu, valid && dl >= 0.0f);
          if (lane == 0 && (base + r * 32) < it.cnt) wp[(base + r * 32) >> 5] = wd;
        }
      }
    }
  }
  if (SIGN && acc_items) warp_commit(acc, A.recs + (long long)acc_k * P.T + acc_j, A.status);
  if (TOPK) stage_flush(stg, A.cand, stg_k, stg_j);
}

}  // namespace sae
