// Worker pass with the pending error averaging folded in (scaled sign, averaging period 1).
//
// With p = 1 every step ends with "average the local errors" (Algorithm 1, pre-step):
//     ebar' = (1/K) sum_k ( Delta^(k) - C(Delta^(k)) ),     Delta^(k) = fma(eta, m^(k), ebar).
// Doing that in the apply kernel costs a second read of all K momentum rows.  This kernel instead
// leaves the average pending and computes it at the head of the NEXT step's worker pass, which has to
// read the same momentum rows anyway:
//   averaging (per tile, all K workers): ebar' from the rows of m in shared memory, k = 0..K-1 in order,
//            with last step's learning rate and scales (same fused op, same order: same bits);
//   worker lines with e^(k) = ebar': momentum, Delta, exact L1 partials, sign words.
// The two are done by different warps: four "averager" warps run one tile ahead of sixteen "worker"
// warps and hand each tile over through an mbarrier, so the averaging overlaps the worker lines.
// One block handles a tile for ALL workers: the producer warp brings the tile of all K momentum rows in
// with 2-D tensor-map TMA copies (one request per box of up to 256 elements x K rows -- per-row copies of
// 1-2 KB each were limited by the per-request cost), likewise the K gradient rows when the caller's
// layout allows a tensor map (16-byte aligned base and row pitch), and the ebar tile with a 1-D bulk
// copy; 3- or 6-stage ring (by K), full/empty mbarriers.  The consumers touch global memory only to store.
// In phase B a consumer warp always works for the same worker(s), so it carries their L1 partials
// across tiles and adds them to the (worker, tensor) records only when the tensor changes.
// All waits are bounded (STATUS_TIMEOUT).
#pragma once
#include "sae_worker_tma.cuh"
#include <cuda.h>

namespace sae {

constexpr int FW_WARPS = 16;                       // worker warps (warps 0..15)
#ifndef SAE_FW_AVG_WARPS
#define SAE_FW_AVG_WARPS 4
#endif
constexpr int FW_AVG_WARPS = SAE_FW_AVG_WARPS;     // averager warps (warps 17..); warp 16 is the producer
constexpr int FW_THREADS = (FW_WARPS + 1 + FW_AVG_WARPS) * 32;
constexpr int FW_MAXTILE = 2048;
constexpr int FW_MAXBOX = 256;                     // inner extent of a TMA box (the hardware limit)
// From this many workers on, an item is half as large and the ring twice as deep (6 stages of 2 x 16 KB
// instead of 3 of 2 x 32 KB): with few, large stages the copies in flight -- (stages - 1) x stage size --
// do not cover the memory latency at full bandwidth.
#ifndef SAE_FW_SPLIT_K
#define SAE_FW_SPLIT_K 16
#endif
// K = 32: a stage of all 32 rows x 256 elements is 2 x 32 KB, so only three fit; the element range is
// instead handled as two consecutive items of 16 workers each (boxes of 16 rows), which makes the stages
// half as large without shortening the 1 KB box rows (512-byte rows were slower).
#ifndef SAE_FW_HALVES32
#define SAE_FW_HALVES32 2
#endif
constexpr int fw_halves(int K) { return K == 32 ? SAE_FW_HALVES32 : 1; }
constexpr int fw_kh(int K) { return K / fw_halves(K); }                         // workers (box rows) per item
constexpr bool fw_split(int K) { return (K >= SAE_FW_SPLIT_K && K <= 16) || fw_halves(K) > 1; }
constexpr int fw_mbuf(int K) { return fw_split(K) ? 4096 : 8192; }   // floats of momentum (and gradient) per stage
constexpr int fw_stages(int K) { return fw_split(K) ? 6 : 3; }
constexpr int fw_tilef(int K) { return (fw_mbuf(K) / fw_kh(K)) < FW_MAXTILE ? (fw_mbuf(K) / fw_kh(K)) : FW_MAXTILE; }
constexpr int fw_box(int K) { return fw_tilef(K) < FW_MAXBOX ? fw_tilef(K) : FW_MAXBOX; }

// MODE 0: scaled sign (folded averaging); 1: Top-K with p = 1 (folded tail, differences not stored);
// 2: Top-K with stored differences (folded tail; a stage carries three arrays -- momentum, gradient and
// stored difference rows -- so the stages are 3 x 16 KB and there are four of them).
template <int K, int MODE = 0>
struct FwGeom {
  static constexpr int HALVES = fw_halves(K);                 // items per element range
  static constexpr int KH = fw_kh(K);                         // workers per item
  static constexpr int MBUF = MODE == 2 ? 4096 : fw_mbuf(K);
  static constexpr int STAGES = MODE == 2 ? 4 : fw_stages(K);
  static constexpr int TILEF = (MBUF / KH) < FW_MAXTILE ? (MBUF / KH) : FW_MAXTILE;   // elements per item
  static constexpr int BOX = TILEF < FW_MAXBOX ? TILEF : FW_MAXBOX;                  // inner extent of the TMA boxes
  static_assert(BOX == fw_box(K), "one tensor map per array serves every mode");
  static constexpr int SUB = TILE / TILEF;                    // element ranges per 4096-element plan tile
  static constexpr int ROWS_PER_WORKER = TILEF / 128;
  static constexpr int RPW = KH * ROWS_PER_WORKER / FW_WARPS; // 128-element rows per warp and item
  static constexpr int WPW = RPW > ROWS_PER_WORKER ? RPW / ROWS_PER_WORKER : 1;   // workers per warp and item
  static constexpr int NACC = WPW * HALVES;                   // workers a warp ever works for
  static_assert(K >= 1 && K <= 32 && (K & (K - 1)) == 0, "power-of-two worker counts up to 32");
  static constexpr int CHUNKS = TILEF / BOX;                  // TMA boxes per array and item
  static_assert(RPW >= 1 && NACC <= 2 && CHUNKS >= 1 && BOX % 128 == 0 && STAGES % HALVES == 0, "geometry");
  // position of element e of the item's worker kl inside a stage buffer: boxes of [KH][BOX] one after the other
  __device__ static __forceinline__ int idx(int kl, int e) { return (e / BOX) * (KH * BOX) + kl * BOX + (e % BOX); }
};

// 2-D tiled TMA load of one box at element coordinates (x, y), completing on `bar`.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, u64* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(reinterpret_cast<unsigned long long>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

struct FwItem {
  long long pbase;   // first element in the [dpad] arrays
  long long goff;    // first element inside a gradient row (caller layout)
  int j, cnt, gvec;  // tensor, valid elements (0 = empty item), gradient tile fetched by TMA into the stage
  int h;             // which group of KH workers
};

template <int K, int MODE = 0>
struct FwSmemT {
  typedef FwGeom<K, MODE> G;
  static constexpr bool TOPK = MODE != 0;
  alignas(128) float m[G::STAGES][G::MBUF];
  alignas(128) float g[G::STAGES][G::MBUF];
  alignas(128) float dd[MODE == 2 ? G::STAGES : 1][MODE == 2 ? G::MBUF : 32];   // stored differences (MODE 2)
  alignas(128) float e[G::STAGES][G::TILEF];
  alignas(8) u64 full[G::STAGES];
  alignas(8) u64 empty[G::STAGES];
  alignas(8) u64 avgd[G::STAGES];   // "ebar' of this stage is ready": one arrival per averager warp
  FwItem item[G::STAGES];
  float sc[G::STAGES][32];      // last step's scales (Top-K: threshold bit patterns) of the item's tensor, one per worker
  u32 cstage[TOPK ? FW_WARPS : 1][TOPK ? CAND_STAGE : 1];   // Top-K: per-warp staging of candidate keys
};

struct FusedArgs {
  const float* g;
  float* m;
  float* ebar;             // in: ebar of the previous step
  float* ebar_out;         // out: the averaged error of this pre-step (scaled sign: the same buffer)
  const u32* tau_prev;     // Top-K: [K][T] thresholds of the previous step
  float* D;                // Top-K with stored differences: [K][dpad] in: last step's, out: this step's
  float* ssum;             // [dpad] out: sum_k C(Delta^(k)) of the previous step, k in order, not divided by K
                           // (Top-K: always; scaled sign: when not null)
  CandArgs cand;           // Top-K: candidate lists for this step's differences
  const float* x;
  const float* scale_prev; // [K][T] scales of the previous step
  u32* words;
  L1Record* recs;
  u32* status;
  float eta_prev;
  int g_tma_ok;            // the gradient buffer admits a tensor map (16-byte aligned base and row pitch)
  WaitCfg wc;
};

template <int K, int MODE>
__device__ __forceinline__ FwItem fw_lookup(const Plan& P, int g_tma_ok, long long w, long long nitems) {
  typedef FwGeom<K, MODE> G;
  FwItem it;
  it.pbase = 0; it.goff = 0; it.j = 0; it.cnt = 0; it.gvec = 0; it.h = 0;
  if (w >= nitems) { it.cnt = -1; return it; }
  const int tile = (int)(w / G::SUB);
  const int sub = (int)(w - (long long)tile * G::SUB);
  const TileInfo ti = tile_info(P, tile);
  const int t0 = ti.t0 + sub * G::TILEF;
  const int cnt = min(G::TILEF, ti.n - t0);
  if (cnt <= 0) return it;
  it.j = ti.j; it.cnt = cnt;
  it.pbase = ti.poff + t0;
  it.goff = ti.off + t0;
  it.gvec = g_tma_ok && ((it.goff & 3) == 0);
  return it;
}

// The q-th element range of block b: the blocks take runs of `chunk` consecutive ranges in turn.  With runs
// of one plan tile (chunk = SUB) the consecutive ranges of a block mostly belong to the same tensor even when
// the tensors are single tiles (block-wise compression), so the L1 partials are committed once per run
// instead of once per range; chunk = 1 (long tensors, small problems) deals the ranges out one by one.
// (chunk = 2^chunk_log2)
__device__ __forceinline__ long long fw_range_of(int q, int chunk_log2) {
  return (((long long)(q >> chunk_log2) * gridDim.x + blockIdx.x) << chunk_log2) + (q & ((1 << chunk_log2) - 1));
}
// how many ranges this block takes in all
__device__ __forceinline__ int fw_ranges_of_block(long long nitems, int chunk_log2) {
  const long long cycle = (long long)gridDim.x << chunk_log2;
  const long long full = nitems / cycle;
  const long long rest = nitems - full * cycle - ((long long)blockIdx.x << chunk_log2);
  const long long tail = rest < 0 ? 0 : (rest > (1LL << chunk_log2) ? (1LL << chunk_log2) : rest);
  return (int)((full << chunk_log2) + tail);
}

// TOPK (Top-K, p = 1, K = 8 or 16): the same structure with the compressor changed.  The averagers apply the
// previous step's thresholds instead of its scales and also form that step's ordered worker-axis sum of the
// selected entries (the aggregation of the server line: it needs the same rows in the same order), which a
// parameter-sized server pass then only reads; the workers collect this step's candidate keys instead of L1
// partials and sign bits.  The differences are never stored.
template <int K, bool WD, int MODE = 0>
__global__ void __launch_bounds__(FW_THREADS, 1) k_worker_fused(Plan P, StepParams sp, FusedArgs A, long long nitems,
                                                                 int chunk_log2,
                                                                 const __grid_constant__ CUtensorMap tm_m,
                                                                 const __grid_constant__ CUtensorMap tm_g,
                                                                 const __grid_constant__ CUtensorMap tm_d) {
  typedef FwGeom<K, MODE> G;
  constexpr bool TOPK = MODE != 0, GEN = MODE == 2;
  extern __shared__ unsigned char smem_raw[];
  typedef FwSmemT<K, MODE> Smem;
  static_assert(!TOPK || (G::WPW == 1 && G::HALVES == 1), "Top-K form: a worker warp serves one worker");
  constexpr int FW_STAGES = G::STAGES;
  constexpr int FW_BOX = G::BOX;
  Smem& S = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nmine = fw_ranges_of_block(nitems, chunk_log2);
  if (tid == 0) {
    for (int s = 0; s < FW_STAGES; ++s) {
      mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], FW_WARPS); mbar_init(&S.avgd[s], FW_AVG_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == FW_WARPS) {
    // ---------------- producer ----------------
    // nitems counts element ranges; each is issued as HALVES consecutive items (one per group of KH workers)
    FwItem nxt = fw_lookup<K, MODE>(P, A.g_tma_ok, fw_range_of(lane, chunk_log2), nitems);
    for (int p0 = 0; p0 < nmine; p0 += 32) {
      const FwItem cur = nxt;
      nxt = fw_lookup<K, MODE>(P, A.g_tma_ok, fw_range_of(p0 + 32 + lane, chunk_log2), nitems);
      for (int l = 0; l < 32; ++l) {
        // the range of lane l, broadcast so that the lanes can share the issue of its copies
        const int cnt = __shfl_sync(0xffffffffu, cur.cnt, l);
        if (cnt < 0) break;                                   // past the last range (uniform)
        const long long pbase = __shfl_sync(0xffffffffu, cur.pbase, l);
        const int j = __shfl_sync(0xffffffffu, cur.j, l);
        const int gtma = __shfl_sync(0xffffffffu, cur.gvec, l);
        const long long goff = __shfl_sync(0xffffffffu, cur.goff, l);
#pragma unroll
        for (int hh = 0; hh < G::HALVES; ++hh) {
          float scale_k = 0.0f;
          if (cnt > 0 && lane < G::KH) {
            if (TOPK) scale_k = __uint_as_float(__ldg(A.tau_prev + (long long)(hh * G::KH + lane) * P.T + j));
            else scale_k = __ldg(A.scale_prev + (long long)(hh * G::KH + lane) * P.T + j);
          }
          const int i = (p0 + l) * G::HALVES + hh;
          const int s = i % FW_STAGES;
          int ok = 1;
          if (lane == 0) {
            if (i >= FW_STAGES && !mbar_wait(&S.empty[s], ((i / FW_STAGES) - 1) & 1, A.wc)) {
              atomicOr(A.status, STATUS_TIMEOUT);
              ok = 0;
            }
          }
          if (!__shfl_sync(0xffffffffu, ok, 0)) {
            // Gave up on item i: nobody releases a stage again.  Before this warp returns it waits (bounded) for
            // the copies it already issued into each stage.
            if (lane < FW_STAGES) {
              const int last = i - 1;
              const int j = last - ((last - lane) % FW_STAGES + FW_STAGES) % FW_STAGES;
              if (last >= 0 && j >= 0) mbar_wait(&S.full[lane], (j / FW_STAGES) & 1, A.wc);
            }
            return;
          }
          if (lane == l) { FwItem t = cur; t.h = hh; S.item[s] = t; }
          if (lane < G::KH) S.sc[s][lane] = scale_k;
          __syncwarp();
          if (cnt == 0) {
            if (lane == 0) mbar_arrive(&S.full[s]);
          } else if (lane == 0) {
            const bool drop = A.wc.drop_item == (u32)fw_range_of(p0 + l, chunk_log2) + 1u;   // (testing only)
            const u32 ebytes = (hh == 0 && !GEN) ? (u32)((cnt + 31) & ~31) * 4u : 0u;    // rows are padded to 32 elements
            const int chunks = (cnt + FW_BOX - 1) / FW_BOX;
            constexpr u32 BOXB = (u32)(G::KH * FW_BOX * 4);
            mbar_arrive_expect_tx(&S.full[s], ebytes + (u32)chunks * BOXB * ((gtma ? 2u : 1u) + (GEN ? 1u : 0u)));
            if (hh == 0 && !GEN && !drop) bulk_load(S.e[s], A.ebar + pbase, ebytes, &S.full[s]);  // the old ebar travels with the first group
            for (int c = 0; c < (drop ? 0 : chunks); ++c) {
              tma_load_2d(&S.m[s][c * G::KH * FW_BOX], &tm_m, (int)pbase + c * FW_BOX, hh * G::KH, &S.full[s]);
              if (GEN) tma_load_2d(&S.dd[s][c * G::KH * FW_BOX], &tm_d, (int)pbase + c * FW_BOX, hh * G::KH, &S.full[s]);
              if (gtma) tma_load_2d(&S.g[s][c * G::KH * FW_BOX], &tm_g, (int)goff + c * FW_BOX, hh * G::KH, &S.full[s]);
            }
          }
        }
      }
    }
    return;
  }

  if (warp > FW_WARPS) {
    // ---------------- averagers: ebar' = (1/K) sum_k ( fma(eta_prev, m_k, ebar) - C(.) ), k in order ----------------
    // With two groups of workers per range the partial sums are carried from the first item to the second
    // (k = 0..KH-1, then KH..K-1: still one sequential sum), and ebar' is written into both stages.
    constexpr int NA = FW_AVG_WARPS * 32;
    constexpr int EPT = G::TILEF / NA;               // elements per thread: 1, 2, 4, 8 or 16
    static_assert(EPT >= 1, "an item has at least one element per averager thread");
    constexpr int V = EPT < 4 ? EPT : 4;             // handled in chunks of V consecutive elements
    constexpr int CH = EPT / V;
    const int ta = tid - (FW_WARPS + 1) * 32;
    // scaled sign: the addends sign_code(...) are the previous step's messages C(Delta^(k)); their ordered sum is
    // that step's worker-axis aggregation, written out when the caller left that step's server pass open
    const bool emit_sum = TOPK || A.ssum != nullptr;
    float eb[CH][V], a[CH][V], s2[CH][V];          // (s2: the ordered sum of the messages)
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
      for (int v = 0; v < V; ++v) { eb[c][v] = 0.0f; a[c][v] = 0.0f; s2[c][v] = 0.0f; }
    for (int i = 0; i < nmine * G::HALVES; ++i) {
      const int hh = i % G::HALVES;
      const int s = i % FW_STAGES;
      if (!mbar_wait(&S.full[s], (i / FW_STAGES) & 1, A.wc)) {
        if (lane == 0) atomicOr(A.status, STATUS_TIMEOUT);
        return;
      }
      const FwItem it = S.item[s];
      if (it.cnt > 0) {
        const float* sm = GEN ? S.dd[s] : S.m[s];           // (MODE 2: the stored differences themselves)
        const float* se0 = S.e[(i - hh) % FW_STAGES];       // the first group's stage holds the old ebar
        const float* sc = S.sc[s];
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const int e0 = c * (NA * V) + ta * V;
          if (e0 < it.cnt) {
            if (hh == 0) {
#pragma unroll
              for (int v = 0; v < V; ++v) { eb[c][v] = GEN ? 0.0f : se0[e0 + v]; a[c][v] = 0.0f; s2[c][v] = 0.0f; }
            }
#pragma unroll
            for (int k = 0; k < G::KH; ++k) {
              const float sk = sc[k];
#pragma unroll
              for (int v = 0; v < V; ++v) {
                const float dk = GEN ? sm[G::idx(k, e0) + v] : __fmaf_rn(A.eta_prev, sm[G::idx(k, e0) + v], eb[c][v]);
                if (GEN) {
                  s2[c][v] = __fadd_rn(s2[c][v], topk_selected(dk, __float_as_uint(sk)) ? dk : 0.0f);
                } else if (TOPK) {
                  const float ck = topk_selected(dk, __float_as_uint(sk)) ? dk : 0.0f;
                  a[c][v] = __fadd_rn(a[c][v], __fsub_rn(dk, ck));
                  s2[c][v] = __fadd_rn(s2[c][v], ck);
                } else {
                  const float ck = sign_code(dk, sk);
                  a[c][v] = __fadd_rn(a[c][v], __fsub_rn(dk, ck));
                  if (emit_sum) s2[c][v] = __fadd_rn(s2[c][v], ck);
                }
              }
            }
            if (hh == G::HALVES - 1) {
#pragma unroll
              for (int v = 0; v < V; ++v) {
                if (e0 + v < it.cnt) {
                  if (!GEN) {
                    const float en = div_by_k(P, a[c][v]);
#pragma unroll
                    for (int hq = 0; hq < G::HALVES; ++hq) S.e[(i - hh + hq) % FW_STAGES][e0 + v] = en;
                    A.ebar_out[it.pbase + e0 + v] = en;
                  }
                  if (emit_sum) A.ssum[it.pbase + e0 + v] = s2[c][v];
                }
              }
            }
          }
        }
      }
      __syncwarp();
      if (hh == G::HALVES - 1 && lane == 0) {
#pragma unroll
        for (int hq = 0; hq < G::HALVES; ++hq) mbar_arrive(&S.avgd[(i - hh + hq) % FW_STAGES]);
      }
    }
    return;
  }

  // ---------------- workers ----------------
  // accumulator a belongs to worker (a / WPW) * KH + kl0 + (a % WPW)
  LaneAcc acc[G::NACC];
#pragma unroll
  for (int a = 0; a < G::NACC; ++a) lane_acc_init(acc[a]);
  int acc_j = -1;
  const int row0 = warp * G::RPW;                       // first row of this warp inside an item
  const int kl0 = row0 / G::ROWS_PER_WORKER;            // its (first) worker inside the item's group
  WarpStage stg; stg.buf = S.cstage[TOPK ? warp : 0]; stg.n = 0;   // Top-K: this warp's candidate keys of (kl0, stg_j)
  int stg_j = 0;
  for (int i = 0; i < nmine * G::HALVES; ++i) {
    const int hh = i % G::HALVES;
    const int s = i % FW_STAGES;
    if (!mbar_wait(&S.full[s], (i / FW_STAGES) & 1, A.wc)) {
      if (lane == 0) atomicOr(A.status, STATUS_TIMEOUT);
      return;
    }
    const FwItem it = S.item[s];
    if (it.cnt > 0) {
      if (TOPK) {
        if (it.j != stg_j) { stage_flush(stg, A.cand, kl0, stg_j); stg_j = it.j; }
      } else if (it.j != acc_j) {
        if (acc_j >= 0) {
#pragma unroll
          for (int a = 0; a < G::NACC; ++a) {
            const int kk = (a / G::WPW) * G::KH + kl0 + (a % G::WPW);
            warp_commit(acc[a], A.recs + (long long)kk * P.T + acc_j, A.status);
            lane_acc_init(acc[a]);
          }
        }
        acc_j = it.j;
      }
      const u32 lo = TOPK ? window_lo(__float_as_uint(S.sc[s][kl0]), A.cand.wlog2[it.j]) : NO_GUESS;
      const float* sm = S.m[s];
      const float* sg = S.g[s];
      const float* se = S.e[s];
      const float* sd = S.dd[GEN ? s : 0];
      const u32 tk = TOPK ? __float_as_uint(S.sc[s][kl0]) : 0u;
      // ebar' of this range comes from the averager warps (MODE 2: nothing is handed over, but the averagers
      // must be done with the stage before the workers release it)
      if (!mbar_wait(&S.avgd[s], (i / FW_STAGES) & 1, A.wc)) {
        if (lane == 0) atomicOr(A.status, STATUS_TIMEOUT);
        return;
      }
      // ---- worker lines with e^(k) = ebar' ----
#pragma unroll
      for (int q = 0; q < G::RPW; ++q) {
        const int r = row0 + q;
        const int kl = r / G::ROWS_PER_WORKER, rr = r % G::ROWS_PER_WORKER;
        const int k = hh * G::KH + kl;
        const int a = hh * G::WPW + ((G::WPW == 1) ? 0 : (kl - kl0));
        float* mp = A.m + (long long)k * P.dpad + it.pbase;
        float* dp = A.D + (long long)k * P.dpad + it.pbase;                        // (MODE 2)
        u32* wp = A.words + (long long)k * P.nwords + (it.pbase >> 5);
        const int rbase = G::idx(kl, rr * 128);                // the row's position in the stage buffers
        if (it.gvec && rr * 128 + 128 <= it.cnt) {
          const int e0 = rr * 128 + lane * 4;
          const float4 Gq = *reinterpret_cast<const float4*>(sg + rbase + lane * 4);
          const float4 M = *reinterpret_cast<const float4*>(sm + rbase + lane * 4);
          float4 E;
          if (GEN) {                             // e^(k) = D - C(D) with last step's threshold, formed on the fly
            const float4 Dv = *reinterpret_cast<const float4*>(sd + rbase + lane * 4);
            E.x = prev_error<ESRC_LAZY_TOPK>(Dv.x, 0.0f, tk); E.y = prev_error<ESRC_LAZY_TOPK>(Dv.y, 0.0f, tk);
            E.z = prev_error<ESRC_LAZY_TOPK>(Dv.z, 0.0f, tk); E.w = prev_error<ESRC_LAZY_TOPK>(Dv.w, 0.0f, tk);
          } else {
            E = *reinterpret_cast<const float4*>(se + e0);
          }
          float4 X = make_float4(0.f, 0.f, 0.f, 0.f);
          if (WD) X = ld4(A.x + it.pbase + e0);
          float4 mn, dl;
          dl.x = worker_update<WD>(Gq.x, M.x, E.x, X.x, sp, mn.x);
          dl.y = worker_update<WD>(Gq.y, M.y, E.y, X.y, sp, mn.y);
          dl.z = worker_update<WD>(Gq.z, M.z, E.z, X.z, sp, mn.z);
          dl.w = worker_update<WD>(Gq.w, M.w, E.w, X.w, sp, mn.w);
          st4(mp + e0, mn);
          if (GEN) st4(dp + e0, dl);
          if (TOPK) {
            if (lo != NO_GUESS) {
              if (stg.n > CAND_STAGE - 128) stage_flush(stg, A.cand, kl0, stg_j);
              stage_row4(stg, lo, mag_key(dl.x), mag_key(dl.y), mag_key(dl.z), mag_key(dl.w));
            }
          } else {
            if (G::NACC == 1 || a == 0) lane_add4(acc[0], dl);
            else lane_add4(acc[G::NACC - 1], dl);
            const u32 wd = pack_row4(dl.x >= 0.0f, dl.y >= 0.0f, dl.z >= 0.0f, dl.w >= 0.0f);
            if ((lane & 7) == 0) wp[e0 >> 5] = wd;
          }
        } else if (rr * 128 < it.cnt) {
          // ragged last row of a tensor, or gradients that could not be fetched by TMA
          const float* gp = A.g + (long long)k * P.d + it.goff;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int e = rr * 128 + c * 32 + lane;
            const bool valid = e < it.cnt;
            float dl = 0.0f;
            if (valid) {
              const float xv = WD ? A.x[it.pbase + e] : 0.0f;
              const float gv = it.gvec ? sg[rbase + c * 32 + lane] : __ldcs(gp + e);
              float mn;
              const float ev = GEN ? prev_error<ESRC_LAZY_TOPK>(sd[rbase + c * 32 + lane], 0.0f, tk) : se[e];
              dl = worker_update<WD>(gv, sm[rbase + c * 32 + lane], ev, xv, sp, mn);
              mp[e] = mn;
              if (GEN) dp[e] = dl;
              if (!TOPK) {
                if (G::NACC == 1 || a == 0) lane_add(acc[0], dl);
                else lane_add(acc[G::NACC - 1], dl);
              }
            }
            if (TOPK) {
              if (lo != NO_GUESS) {
                if (stg.n > CAND_STAGE - 32) stage_flush(stg, A.cand, kl0, stg_j);
                stage_row1(stg, lo, valid, mag_key(dl));
              }
            } else {
              const u32 wd = __ballot_sync(0xffffffffu, valid && dl >= 0.0f);
              if (lane == 0 && (rr * 128 + c * 32) < it.cnt) wp[(rr * 128 + c * 32) >> 5] = wd;
            }
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&S.empty[s]);
  }
  if (TOPK) {
    stage_flush(stg, A.cand, kl0, stg_j);
  } else if (acc_j >= 0) {
#pragma unroll
    for (int a = 0; a < G::NACC; ++a) {
      const int kk = (a / G::WPW) * G::KH + kl0 + (a % G::WPW);
      warp_commit(acc[a], A.recs + (long long)kk * P.T + acc_j, A.status);
    }
  }
}

// The pending average on its own (getters): etmp = (1/K) sum_k ( fma(eta, m_k, ebar) - C(...) ).  etmp may be
// ebar itself: a thread reads its element of ebar before it writes it.
__global__ void __launch_bounds__(THREADS) k_materialize_avg(Plan P, const float* __restrict__ m, const float* ebar,
                                                              const float* __restrict__ scale_prev, float eta_prev,
                                                              float* etmp) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) {
    const long long p = ti.poff + ti.t0 + i;
    const float eb = ebar[p];
    float a = 0.0f;
    for (int k = 0; k < P.K; ++k) {
      const float dk = __fmaf_rn(eta_prev, m[(long long)k * P.dpad + p], eb);
      a = __fadd_rn(a, __fsub_rn(dk, sign_code(dk, scale_prev[(long long)k * P.T + ti.j])));
    }
    etmp[p] = div_by_k(P, a);
  }
}

}  // namespace sae
