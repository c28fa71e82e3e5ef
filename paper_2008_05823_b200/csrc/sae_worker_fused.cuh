// Worker pass with the pending error averaging folded in (scaled sign, averaging period 1).
//
// With p = 1 every step ends with "average the local errors" (Algorithm 1, pre-step):
//     ebar' = (1/K) sum_k ( Delta^(k) - C(Delta^(k)) ),     Delta^(k) = fma(eta, m^(k), ebar).
// Doing that in the apply kernel costs a second read of all K momentum rows.  This kernel instead
// leaves the average pending and computes it at the head of the NEXT step's worker pass, which has to
// read the same momentum rows anyway:
//   phase A (per tile, all K workers): ebar' from the rows of m in shared memory, k = 0..K-1 in order,
//            with last step's learning rate and scales (same fused op, same order: same bits);
//   phase B: the usual worker lines with e^(k) = ebar' -- momentum, Delta, exact L1 partials, sign words.
// One block handles a tile for ALL workers: the producer warp brings the K momentum tiles and the ebar
// tile -- and the K gradient tiles when they are 16-byte aligned -- in with bulk asynchronous copies
// (3-stage ring, full/empty mbarriers), so the consumers touch global memory only to store.
// In phase B a consumer warp always works for the same worker(s), so it carries their L1 partials
// across tiles and adds them to the (worker, tensor) records only when the tensor changes.
// All waits are bounded (STATUS_TIMEOUT).
#pragma once
#include "sae_worker_tma.cuh"

namespace sae {

constexpr int FW_WARPS = 16;                       // consumer warps
constexpr int FW_THREADS = FW_WARPS * 32 + 32;     // + producer warp
constexpr int FW_STAGES = 3;
constexpr int FW_MAXTILE = 2048;
constexpr int FW_MBUF = 8192;                      // floats of momentum (and of gradient) per stage (32 KB each)

template <int K>
struct FwGeom {
  static constexpr int TILEF = (FW_MBUF / K) < FW_MAXTILE ? (FW_MBUF / K) : FW_MAXTILE;   // elements per item
  static constexpr int SUB = TILE / TILEF;                    // items per 4096-element plan tile
  static constexpr int ROWS_PER_WORKER = TILEF / 128;
  static constexpr int RPW = K * ROWS_PER_WORKER / FW_WARPS;  // 128-element rows per warp and item
  static constexpr int WPW = RPW > ROWS_PER_WORKER ? RPW / ROWS_PER_WORKER : 1;   // workers per warp
  static_assert(K >= 1 && K <= 32 && (K & (K - 1)) == 0, "power-of-two worker counts up to 32");
  static_assert(RPW >= 1 && WPW <= 2, "geometry");
};

struct FwItem {
  long long pbase;   // first element in the [dpad] arrays
  long long goff;    // first element inside a gradient row (caller layout)
  int j, cnt, gvec;  // tensor, valid elements (0 = empty item), gradients 16-byte aligned for every worker
};

struct FwSmem {
  alignas(128) float m[FW_STAGES][FW_MBUF];
  alignas(128) float g[FW_STAGES][FW_MBUF];
  alignas(128) float e[FW_STAGES][FW_MAXTILE];
  alignas(8) u64 full[FW_STAGES];
  alignas(8) u64 empty[FW_STAGES];
  FwItem item[FW_STAGES];
  float sc[FW_STAGES][32];      // last step's scales of the item's tensor, one per worker
};

struct FusedArgs {
  const float* g;
  float* m;
  float* ebar;             // in: ebar of the previous step, out: the averaged error of this pre-step
  const float* x;
  const float* scale_prev; // [K][T] scales of the previous step
  u32* words;
  L1Record* recs;
  u32* status;
  float eta_prev;
};

template <int K>
__device__ __forceinline__ FwItem fw_lookup(const Plan& P, const float* g, long long w, long long nitems) {
  typedef FwGeom<K> G;
  FwItem it;
  it.pbase = 0; it.goff = 0; it.j = 0; it.cnt = 0; it.gvec = 0;
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
  it.gvec = ((reinterpret_cast<uintptr_t>(g + it.goff) & 15) == 0) && (K == 1 || (P.d & 3) == 0);
  return it;
}

template <int K, bool WD>
__global__ void __launch_bounds__(FW_THREADS, 1) k_worker_fused(Plan P, StepParams sp, FusedArgs A, long long nitems) {
  typedef FwGeom<K> G;
  extern __shared__ unsigned char smem_raw[];
  FwSmem& S = *reinterpret_cast<FwSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < FW_STAGES; ++s) { mbar_init(&S.full[s], 1); mbar_init(&S.empty[s], FW_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == FW_WARPS) {
    // ---------------- producer ----------------
    const long long GR = gridDim.x;
    long long wb = blockIdx.x;
    FwItem nxt = fw_lookup<K>(P, A.g, wb + lane * GR, nitems);
    for (int i0 = 0; wb < nitems; i0 += 32, wb += 32 * GR) {
      const FwItem cur = nxt;
      nxt = fw_lookup<K>(P, A.g, wb + (32 + lane) * GR, nitems);
      for (int l = 0; l < 32; ++l) {
        // the item of lane l, broadcast so that the lanes can share the issue of its copies
        const int cnt = __shfl_sync(0xffffffffu, cur.cnt, l);
        if (cnt < 0) break;                                   // past the last item (uniform)
        const long long pbase = __shfl_sync(0xffffffffu, cur.pbase, l);
        const int j = __shfl_sync(0xffffffffu, cur.j, l);
        float scale_k = 0.0f;
        if (cnt > 0 && lane < K) scale_k = __ldg(A.scale_prev + (long long)lane * P.T + j);
        const int i = i0 + l;
        const int s = i % FW_STAGES;
        int ok = 1;
        if (lane == 0) {
          if (i >= FW_STAGES && !mbar_wait(&S.empty[s], ((i / FW_STAGES) - 1) & 1)) {
            atomicOr(A.status, STATUS_TIMEOUT);
            ok = 0;
          }
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) return;
        if (lane == l) S.item[s] = cur;
        if (lane < K) S.sc[s][lane] = scale_k;
        __syncwarp();
        if (cnt == 0) {
          if (lane == 0) mbar_arrive(&S.full[s]);
        } else {
          const u32 bytes = (u32)((cnt + 31) & ~31) * 4u;     // rows are padded to 32 elements
          const int gfast = __shfl_sync(0xffffffffu, cur.gvec, l) && cnt == G::TILEF;
          const long long goff = __shfl_sync(0xffffffffu, cur.goff, l);
          if (lane == 0) {
            mbar_arrive_expect_tx(&S.full[s], bytes * (K + 1) + (gfast ? (u32)(G::TILEF * 4 * K) : 0u));
            bulk_load(S.e[s], A.ebar + pbase, bytes, &S.full[s]);
          }
          __syncwarp();
          if (lane < K) {
            bulk_load(&S.m[s][lane * G::TILEF], A.m + (long long)lane * P.dpad + pbase, bytes, &S.full[s]);
            if (gfast)
              bulk_load(&S.g[s][lane * G::TILEF], A.g + (long long)lane * P.d + goff, G::TILEF * 4, &S.full[s]);
          }
        }
      }
    }
    return;
  }

  // ---------------- consumers ----------------
  LaneAcc acc[G::WPW];
#pragma unroll
  for (int a = 0; a < G::WPW; ++a) lane_acc_init(acc[a]);
  int acc_j = -1;
  const int row0 = warp * G::RPW;                       // first row of this warp inside an item
  const int k0 = row0 / G::ROWS_PER_WORKER;             // its (first) worker
  const float Kf = (float)K;
  long long w = blockIdx.x;
  for (int i = 0; w < nitems; ++i, w += gridDim.x) {
    const int s = i % FW_STAGES;
    if (!mbar_wait(&S.full[s], (i / FW_STAGES) & 1)) {
      if (lane == 0) atomicOr(A.status, STATUS_TIMEOUT);
      return;
    }
    const FwItem it = S.item[s];
    if (it.cnt > 0) {
      if (it.j != acc_j) {
        if (acc_j >= 0) {
#pragma unroll
          for (int a = 0; a < G::WPW; ++a) {
            warp_commit(acc[a], A.recs + (long long)(k0 + a) * P.T + acc_j, A.status);
            lane_acc_init(acc[a]);
          }
        }
        acc_j = it.j;
      }
      const bool gfast = it.gvec && it.cnt == G::TILEF;
      // ---- phase A: the pending average, ebar' ----
      const float* sm = S.m[s];
      float* se = S.e[s];
      {
        const float* sc = S.sc[s];
        for (int e = tid; e < it.cnt; e += FW_WARPS * 32) {
          {
            const float eb = se[e];
            float a = 0.0f;
#pragma unroll
            for (int k = 0; k < K; ++k) {
              const float dk = __fmaf_rn(A.eta_prev, sm[k * G::TILEF + e], eb);
              a = __fadd_rn(a, __fsub_rn(dk, sign_code(dk, sc[k])));
            }
            const float en = __fdiv_rn(a, Kf);
            se[e] = en;
            A.ebar[it.pbase + e] = en;
          }
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(FW_WARPS * 32) : "memory");
      // ---- phase B: worker lines with e^(k) = ebar' ----
#pragma unroll
      for (int q = 0; q < G::RPW; ++q) {
        const int r = row0 + q;
        const int k = r / G::ROWS_PER_WORKER, rr = r % G::ROWS_PER_WORKER;
        const int a = (G::WPW == 1) ? 0 : (k - k0);
        float* mp = A.m + (long long)k * P.dpad + it.pbase;
        u32* wp = A.words + (long long)k * P.nwords + (it.pbase >> 5);
        const float* smk = sm + k * G::TILEF;
        const float* sgk = S.g[s] + k * G::TILEF;
        if (gfast) {
          const int e0 = rr * 128 + lane * 4;
          const float4 Gq = *reinterpret_cast<const float4*>(sgk + e0);
          const float4 M = *reinterpret_cast<const float4*>(smk + e0);
          const float4 E = *reinterpret_cast<const float4*>(se + e0);
          float4 X = make_float4(0.f, 0.f, 0.f, 0.f);
          if (WD) X = ld4(A.x + it.pbase + e0);
          float4 mn, dl;
          dl.x = worker_update<WD>(Gq.x, M.x, E.x, X.x, sp, mn.x);
          dl.y = worker_update<WD>(Gq.y, M.y, E.y, X.y, sp, mn.y);
          dl.z = worker_update<WD>(Gq.z, M.z, E.z, X.z, sp, mn.z);
          dl.w = worker_update<WD>(Gq.w, M.w, E.w, X.w, sp, mn.w);
          st4(mp + e0, mn);
          if (G::WPW == 1) lane_add4(acc[0], dl);
          else if (a == 0) lane_add4(acc[0], dl);
          else lane_add4(acc[G::WPW - 1], dl);
          const u32 wd = pack_row4(dl.x >= 0.0f, dl.y >= 0.0f, dl.z >= 0.0f, dl.w >= 0.0f);
          if ((lane & 7) == 0) wp[e0 >> 5] = wd;
        } else if (rr * 128 < it.cnt) {
          const float* gp = A.g + (long long)k * P.d + it.goff;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int e = rr * 128 + c * 32 + lane;
            const bool valid = e < it.cnt;
            float dl = 0.0f;
            if (valid) {
              const float xv = WD ? A.x[it.pbase + e] : 0.0f;
              float mn;
              dl = worker_update<WD>(__ldcs(gp + e), smk[e], se[e], xv, sp, mn);
              mp[e] = mn;
              if (G::WPW == 1) lane_add(acc[0], dl);
              else if (a == 0) lane_add(acc[0], dl);
              else lane_add(acc[G::WPW - 1], dl);
            }
            const u32 wd = __ballot_sync(0xffffffffu, valid && dl >= 0.0f);
            if (lane == 0 && (rr * 128 + c * 32) < it.cnt) wp[(rr * 128 + c * 32) >> 5] = wd;
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&S.empty[s]);
  }
  if (acc_j >= 0) {
#pragma unroll
    for (int a = 0; a < G::WPW; ++a) warp_commit(acc[a], A.recs + (long long)(k0 + a) * P.T + acc_j, A.status);
  }
}

// The pending average on its own (getters): etmp = (1/K) sum_k ( fma(eta, m_k, ebar) - C(...) ).
__global__ void __launch_bounds__(THREADS) k_materialize_avg(Plan P, const float* __restrict__ m,
                                                              const float* __restrict__ ebar,
                                                              const float* __restrict__ scale_prev, float eta_prev,
                                                              float* __restrict__ etmp) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  const float Kf = (float)P.K;
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) {
    const long long p = ti.poff + ti.t0 + i;
    const float eb = ebar[p];
    float a = 0.0f;
    for (int k = 0; k < P.K; ++k) {
      const float dk = __fmaf_rn(eta_prev, m[(long long)k * P.dpad + p], eb);
      a = __fadd_rn(a, __fsub_rn(dk, sign_code(dk, scale_prev[(long long)k * P.T + ti.j])));
    }
    etmp[p] = __fdiv_rn(a, Kf);
  }
}

}  // namespace sae
