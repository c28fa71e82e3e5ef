// Kernels of one iteration of Algorithm 1.  One thread block handles one tile (TILE consecutive
// elements of one tensor), for one worker in the worker pass, for all workers in the server passes.
// Full tiles whose gradient pointer is 16-byte aligned take a 128-bit vector path; ragged tails and
// misaligned gradient rows take a lane-strided scalar path.  Both produce identical bits.
#pragma once
#include "sae_device.cuh"
#include "sae_topk.cuh"

namespace sae {

struct StepParams {
  float mu, eta, lambda;
  int saef;   // 1: gradient point is x - e^(k), 0: x
  int wd;     // lambda != 0
};

// where the previous local error e_t^(k) comes from
constexpr int ESRC_UNIFORM = 0;    // e^(k) = ebar for all k (after an averaging pre-step, or at t = 0)
constexpr int ESRC_LAZY_SIGN = 1;  // e^(k) = D^(k) - C(D^(k)) with last step's scales, D^(k) = last Delta^(k)
constexpr int ESRC_LAZY_TOPK = 2;  // same with last step's Top-K thresholds
constexpr int ESRC_PENDING_AVG = 3;  // p = 1, scaled sign: e^(k) = mean_k(fma(eta_prev, m^(k), ebar) - C(.)), not yet formed
constexpr int ESRC_LOCAL_D = 4;    // local steps: D^(k) is the running local model difference (the error plus the
                                   // local updates not yet communicated) and takes the place of e^(k) as it is

template <int ESRC>
__device__ __forceinline__ float prev_error(float v, float sprev, u32 tprev) {
  if (ESRC == ESRC_UNIFORM || ESRC == ESRC_LOCAL_D) return v;
  if (ESRC == ESRC_LAZY_SIGN) return __fsub_rn(v, sign_code(v, sprev));
  return __fsub_rn(v, topk_selected(v, tprev) ? v : 0.0f);
}

// Algorithm 1, worker lines: step-ahead point, local momentum, local model difference.
template <bool WD>
__device__ __forceinline__ float worker_update(float g, float mo, float e, float x, const StepParams& sp,
                                               float& mn) {
  float ge = g;
  if (WD) {
    float xh = sp.saef ? __fsub_rn(x, e) : x;
    ge = __fmaf_rn(sp.lambda, xh, g);
  }
  mn = __fmaf_rn(sp.mu, mo, ge);
  return __fmaf_rn(sp.eta, mn, e);
}

struct WorkerArgs {
  const float* g;         // [K][d] caller layout
  float* m;               // [K][dpad]
  float* D;               // [K][dpad] last model difference (read when lazy, written when WRITE_D)
  const float* ebar;      // [dpad]
  const float* x;         // [dpad]
  const float* scale_prev;  // [K][T]
  const u32* tau_prev;      // [K][T] last step's thresholds (lazy error, and the guess of the candidate window)
  CandArgs cand;            // Top-K candidate lists of the workers
  u32* words;             // [K][nwords]
  float* scale_cur;       // [K][T]
  L1Record* recs;         // [K][T]
  u32* status;
  WaitCfg wc;
};

// ---------------------------------------------------------------------------------------------------
struct ServerArgs {
  float* e_srv;            // [dpad]: in: server error e_t, out: server model difference Delta_{t+1}
  const u32* words;        // [K][nwords] worker sign words
  const float* scale_cur;  // [K][T] worker scales of this step
  const float* D;          // [K][dpad] (dense variants)
  const u32* tau_cur;      // [K][T] (Top-K)
  u32* words_srv;          // [nwords]
  float* scale_srv;        // [T]
  L1Record* recs_srv;      // [T]
  u32* status;
  CandArgs cand_srv;       // Top-K candidate list of the server (one row)
  const u32* tau_srv_prev; // [T] last step's server thresholds: the guess of the server's window
  int emit_srv;            // double-way Top-K: collect the server's candidates in this pass
  float* ebar;             // [dpad] averaged local error (dense variants, when the pre-step averages)
  const float* m;          // [K][dpad] } recompute variant: Delta^(k) = fma(eta, m^(k), ebar_in), not stored
  const float* ebar_in;    // [dpad]    } (ebar_in and ebar are different buffers)
  float eta;
  const float* ssum;       // [dpad] (SUM variant) ordered worker-axis sum of the selected entries, not yet divided by K
  // sharded operation: worker k's message lives with its owner (possibly another GPU's memory, read in place)
  const u32* const* word_rows;     // [K] -> worker k's [nwords] sign words
  const float* const* scale_rows;  // [K] -> worker k's [T] scales of this step
  // small problems: the scales are formed here from the workers' exact L1 records (no separate launch)
  const L1Record* recs;            // [K][T]
  float* scale_out;                // [K][T] this step's scales, written by the block that holds a tensor's first tile
  L1Record* recs_clear;            // [K][T] the other worker-record buffer: cleared here for the next worker pass
  L1Record* recs_srv_clear;        // [T] the server-record buffer the next step accumulates into: cleared here
  const L1Record* recs_srv_prev;   // [T] the previous step's server records (LAZY: its server scale comes from them)
  // deferred server update of the previous step (LAZY): e_srv still holds that step's Delta and x is not yet
  // re-updated; both are brought up to date here, element by element, before this step's Delta is formed
  float* x;                        // [dpad]
  const float* scale_srv_prev;     // [T] server scales of the previous step (double-way)
  u32* mask_srv;                   // [nwords] Top-K: the server's selection of the previous step (written when pending)
  WaitCfg wc;
};

// K3 (scaled sign): Delta = e + (1/K) sum_k C(Delta^(k)) from the packed messages; with double-way
// compression also the server's L1 partials and sign words.  A block walks `tiles_per_block` consecutive
// tiles, so the scales are staged and the L1 partials committed once per run of tiles of one tensor.
//
// The pass is bound by instruction issue, not by memory: K order-fixed additions per parameter, each of
// +-s_k chosen by one message bit.  A thread owns 16 consecutive parameters (half a sign word): per worker
// it loads the word once, and per parameter moves the bit to the sign position (shift), flips the sign of
// s_k with it (one three-input logic operation) and adds; the additions are issued two at a time as
// packed fp32 pairs (add.rn.f32x2: two independent round-to-nearest fp32 additions, same results as two
// scalar ones).
//
// TABLE: the K messages are not rows of one local array but are read in place from their owners through a
// table of row pointers (sharded operation: the gather of the messages and the aggregation are this one
// pass; plain loads, also from a peer GPU's memory).
constexpr int SRV_E = 16;   // consecutive parameters per thread; THREADS * SRV_E == TILE
constexpr int SRV_B = 8;    // workers per batch of word loads
#ifndef SAE_K3_STAGE
#define SAE_K3_STAGE 1
#endif
#ifndef SAE_K3_FIN_EARLY
#define SAE_K3_FIN_EARLY 1
#endif
#ifndef SAE_K3_SUM_DIRECT
#define SAE_K3_SUM_DIRECT 1
#endif
static_assert(THREADS * SRV_E == TILE, "one pass of the block covers one tile");

__device__ __forceinline__ u64 pack2(u32 lo, u32 hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 add_f32x2(u64 a, u64 b) {
  u64 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// FIN (small, latency-bound problems): the worker scales are not read but formed here from the exact L1
// records, which saves the launch of k_finalize_scales.  The record buffers rotate (two for the workers,
// three for the server) so that this pass can also clear the ones the next step accumulates into: nobody
// reads those any more, and nothing else would clear them.
// LAZY: the previous step left its server lines pending (e = Delta - C(Delta), x = x - C(Delta): the work of
// k_apply); they are carried out here on the fly -- the same two subtractions per parameter -- so that the
// server error and the parameters make one trip through memory per step instead of two.  This pass has
// the memory bandwidth to spare (it is bound by instruction issue).
// Staging (all but FIN): a full tile's server error (LAZY: and parameters) is fetched by one bulk
// asynchronous copy (TMA) into shared memory when the block reaches the tile and is first read after the
// worker loop, so that its memory latency passes under the loop without holding registers for it.
// SUM (p = 1, folded form): the ordered sum of the workers' messages was already formed by the following step's
// worker pass (its averager warps add the same +-s_k in the same order) and is only read here: no message
// words, no worker loop -- a plain streaming pass.
template <bool DC, bool TABLE = false, bool FIN = false, bool LAZY = false, bool SUM = false>
__global__ void __launch_bounds__(THREADS) k_server_sign(Plan P, ServerArgs A, int tiles_per_block) {
  __shared__ float s_k[MAX_WORKERS];
  __shared__ float sh_s_old;
  __shared__ const u32* s_row[TABLE ? MAX_WORKERS : 1];
  // (SUM: there is no worker loop for the staged copy to pass under -- staging would only put a wait between a
  // tile's loads and its arithmetic -- so a thread fetches its 16 parameters of the sum, the server error and
  // the parameters with twelve independent 16-byte loads up front.)
  constexpr bool DIRECT = SUM && SAE_K3_SUM_DIRECT;
  constexpr bool STAGE = SAE_K3_STAGE && !FIN && !DIRECT;
  // the server error (and parameters) fetched by the thread itself ahead of the worker loop: the streaming form,
  // and the small problems, where a step is a chain of latencies and registers are not what limits the pass
  constexpr bool EARLY = DIRECT || (FIN && SAE_K3_FIN_EARLY);
  __shared__ alignas(128) float s_e[STAGE ? TILE : 4];
  __shared__ alignas(128) float s_x[(STAGE && LAZY) ? TILE : 4];
  __shared__ alignas(8) u64 s_bar;
  u32 phase = 0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (STAGE && tid == 0) {
    mbar_init(&s_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");   // (made visible by the first barrier below)
  }
  if (TABLE) {
    for (int k = tid; k < P.K; k += THREADS) s_row[k] = A.word_rows[k];     // visible after the barrier below
  }
  const int tile0 = blockIdx.x * tiles_per_block;
  const int tile1 = min(P.ntiles, tile0 + tiles_per_block);
  LaneAcc acc; lane_acc_init(acc);
  int cur_j = -1;

  for (int tile = tile0; tile < tile1; ++tile) {
    const TileInfo ti = tile_info(P, tile);
    if (ti.j != cur_j) {
      if (DC && cur_j >= 0) { warp_commit(acc, A.recs_srv + cur_j, A.status); lane_acc_init(acc); }
      __syncthreads();                            // the previous tensor's scales are no longer read
      for (int k = tid; k < (SUM ? 0 : P.K); k += THREADS) {
        if (FIN) {
          const L1Record r = A.recs[(long long)k * P.T + ti.j];
          const float s = scale_from_limbs(r.limb[0], r.limb[1], r.limb[2], ti.n);
          s_k[k] = s;
          if (ti.t0 == 0) {
            A.scale_out[(long long)k * P.T + ti.j] = s;
            L1Record* c = A.recs_clear + (long long)k * P.T + ti.j;
            c->limb[0] = 0; c->limb[1] = 0; c->limb[2] = 0;
          }
        } else {
          s_k[k] = TABLE ? A.scale_rows[k][ti.j] : A.scale_cur[(long long)k * P.T + ti.j];
        }
      }
      if (FIN && tid == 0 && ti.t0 == 0) {
        L1Record* c = A.recs_srv_clear + ti.j;
        c->limb[0] = 0; c->limb[1] = 0; c->limb[2] = 0;
      }
      if (LAZY && DC && tid == 0) {
        if (FIN) {
          const L1Record r = A.recs_srv_prev[ti.j];
          sh_s_old = scale_from_limbs(r.limb[0], r.limb[1], r.limb[2], ti.n);
          if (ti.t0 == 0) A.scale_srv[ti.j] = sh_s_old;
        } else {
          sh_s_old = A.scale_srv_prev[ti.j];
        }
      }
      __syncthreads();
      cur_j = ti.j;
    }
    const long long pbase = ti.poff + ti.t0;
    float* ep = A.e_srv + pbase;
    float* xp = A.x + pbase;                       // (LAZY only)
    const float s_old = (LAZY && DC) ? sh_s_old : 0.0f;
    const u32* __restrict__ wp = A.words + (pbase >> 5);
    u32* wsp = A.words_srv + (pbase >> 5);

    if (ti.cnt == TILE) {
      if constexpr (STAGE) {
        __syncthreads();                          // nobody still reads the previous tile's staged rows
        if (tid == 0) {
          mbar_arrive_expect_tx(&s_bar, (LAZY ? 2u : 1u) * TILE * (u32)sizeof(float));
          if (A.wc.drop_item != (u32)tile + 1u) {
            bulk_load(s_e, ep, TILE * (u32)sizeof(float), &s_bar);
            if (LAZY) bulk_load(s_x, xp, TILE * (u32)sizeof(float), &s_bar);
          }
        }
      }
      const int i = tid * SRV_E;
      const int wi = i >> 5, sh = (32 - SRV_E) - (i & 31);   // this thread's bits go to the top of the word
      u64 a2[SRV_E / 2];
#pragma unroll
      for (int j = 0; j < SRV_E / 2; ++j) a2[j] = 0ull;      // (+0, +0)
      // Single-way: the server error is fetched ahead of the worker loop, so that its latency hides under
      // the loop.  (Double-way has enough independent work after the loop; fetching early there only
      // costs registers.)
      float4 sv[SUM ? SRV_E / 4 : 1];              // (SUM) the tile of the sum: fetched while the staged rows arrive
      if constexpr (SUM) {
#pragma unroll
        for (int q = 0; q < SRV_E / 4; ++q) sv[q] = ld4_stream(A.ssum + pbase + i + 4 * q);
      }
      float4 ev[((DC || STAGE) && !EARLY) ? 1 : SRV_E / 4];
      float4 xd[(EARLY && LAZY) ? SRV_E / 4 : 1];
      if constexpr (EARLY || (!DC && !STAGE)) {
#pragma unroll
        for (int q = 0; q < SRV_E / 4; ++q) ev[q] = ld4(ep + i + 4 * q);
      }
      if constexpr (EARLY && LAZY) {
#pragma unroll
        for (int q = 0; q < SRV_E / 4; ++q) xd[q] = ld4(xp + i + 4 * q);
      }
      // The words of SRV_B workers are fetched as one batch of independent loads, the next batch while
      // this one is consumed: without that the loop waits out one memory latency per worker.
      const u32* wk = wp + wi;                     // worker k's word: stepped by the row pitch, no multiply
      const long long wofs = (pbase >> 5) + wi;    // (TABLE) the same word inside every worker's own row
      u32 wn[SRV_B];
#pragma unroll
      for (int u = 0; u < SRV_B; ++u)
        wn[u] = (!SUM && u < P.K) ? __ldg(TABLE ? s_row[u] + wofs : wk + (long long)u * P.nwords) : 0u;
      for (int k0 = 0; k0 < (SUM ? 0 : P.K); k0 += SRV_B) {
        u32 w[SRV_B];
#pragma unroll
        for (int u = 0; u < SRV_B; ++u) w[u] = wn[u];
        wk += (long long)SRV_B * P.nwords;
#pragma unroll
        for (int u = 0; u < SRV_B; ++u)
          wn[u] = (k0 + SRV_B + u < P.K)
                      ? __ldg(TABLE ? s_row[k0 + SRV_B + u] + wofs : wk + (long long)u * P.nwords) : 0u;
#pragma unroll
        for (int u = 0; u < SRV_B; ++u) {
          if (k0 + u < P.K) {
            const u32 t = ~(w[u] << sh);           // a clear bit is a negative code: it flips the sign of s_k
            const u32 sb = __float_as_uint(s_k[k0 + u]);
#pragma unroll
            for (int j = 0; j < SRV_E; j += 2) {
              const u32 c0 = ((t << (SRV_E - 1 - j)) & 0x80000000u) ^ sb;
              const u32 c1 = ((t << (SRV_E - 2 - j)) & 0x80000000u) ^ sb;
              a2[j / 2] = add_f32x2(a2[j / 2], pack2(c0, c1));
            }
          }
        }
      }
      if constexpr (STAGE) {
        if (!mbar_wait(&s_bar, phase, A.wc)) {           // gave up: flag it and leave (the whole block does)
          if (tid == 0) atomicOr(A.status, STATUS_TIMEOUT);
          return;
        }
        phase ^= 1u;
      }
      u32 bits = 0;
#pragma unroll
      for (int q = 0; q < SRV_E / 4; ++q) {
        float a0, a1, a3, a4;
        if constexpr (SUM) {
          a0 = sv[q].x; a1 = sv[q].y; a3 = sv[q].z; a4 = sv[q].w;
        } else {
          unpack2(a2[2 * q], a0, a1);
          unpack2(a2[2 * q + 1], a3, a4);
        }
        float4 e;
        if constexpr (STAGE) e = ld4(s_e + i + 4 * q);
        else if constexpr (EARLY) e = ev[q];
        else if constexpr (DC) e = ld4(ep + i + 4 * q);
        else e = ev[q];
        if constexpr (LAZY) {
          // e holds the previous step's Delta: C(Delta) is its scaled sign (double-way) or Delta itself
          float4 xv;
          if constexpr (EARLY) xv = xd[q];
          else xv = STAGE ? ld4(s_x + i + 4 * q) : ld4(xp + i + 4 * q);
          float4 cs;
          cs.x = DC ? sign_code(e.x, s_old) : e.x; cs.y = DC ? sign_code(e.y, s_old) : e.y;
          cs.z = DC ? sign_code(e.z, s_old) : e.z; cs.w = DC ? sign_code(e.w, s_old) : e.w;
          xv.x = __fsub_rn(xv.x, cs.x); xv.y = __fsub_rn(xv.y, cs.y);
          xv.z = __fsub_rn(xv.z, cs.z); xv.w = __fsub_rn(xv.w, cs.w);
          st4(xp + i + 4 * q, xv);
          e.x = __fsub_rn(e.x, cs.x); e.y = __fsub_rn(e.y, cs.y);
          e.z = __fsub_rn(e.z, cs.z); e.w = __fsub_rn(e.w, cs.w);
        }
        float4 ds;
        ds.x = __fadd_rn(e.x, div_by_k(P, a0));
        ds.y = __fadd_rn(e.y, div_by_k(P, a1));
        ds.z = __fadd_rn(e.z, div_by_k(P, a3));
        ds.w = __fadd_rn(e.w, div_by_k(P, a4));
        st4(ep + i + 4 * q, ds);
        if (DC) {
          lane_add4(acc, ds);
          bits |= ((ds.x >= 0.0f ? 1u : 0u) | (ds.y >= 0.0f ? 2u : 0u) | (ds.z >= 0.0f ? 4u : 0u) |
                   (ds.w >= 0.0f ? 8u : 0u)) << (4 * q);
        }
      }
      if (DC) {
        u32 w = bits << (SRV_E * (lane & 1));      // two lanes share a word
        w |= __shfl_xor_sync(0xffffffffu, w, 1);
        if ((lane & 1) == 0) wsp[wi] = w;
      }
    } else {
      for (int r = 0; r < ROWS; ++r) {
        const int i = r * THREADS + tid;
        const bool valid = i < ti.cnt;
        float ds = 0.0f;
        if (valid) {
          float a = SUM ? A.ssum[pbase + i] : 0.f;
          const int wi = i >> 5;
          for (int k = 0; k < (SUM ? 0 : P.K); ++k) {
            const u32 w = __ldg(TABLE ? s_row[k] + (pbase >> 5) + wi : wp + (long long)k * P.nwords + wi) >> lane;
            const float s = s_k[k];
            a = __fadd_rn(a, (w & 1u) ? s : -s);
          }
          float eo = ep[i];
          if (LAZY) {
            const float cs = DC ? sign_code(eo, s_old) : eo;
            xp[i] = __fsub_rn(xp[i], cs);
            eo = __fsub_rn(eo, cs);
          }
          ds = __fadd_rn(eo, div_by_k(P, a));
          ep[i] = ds;
          if (DC) lane_add(acc, ds);
        }
        if (DC) {
          u32 w = __ballot_sync(0xffffffffu, valid && ds >= 0.0f);
          if (lane == 0 && (r * THREADS + warp * 32) < ti.cnt) wsp[(r * THREADS + warp * 32) >> 5] = w;
        }
      }
    }
  }
  if (DC && cur_j >= 0) warp_commit(acc, A.recs_srv + cur_j, A.status);
}

// K3 (identity / Top-K): the same aggregation from the dense model differences.
// COMP 0: C = identity, 2: Top-K with this step's thresholds, 1: scaled sign with this step's scales (the form
// that closes a p = 1 scaled-sign step in one pass when the caller wants the state right after it: the messages
// C(Delta^(k)) are re-formed from the momentum rows instead of unpacked from the sign words, so that the same
// pass over the rows also yields the averaged error; with double-way compression it adds the server's exact
// L1 partials and sign words like k_server_sign).
// AVG: the next pre-step averages the local errors; they are functions of the same D^(k) and thresholds
// this pass already reads, so ebar = (1/K) sum_k (D^(k) - C(D^(k))) is formed here, in k order, instead of
// in a further pass over D.
// RECOMP (Top-K with p = 1: the previous error is uniform and the pre-step averages, every step): the worker
// pass did not store D^(k); it is recomputed here from m^(k) and the previous uniform error with the fused
// operation that formed it, so the step moves 4 bytes per worker-element less.
// LSRV != 0 (Top-K): the previous step left its server lines pending -- e = Delta - C(Delta), x = x - C(Delta)
// and the server's selection words; they are carried out here on the fly with last step's server threshold
// (LSRV 2), with last step's server scale (LSRV 3, scaled sign) or with C = identity (LSRV 1, single-way), the
// same operations the apply kernel would have done.
// Full tiles are read through a ring of DENSE_RING thread-private 16-byte slots in shared memory filled by
// asynchronous copies (cp.async): the reads of a thread -- per group of four parameters the server error,
// (deferred lines) the parameters, (recompute) the old averaged error, then the K rows in k order -- form one
// sequence, and the copy of element q + DENSE_RING - 1 of that sequence is issued when element q is consumed,
// so about DENSE_RING - 1 loads per thread are in flight at any time whatever K is and without holding
// registers for them.  A thread reads back only what it copied itself: no block-level synchronisation.
#ifndef SAE_DENSE_RING
#define SAE_DENSE_RING 8
#endif
constexpr int DENSE_RING = SAE_DENSE_RING;
constexpr size_t kDenseSmem = (size_t)DENSE_RING * THREADS * sizeof(float4);

__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((u32)__cvta_generic_to_shared(dst_smem)), "l"(src)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// SUM (Top-K, p = 1, folded form): the ordered worker-axis sum of the selected entries was already formed by
// the worker pass of the following step (k_worker_fused<.., TOPK>) and is only read here; no rows are touched.
template <int COMP, bool AVG, bool RECOMP = false, int LSRV = 0, bool SUM = false>
__global__ void __launch_bounds__(THREADS) k_server_dense(Plan P, ServerArgs A) {
  __shared__ u32 t_k[MAX_WORKERS];
  __shared__ u32 cstage[(COMP == 2) ? (THREADS / 32) * CAND_STAGE : 1];
  extern __shared__ float4 ring[];                       // [DENSE_RING][THREADS]
  const TileInfo ti = tile_info(P, blockIdx.x);
  const int tid = threadIdx.x;
  const bool emit = (COMP == 2) && A.emit_srv;
  const bool sign_dc = (COMP == 1) && A.emit_srv;        // scaled sign, double-way: the server's L1 partials and words
  const u32 lo = emit ? window_lo(A.tau_srv_prev[ti.j], A.cand_srv.wlog2[ti.j]) : NO_GUESS;
  WarpStage stg; stg.buf = cstage + ((COMP == 2) ? (tid >> 5) * CAND_STAGE : 0); stg.n = 0;
  LaneAcc acc; lane_acc_init(acc);
  if (COMP != 0 && !SUM) {                               // (SUM: no rows are read, so no worker thresholds either)
    for (int k = tid; k < P.K; k += THREADS)
      t_k[k] = (COMP == 2) ? A.tau_cur[(long long)k * P.T + ti.j]
                           : __float_as_uint(A.scale_cur[(long long)k * P.T + ti.j]);
    __syncthreads();
  }
  const long long pbase = ti.poff + ti.t0;
  float* ep = A.e_srv + pbase;
  const float* __restrict__ dp = (RECOMP ? A.m : A.D) + pbase;
  const float* eo = A.ebar_in + pbase;                   // read only when RECOMP (may be the buffer A.ebar writes)
  const float* __restrict__ sump = A.ssum + pbase;       // read only when SUM
  float* xp = A.x + pbase;                               // (LSRV only)
  u32* mwp = A.mask_srv + (pbase >> 5);                  // (LSRV 2 only)
  const u32 t_old = (LSRV == 2) ? A.tau_srv_prev[ti.j] : 0u;
  const float s_old = (LSRV == 3) ? A.scale_srv_prev[ti.j] : 0.0f;
  u32* wsp = A.words_srv + (pbase >> 5);                 // (scaled sign, double-way)
  const int lane = tid & 31, warp = tid >> 5;
  if (ti.cnt == TILE) {
    constexpr int NPRE = 1 + (LSRV != 0 ? 1 : 0) + ((RECOMP || SUM) ? 1 : 0);   // reads ahead of the rows, per iteration
    const int nrows = SUM ? 0 : P.K;
    const int per_it = NPRE + nrows;
    // the prefetch stream: element `pq` of iteration `pit` goes into slot `pslot`
    int pit = 0, pq = 0, pslot = 0;
    auto issue_next = [&]() {
      if (pit < VEC_ITERS) {
        const int i = pit * (THREADS * 4) + tid * 4;
        const float* src;
        if (pq == 0) src = ep + i;
        else if (LSRV != 0 && pq == 1) src = xp + i;
        else if (RECOMP && pq == NPRE - 1) src = eo + i;
        else if (SUM && pq == NPRE - 1) src = sump + i;
        else src = dp + (long long)(pq - NPRE) * P.dpad + i;
        cp_async16(&ring[pslot * THREADS + tid], src);
        if (++pq == per_it) { pq = 0; ++pit; }
        if (++pslot == DENSE_RING) pslot = 0;
      }
      cp_async_commit();                                  // (an empty group past the end keeps the count uniform)
    };
    // the consumer: waits until the oldest outstanding copy has landed, reads it, and issues the next copy
    int cslot = 0;
    auto take = [&]() -> float4 {
      cp_async_wait<DENSE_RING - 2>();
      const float4 v = ring[cslot * THREADS + tid];
      if (++cslot == DENSE_RING) cslot = 0;
      issue_next();
      return v;
    };
#pragma unroll 1
    for (int q = 0; q < DENSE_RING - 1; ++q) issue_next();
#pragma unroll 1
    for (int it = 0; it < VEC_ITERS; ++it) {
      const int i = it * (THREADS * 4) + tid * 4;
      float4 e = take();
      if (LSRV != 0) {
        float4 xv = take();
        const bool q0 = LSRV != 2 || topk_selected(e.x, t_old), q1 = LSRV != 2 || topk_selected(e.y, t_old);
        const bool q2 = LSRV != 2 || topk_selected(e.z, t_old), q3 = LSRV != 2 || topk_selected(e.w, t_old);
        float c0 = q0 ? e.x : 0.0f, c1 = q1 ? e.y : 0.0f, c2 = q2 ? e.z : 0.0f, c3 = q3 ? e.w : 0.0f;
        if (LSRV == 3) { c0 = sign_code(e.x, s_old); c1 = sign_code(e.y, s_old); c2 = sign_code(e.z, s_old); c3 = sign_code(e.w, s_old); }
        xv.x = __fsub_rn(xv.x, c0); xv.y = __fsub_rn(xv.y, c1); xv.z = __fsub_rn(xv.z, c2); xv.w = __fsub_rn(xv.w, c3);
        st4(xp + i, xv);
        e.x = __fsub_rn(e.x, c0); e.y = __fsub_rn(e.y, c1); e.z = __fsub_rn(e.z, c2); e.w = __fsub_rn(e.w, c3);
        if (LSRV == 2) {
          const u32 w = pack_row4(q0, q1, q2, q3);
          if ((lane & 7) == 0) mwp[i >> 5] = w;
        }
      }
      float4 eold = make_float4(0.f, 0.f, 0.f, 0.f);
      if (RECOMP) eold = take();
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      float b0 = 0.f, b1 = 0.f, b2 = 0.f, b3 = 0.f;
      if (SUM) { const float4 sv = take(); a0 = sv.x; a1 = sv.y; a2 = sv.z; a3 = sv.w; }
#pragma unroll 4
      for (int k = 0; k < nrows; ++k) {
        float4 v = take();
        if (RECOMP) {
          v.x = __fmaf_rn(A.eta, v.x, eold.x); v.y = __fmaf_rn(A.eta, v.y, eold.y);
          v.z = __fmaf_rn(A.eta, v.z, eold.z); v.w = __fmaf_rn(A.eta, v.w, eold.w);
        }
        const u32 t = (COMP != 0) ? t_k[k] : 0u;
        float c0, c1, c2, c3;
        if (COMP == 1) {
          const float sk = __uint_as_float(t);
          c0 = sign_code(v.x, sk); c1 = sign_code(v.y, sk); c2 = sign_code(v.z, sk); c3 = sign_code(v.w, sk);
        } else {
          c0 = (COMP == 0 || topk_selected(v.x, t)) ? v.x : 0.0f;
          c1 = (COMP == 0 || topk_selected(v.y, t)) ? v.y : 0.0f;
          c2 = (COMP == 0 || topk_selected(v.z, t)) ? v.z : 0.0f;
          c3 = (COMP == 0 || topk_selected(v.w, t)) ? v.w : 0.0f;
        }
        a0 = __fadd_rn(a0, c0); a1 = __fadd_rn(a1, c1); a2 = __fadd_rn(a2, c2); a3 = __fadd_rn(a3, c3);
        if (AVG) {
          b0 = __fadd_rn(b0, __fsub_rn(v.x, c0)); b1 = __fadd_rn(b1, __fsub_rn(v.y, c1));
          b2 = __fadd_rn(b2, __fsub_rn(v.z, c2)); b3 = __fadd_rn(b3, __fsub_rn(v.w, c3));
        }
      }
      if (AVG) st4(A.ebar + pbase + i, make_float4(div_by_k(P, b0), div_by_k(P, b1), div_by_k(P, b2), div_by_k(P, b3)));
      float4 ds;
      ds.x = __fadd_rn(e.x, div_by_k(P, a0));
      ds.y = __fadd_rn(e.y, div_by_k(P, a1));
      ds.z = __fadd_rn(e.z, div_by_k(P, a2));
      ds.w = __fadd_rn(e.w, div_by_k(P, a3));
      st4(ep + i, ds);
      if (COMP == 2 && lo != NO_GUESS) {
        if (stg.n > CAND_STAGE - 128) stage_flush(stg, A.cand_srv, 0, ti.j);
        stage_row4(stg, lo, mag_key(ds.x), mag_key(ds.y), mag_key(ds.z), mag_key(ds.w));
      }
      if (COMP == 1 && sign_dc) {                          // (uniform over the block)
        lane_add4(acc, ds);
        const u32 w = pack_row4(ds.x >= 0.0f, ds.y >= 0.0f, ds.z >= 0.0f, ds.w >= 0.0f);
        if ((lane & 7) == 0) wsp[i >> 5] = w;
      }
    }
    cp_async_wait<0>();
  } else {
    for (int r = 0; r < ROWS; ++r) {
      const int i = r * THREADS + tid;
      float ds = 0.0f;
      bool qs = false;
      if (i < ti.cnt) {
        float a = SUM ? sump[i] : 0.f, b = 0.f;
        const float ebo = RECOMP ? eo[i] : 0.0f;
        for (int k = 0; k < (SUM ? 0 : P.K); ++k) {
          float v = dp[(long long)k * P.dpad + i];
          if (RECOMP) v = __fmaf_rn(A.eta, v, ebo);
          const float c = (COMP == 1) ? sign_code(v, __uint_as_float(t_k[k]))
                                      : ((COMP == 0 || topk_selected(v, t_k[k])) ? v : 0.0f);
          a = __fadd_rn(a, c);
          if (AVG) b = __fadd_rn(b, __fsub_rn(v, c));
        }
        if (AVG) A.ebar[pbase + i] = div_by_k(P, b);
        float eold = ep[i];
        if (LSRV != 0) {
          qs = LSRV != 2 || topk_selected(eold, t_old);
          const float cs = (LSRV == 3) ? sign_code(eold, s_old) : (qs ? eold : 0.0f);
          xp[i] = __fsub_rn(xp[i], cs);
          eold = __fsub_rn(eold, cs);
        }
        ds = __fadd_rn(eold, div_by_k(P, a));
        ep[i] = ds;
        if (COMP == 1 && sign_dc) lane_add(acc, ds);
      }
      if (LSRV == 2) {
        const u32 w = __ballot_sync(0xffffffffu, qs);
        if (lane == 0 && (r * THREADS + warp * 32) < ti.cnt) mwp[(r * THREADS + warp * 32) >> 5] = w;
      }
      if (COMP == 1 && sign_dc) {
        const u32 w = __ballot_sync(0xffffffffu, i < ti.cnt && ds >= 0.0f);
        if (lane == 0 && (r * THREADS + warp * 32) < ti.cnt) wsp[(r * THREADS + warp * 32) >> 5] = w;
      }
      if (COMP == 2 && lo != NO_GUESS) {
        if (stg.n > CAND_STAGE - 32) stage_flush(stg, A.cand_srv, 0, ti.j);
        stage_row1(stg, lo, i < ti.cnt, mag_key(ds));
      }
    }
  }
  if (COMP == 2) stage_flush(stg, A.cand_srv, 0, ti.j);
  if (COMP == 1 && sign_dc) warp_commit(acc, A.recs_srv + ti.j, A.status);
}

// Between the worker pass and the server pass: one thread per (worker, tensor) record turns the exact
// L1 sum into the scale and clears the record; T more threads clear the server records, which the
// previous step's apply kernel has finished reading.
// scale_srv_pending != null: the previous step's server lines are still pending, so its server scales are
// formed here from the server records before those are cleared (the server pass that follows needs them).
__global__ void __launch_bounds__(THREADS) k_finalize_scales(int K, int T, const int* __restrict__ n, L1Record* recs,
                                                              float* __restrict__ scale_cur, L1Record* recs_srv,
                                                              float* scale_srv_pending) {
  const int q = blockIdx.x * THREADS + threadIdx.x;
  if (q < K * T) {
    L1Record r = recs[q];
    recs[q].limb[0] = 0; recs[q].limb[1] = 0; recs[q].limb[2] = 0;
    scale_cur[q] = scale_from_limbs(r.limb[0], r.limb[1], r.limb[2], n[q % T]);
  } else if (q < K * T + T) {
    L1Record* r = recs_srv + (q - K * T);
    if (scale_srv_pending) scale_srv_pending[q - K * T] = scale_from_limbs(r->limb[0], r->limb[1], r->limb[2], n[q - K * T]);
    r->limb[0] = 0; r->limb[1] = 0; r->limb[2] = 0;
  }
}

// Sharded operation, error averaging (Algorithm 1, pre-step): ebar = (1/K) sum_k e^(k) in k order, with
// e^(k) = D^(k) - C(D^(k)) formed from every owner's stored model differences and scales, read in place
// through row tables (the same subtraction, order and division as the unsharded averaging in k_apply).
// SUM_ONLY (rows = this shard's own workers): the undivided partial sum, for an all-reduce across shards.
// COMP 1: aux_rows[k] -> worker k's [T] scales (float); COMP 2: -> its [T] Top-K thresholds (u32).
template <bool SUM_ONLY, int COMP = 1>
__global__ void __launch_bounds__(THREADS) k_avg_pull(Plan P, const float* const* __restrict__ d_rows,
                                                       const void* const* __restrict__ aux_rows, float* ebar) {
  constexpr int ES = (COMP == 1) ? ESRC_LAZY_SIGN : ESRC_LAZY_TOPK;
  __shared__ float s_k[MAX_WORKERS];
  __shared__ u32 t_k[MAX_WORKERS];
  __shared__ const float* s_row[MAX_WORKERS];
  const TileInfo ti = tile_info(P, blockIdx.x);
  const int tid = threadIdx.x;
  for (int k = tid; k < P.K; k += THREADS) {
    s_k[k] = (COMP == 1) ? reinterpret_cast<const float*>(aux_rows[k])[ti.j] : 0.0f;
    t_k[k] = (COMP == 2) ? reinterpret_cast<const u32*>(aux_rows[k])[ti.j] : 0u;
    s_row[k] = d_rows[k];
  }
  __syncthreads();
  const long long pbase = ti.poff + ti.t0;
  if (ti.cnt == TILE) {
    for (int it = 0; it < VEC_ITERS; ++it) {
      const int i = it * (THREADS * 4) + tid * 4;
      float b0 = 0.f, b1 = 0.f, b2 = 0.f, b3 = 0.f;
#pragma unroll 4
      for (int k = 0; k < P.K; ++k) {
        const float4 v = ld4(s_row[k] + pbase + i);
        const float s = s_k[k];
        const u32 t = t_k[k];
        b0 = __fadd_rn(b0, prev_error<ES>(v.x, s, t));
        b1 = __fadd_rn(b1, prev_error<ES>(v.y, s, t));
        b2 = __fadd_rn(b2, prev_error<ES>(v.z, s, t));
        b3 = __fadd_rn(b3, prev_error<ES>(v.w, s, t));
      }
      if (SUM_ONLY) st4(ebar + pbase + i, make_float4(b0, b1, b2, b3));
      else st4(ebar + pbase + i, make_float4(div_by_k(P, b0), div_by_k(P, b1), div_by_k(P, b2), div_by_k(P, b3)));
    }
  } else {
    for (int i = tid; i < ti.cnt; i += THREADS) {
      float b = 0.f;
      for (int k = 0; k < P.K; ++k) b = __fadd_rn(b, prev_error<ES>(s_row[k][pbase + i], s_k[k], t_k[k]));
      ebar[pbase + i] = SUM_ONLY ? b : div_by_k(P, b);
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// ebar = sum / K over the padded layout (the all-reduced sum of the shards' partial sums)
__global__ void __launch_bounds__(THREADS) k_avg_set(Plan P, const float* __restrict__ sum, float* __restrict__ ebar) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  const long long pbase = ti.poff + ti.t0;
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) ebar[pbase + i] = div_by_k(P, sum[pbase + i]);
}

struct ApplyArgs {
  float* e_srv;            // [dpad] in: Delta_{t+1}, out: e_{t+1}
  float* x;                // [dpad]
  float* ebar;             // [dpad] in: previous uniform error (recompute variant), out: averaged error
  const float* m;          // [K][dpad]
  const float* D;          // [K][dpad]
  const float* scale_cur;  // [K][T]
  float* scale_srv;        // [T] written here (scaled sign) from the server's L1 records
  const L1Record* recs_srv;  // [T]
  const u32* tau_cur;      // [K][T]
  const u32* tau_srv;      // [T]
  u32* mask_srv;           // [nwords] Top-K: server selection of this step

  float eta;
  float* out;              // (OUT) [d], caller layout: the re-updated parameters, or the step-ahead point x - ebar
  const float* ebar_out;   // (OUT 2) [dpad] the uniform local error the point is taken at
};

constexpr int AVG_NONE = 0;
constexpr int AVG_FROM_D = 1;        // e^(k) = D^(k) - C(D^(k)) from the stored model differences
constexpr int AVG_RECOMPUTE = 2;     // D^(k) = fma(eta, m^(k), ebar) recomputed (previous error was uniform)

// COMP: compressor of the workers; SRV: what the server applies (0 identity, 1 sign, 2 Top-K).
template <int COMP, int SRV, int AVG>
__device__ __forceinline__ void apply_elem(float ds, float& x, float& es, bool& sel_srv, float s_srv, u32 t_srv) {
  float cs;
  if (SRV == 1) cs = sign_code(ds, s_srv);
  else if (SRV == 2) { sel_srv = topk_selected(ds, t_srv); cs = sel_srv ? ds : 0.0f; }
  else cs = ds;
  es = __fsub_rn(ds, cs);       // e_{t+1} = Delta - C(Delta)
  x = __fsub_rn(x, cs);         // re-update x_{t+1} = x_t - C(Delta)
}

template <int COMP>
__device__ __forceinline__ float worker_err(float dk, float s, u32 t) {
  if (COMP == 1) return __fsub_rn(dk, sign_code(dk, s));
  if (COMP == 2) return __fsub_rn(dk, topk_selected(dk, t) ? dk : 0.0f);
  return __fsub_rn(dk, dk);
}

// K5: server error, re-update, and (when the next pre-step averages) the averaged worker error.
// OUT (a getter that finds the server lines pending and the local errors uniform): the same pass also writes,
// in the caller's layout, what the getter asked for -- 1: the re-updated parameters x_{t+1}; 2: the step-ahead
// point x_{t+1} - ebar (Algorithm 1, "One step ahead"; the same single subtraction the export kernel does).
template <int COMP, int SRV, int AVG, int OUT = 0>
__global__ void __launch_bounds__(THREADS) k_apply(Plan P, ApplyArgs A) {
  __shared__ float s_k[MAX_WORKERS];
  __shared__ u32 t_k[MAX_WORKERS];
  const TileInfo ti = tile_info(P, blockIdx.x);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (AVG != AVG_NONE) {
    for (int k = tid; k < P.K; k += THREADS) {
      if (COMP == 1) s_k[k] = A.scale_cur[(long long)k * P.T + ti.j];
      if (COMP == 2) t_k[k] = A.tau_cur[(long long)k * P.T + ti.j];
    }
    __syncthreads();
  }
  __shared__ float sh_s_srv;
  if (SRV == 1) {
    // the server's scale of this tensor, from the exact sum the server pass accumulated
    if (tid == 0) {
      const L1Record r = A.recs_srv[ti.j];
      sh_s_srv = scale_from_limbs(r.limb[0], r.limb[1], r.limb[2], ti.n);
      if (ti.t0 == 0) A.scale_srv[ti.j] = sh_s_srv;
    }
    __syncthreads();
  }
  const float s_srv = (SRV == 1) ? sh_s_srv : 0.0f;
  const u32 t_srv = (SRV == 2) ? A.tau_srv[ti.j] : 0u;
  const long long pbase = ti.poff + ti.t0;
  float* ep = A.e_srv + pbase;
  float* xp = A.x + pbase;
  float* ebp = A.ebar + pbase;
  const float* __restrict__ src = (AVG == AVG_RECOMPUTE) ? A.m + pbase : A.D + pbase;
  u32* mwp = A.mask_srv + (pbase >> 5);
  float* op = (OUT != 0) ? A.out + ti.off + ti.t0 : nullptr;              // caller layout: any 4-byte alignment
  const float* __restrict__ eop = (OUT == 2) ? A.ebar_out + pbase : nullptr;
  const bool out_vec = (OUT != 0) && (reinterpret_cast<uintptr_t>(op) & 15) == 0;

  if (ti.cnt == TILE) {
#pragma unroll 2
    for (int it = 0; it < VEC_ITERS; ++it) {
      const int i = it * (THREADS * 4) + tid * 4;
      const float4 ds = ld4(ep + i);
      float4 x = ld4(xp + i), es;
      bool q0 = false, q1 = false, q2 = false, q3 = false;
      apply_elem<COMP, SRV, AVG>(ds.x, x.x, es.x, q0, s_srv, t_srv);
      apply_elem<COMP, SRV, AVG>(ds.y, x.y, es.y, q1, s_srv, t_srv);
      apply_elem<COMP, SRV, AVG>(ds.z, x.z, es.z, q2, s_srv, t_srv);
      apply_elem<COMP, SRV, AVG>(ds.w, x.w, es.w, q3, s_srv, t_srv);
      st4(ep + i, es);
      st4(xp + i, x);
      if (OUT != 0) {
        float4 o = x;
        if (OUT == 2) {
          const float4 eb = ld4(eop + i);
          o.x = __fsub_rn(x.x, eb.x); o.y = __fsub_rn(x.y, eb.y); o.z = __fsub_rn(x.z, eb.z); o.w = __fsub_rn(x.w, eb.w);
        }
        if (out_vec) st4(op + i, o);
        else { op[i] = o.x; op[i + 1] = o.y; op[i + 2] = o.z; op[i + 3] = o.w; }
      }
      if (SRV == 2) {
        u32 w = pack_row4(q0, q1, q2, q3);
        if ((lane & 7) == 0) mwp[i >> 5] = w;
      }
      if (AVG != AVG_NONE) {
        float4 eb = make_float4(0.f, 0.f, 0.f, 0.f);
        if (AVG == AVG_RECOMPUTE) eb = ld4(ebp + i);
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
        for (int k = 0; k < P.K; ++k) {
          float4 v = ld4_stream(src + (long long)k * P.dpad + i);
          if (AVG == AVG_RECOMPUTE) {
            v.x = __fmaf_rn(A.eta, v.x, eb.x); v.y = __fmaf_rn(A.eta, v.y, eb.y);
            v.z = __fmaf_rn(A.eta, v.z, eb.z); v.w = __fmaf_rn(A.eta, v.w, eb.w);
          }
          const float s = (COMP == 1) ? s_k[k] : 0.0f;
          const u32 t = (COMP == 2) ? t_k[k] : 0u;
          a0 = __fadd_rn(a0, worker_err<COMP>(v.x, s, t));
          a1 = __fadd_rn(a1, worker_err<COMP>(v.y, s, t));
          a2 = __fadd_rn(a2, worker_err<COMP>(v.z, s, t));
          a3 = __fadd_rn(a3, worker_err<COMP>(v.w, s, t));
        }
        st4(ebp + i, make_float4(div_by_k(P, a0), div_by_k(P, a1), div_by_k(P, a2), div_by_k(P, a3)));
      }
    }
  } else {
    for (int r = 0; r < ROWS; ++r) {
      const int i = r * THREADS + tid;
      const bool valid = i < ti.cnt;
      bool q = false;
      if (valid) {
        float x = xp[i], es;
        apply_elem<COMP, SRV, AVG>(ep[i], x, es, q, s_srv, t_srv);
        ep[i] = es;
        xp[i] = x;
        if (OUT == 1) op[i] = x;
        if (OUT == 2) op[i] = __fsub_rn(x, eop[i]);
        if (AVG != AVG_NONE) {
          const float eb = (AVG == AVG_RECOMPUTE) ? ebp[i] : 0.0f;
          float a = 0.f;
          for (int k = 0; k < P.K; ++k) {
            float v = src[(long long)k * P.dpad + i];
            if (AVG == AVG_RECOMPUTE) v = __fmaf_rn(A.eta, v, eb);
            a = __fadd_rn(a, worker_err<COMP>(v, (COMP == 1) ? s_k[k] : 0.0f, (COMP == 2) ? t_k[k] : 0u));
          }
          ebp[i] = div_by_k(P, a);
        }
      }
      if (SRV == 2) {
        u32 w = __ballot_sync(0xffffffffu, valid && q);
        if (lane == 0 && (r * THREADS + warp * 32) < ti.cnt) mwp[(r * THREADS + warp * 32) >> 5] = w;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// ---------------------------------------------------------------------------------------------------
// Layout conversion and getters (not on the hot path).
constexpr int EXP_X = 0, EXP_ESRV = 1, EXP_M = 2, EXP_WERR = 3, EXP_STEP_AHEAD = 4;

struct ExportArgs {
  const float* x; const float* e_srv; const float* m; const float* D; const float* ebar;
  const float* scale_last; const u32* tau_last;
  int esrc;      // ESRC_* describing how e^(k) is currently held
  int what;      // EXP_*
  int k;
  int saef;
};

__device__ __forceinline__ float current_error(const ExportArgs& A, const Plan& P, int j, long long p) {
  if (A.esrc == ESRC_UNIFORM) return A.ebar[p];
  const float v = A.D[(long long)A.k * P.dpad + p];
  if (A.esrc == ESRC_LOCAL_D) return v;
  if (A.esrc == ESRC_LAZY_SIGN) return prev_error<ESRC_LAZY_SIGN>(v, A.scale_last[(long long)A.k * P.T + j], 0u);
  return prev_error<ESRC_LAZY_TOPK>(v, 0.0f, A.tau_last[(long long)A.k * P.T + j]);
}

__global__ void __launch_bounds__(THREADS) k_export(Plan P, ExportArgs A, float* __restrict__ out) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) {
    const long long p = ti.poff + ti.t0 + i;
    float v;
    switch (A.what) {
      case EXP_X: v = A.x[p]; break;
      case EXP_ESRV: v = A.e_srv[p]; break;
      case EXP_M: v = A.m[(long long)A.k * P.dpad + p]; break;
      case EXP_WERR: v = current_error(A, P, ti.j, p); break;
      default: v = A.saef ? __fsub_rn(A.x[p], current_error(A, P, ti.j, p)) : A.x[p]; break;
    }
    out[ti.off + ti.t0 + i] = v;
  }
}

// Gradient-mismatch bounds of Section 3 (the quantities plotted in Fig. 3, right; L and sigma ignored):
//   out[0] = || e + ebar ||^2                         (local error feedback; ebar = mean_k e^(k))
//   out[1] = (1/K) sum_k || e + ebar - e^(k) ||^2      (step ahead)
// accumulated in fp64.  current_error needs A.k; it is set per worker inside the loop.
__global__ void __launch_bounds__(THREADS) k_mismatch(Plan P, ExportArgs A, double* out) {
  __shared__ double red[2][THREADS / 32];
  const TileInfo ti = tile_info(P, blockIdx.x);
  double s0 = 0.0, s1 = 0.0;
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) {
    const long long p = ti.poff + ti.t0 + i;
    double sum = 0.0;
    for (int k = 0; k < P.K; ++k) { A.k = k; sum += (double)current_error(A, P, ti.j, p); }
    const double base = (double)A.e_srv[p] + sum / (double)P.K;
    s0 += base * base;
    double acc = 0.0;
    for (int k = 0; k < P.K; ++k) { A.k = k; const double v = base - (double)current_error(A, P, ti.j, p); acc += v * v; }
    s1 += acc / (double)P.K;
  }
  for (int o = 16; o > 0; o >>= 1) { s0 += __shfl_xor_sync(0xffffffffu, s0, o); s1 += __shfl_xor_sync(0xffffffffu, s1, o); }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s0; red[1][threadIdx.x >> 5] = s1; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0;
    for (int w = 0; w < THREADS / 32; ++w) { a += red[0][w]; b += red[1][w]; }
    atomicAdd(out, a);
    atomicAdd(out + 1, b);
  }
}

// caller layout -> padded layout
__global__ void __launch_bounds__(THREADS) k_import(Plan P, const float* __restrict__ in, float* __restrict__ out) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  for (int i = threadIdx.x; i < ti.cnt; i += THREADS) out[ti.poff + ti.t0 + i] = in[ti.off + ti.t0 + i];
}

// Top-K selection of one row as bit words; the row is stored (src.buf) or recomputed (src.m, both already
// offset to the row)
__global__ void __launch_bounds__(THREADS) k_mask_words(Plan P, DeltaSrc src,
                                                         const u32* __restrict__ tau, u32* __restrict__ out) {
  const TileInfo ti = tile_info(P, blockIdx.x);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 t = tau[ti.j];
  const long long pbase = ti.poff + ti.t0;
  for (int r = 0; r < ROWS; ++r) {
    const int i = r * THREADS + tid;
    const bool valid = i < ti.cnt;
    float v = 0.0f;
    if (valid) v = src.recompute ? __fmaf_rn(src.eta, src.m[pbase + i], src.ebar[pbase + i]) : src.buf[pbase + i];
    const bool q = valid && topk_selected(v, t);
    u32 w = __ballot_sync(0xffffffffu, q);
    if (lane == 0 && (r * THREADS + warp * 32) < ti.cnt) out[(pbase + r * THREADS + warp * 32) >> 5] = w;
  }
}

}  // namespace sae
