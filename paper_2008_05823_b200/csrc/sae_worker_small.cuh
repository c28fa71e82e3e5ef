// Worker pass for small problems (the whole K x d state fits L2 several times over: K x dpad <= 2^24).
//
// The persistent, warp-specialised passes are built to stream: a ring of bulk copies, hand-overs between
// producer, averager and worker warps.  On a problem of a few MB every block gets one or two work items, and
// what the pass costs is the chain of dependent steps inside one item -- table look-up, copy, average, worker
// lines -- not bytes.  This kernel is the short chain: a block takes a quarter tile (1024 elements) of one
// tensor for ALL workers, a thread four consecutive elements, and everything is plain loads issued together:
//   the K gradient rows of the quarter tile (caller layout, any alignment: coalesced 4-byte loads through
//   shared memory), then per thread the K momentum rows, the uniform error (or the K stored differences);
//   [pending average, p = 1]  ebar' = (1/K) sum_k ( fma(eta_prev, m_k, ebar) - C(.) ), k in order;
//   worker lines per k: momentum, Delta, exact L1 partial (one warp commit per worker), sign words.
// Same operations in the same order as the streaming passes: same bits.  A block reads and writes only its own
// elements of every row, so the in-place updates of ebar and of the momentum rows need no second buffer.
#pragma once
#include "sae_kernels.cuh"

namespace sae {

constexpr int WS_ELEMS = 1024;                       // elements of one tensor per block (a quarter tile)
constexpr int WS_SUB = TILE / WS_ELEMS;
constexpr int WS_MAXK = 32;                          // gradient staging: K x 4 KB of (dynamic) shared memory
constexpr int WS_B = 4;                              // rows a thread fetches together

struct SmallArgs {
  const float* g;            // [K][d] caller layout
  float* m;                  // [K][dpad]
  float* D;                  // [K][dpad] stored differences (read when lazy, written when WRITE_D)
  float* ebar;               // [dpad] in: uniform error (PENDING: of the step before), out (PENDING): the averaged error
  const float* x;            // [dpad] (weight decay)
  const float* scale_prev;   // [K][T] scales of the previous step (lazy error, pending average)
  u32* words;                // [K][nwords]
  L1Record* recs;            // [K][T]
  u32* status;
  float eta_prev;            // learning rate of the previous step (pending average)
  // Weight decay makes the worker lines read x, so the server lines of the previous step (e = Delta - C(Delta),
  // x = x - C(Delta)) cannot wait for the next server pass as they do otherwise; instead of a kernel of their own
  // they are carried out here, element by element, before x is used (lsrv != 0):
  int lsrv, dc;
  float* e_srv;                    // [dpad] in: the pending Delta, out: the server error
  float* x_rw;                     // [dpad] parameters
  const L1Record* recs_srv_prev;   // [T] exact L1 sums of the pending Delta (double-way)
  float* scale_srv;                // [T] out: the server scales formed from them
};

template <int ESRC, bool WRITE_D, bool WD>
__global__ void __launch_bounds__(THREADS) k_worker_small(Plan P, StepParams sp, SmallArgs A) {
  extern __shared__ float4 ws_smem[];                // [K][WS_ELEMS] floats
  float (*s_g)[WS_ELEMS] = reinterpret_cast<float (*)[WS_ELEMS]>(ws_smem);
  __shared__ float s_scale[WS_MAXK];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x / WS_SUB, sub = blockIdx.x - tile * WS_SUB;
  const TileInfo ti = tile_info(P, tile);
  const int t0 = ti.t0 + sub * WS_ELEMS;
  const int cnt = min(WS_ELEMS, ti.n - t0);
  if (cnt <= 0) return;                              // (the tensor ends inside an earlier quarter of this tile)
  const int K = P.K;
  const long long pbase = ti.poff + t0;
  const long long goff = ti.off + t0;
  // gradients of the quarter tile, all workers: coalesced scalar loads (rows of the caller's layout start anywhere)
#pragma unroll 4
  for (int k = 0; k < K; ++k) {
    const float* gp = A.g + (long long)k * P.d + goff;
#pragma unroll
    for (int q = 0; q < WS_ELEMS / THREADS; ++q) {
      const int i = q * THREADS + tid;
      s_g[k][i] = i < cnt ? __ldcs(gp + i) : 0.0f;
    }
  }
  if (ESRC != ESRC_UNIFORM && tid < K) s_scale[tid] = A.scale_prev[(long long)tid * P.T + ti.j];
  __shared__ float s_srv;
  if (WD && A.lsrv && A.dc && tid == 32) {           // (a thread of another warp than the scale loads)
    const L1Record r = A.recs_srv_prev[ti.j];
    s_srv = scale_from_limbs(r.limb[0], r.limb[1], r.limb[2], ti.n);
    if (t0 == 0) A.scale_srv[ti.j] = s_srv;
  }
  __syncthreads();

  const int e0 = tid * 4;                            // this thread's four elements
  const bool full = e0 + 4 <= cnt;                   // (rows are padded to 32 elements: a partly valid group stays inside
  const bool any = e0 < cnt;                         //  the allocation, its invalid elements are masked below)
  float4 eb = make_float4(0.f, 0.f, 0.f, 0.f), xv = make_float4(0.f, 0.f, 0.f, 0.f);
  if (any) {
    if (ESRC != ESRC_LAZY_SIGN) eb = ld4(A.ebar + pbase + e0);
    if (WD) xv = ld4(A.x + pbase + e0);
    if (WD && A.lsrv) {
      // the pending server lines of these four elements (the operations of the apply kernel), then x as re-updated
      const float4 ds = ld4(A.e_srv + pbase + e0);
      const float ss = A.dc ? s_srv : 0.0f;
      float4 cs;
      cs.x = A.dc ? sign_code(ds.x, ss) : ds.x; cs.y = A.dc ? sign_code(ds.y, ss) : ds.y;
      cs.z = A.dc ? sign_code(ds.z, ss) : ds.z; cs.w = A.dc ? sign_code(ds.w, ss) : ds.w;
      float4 es;
      es.x = __fsub_rn(ds.x, cs.x); es.y = __fsub_rn(ds.y, cs.y); es.z = __fsub_rn(ds.z, cs.z); es.w = __fsub_rn(ds.w, cs.w);
      xv.x = __fsub_rn(xv.x, cs.x); xv.y = __fsub_rn(xv.y, cs.y); xv.z = __fsub_rn(xv.z, cs.z); xv.w = __fsub_rn(xv.w, cs.w);
      if (!full) {                                   // the padding past the end of the tensor stays zero
        if (e0 + 1 >= cnt) { es.y = 0.f; xv.y = 0.f; }
        if (e0 + 2 >= cnt) { es.z = 0.f; xv.z = 0.f; }
        if (e0 + 3 >= cnt) { es.w = 0.f; xv.w = 0.f; }
      }
      st4(A.e_srv + pbase + e0, es);
      st4(A.x_rw + pbase + e0, xv);
    }
  }
  if (ESRC == ESRC_PENDING_AVG && any) {
    // the average the previous step left pending, from the K momentum rows as they stand
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = 0; k0 < K; k0 += WS_B) {           // WS_B rows fetched together, then added in order
      float4 mq[WS_B];
#pragma unroll
      for (int u = 0; u < WS_B; ++u)
        mq[u] = k0 + u < K ? ld4(A.m + (long long)(k0 + u) * P.dpad + pbase + e0) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < WS_B; ++u) {
        if (k0 + u < K) {
          const float4 mk = mq[u];
          const float sk = s_scale[k0 + u];
          float4 dk;
          dk.x = __fmaf_rn(A.eta_prev, mk.x, eb.x); dk.y = __fmaf_rn(A.eta_prev, mk.y, eb.y);
          dk.z = __fmaf_rn(A.eta_prev, mk.z, eb.z); dk.w = __fmaf_rn(A.eta_prev, mk.w, eb.w);
          a.x = __fadd_rn(a.x, __fsub_rn(dk.x, sign_code(dk.x, sk))); a.y = __fadd_rn(a.y, __fsub_rn(dk.y, sign_code(dk.y, sk)));
          a.z = __fadd_rn(a.z, __fsub_rn(dk.z, sign_code(dk.z, sk))); a.w = __fadd_rn(a.w, __fsub_rn(dk.w, sign_code(dk.w, sk)));
        }
      }
    }
    eb = make_float4(div_by_k(P, a.x), div_by_k(P, a.y), div_by_k(P, a.z), div_by_k(P, a.w));
    if (!full) {                                     // the padding past the end of the tensor stays zero
      if (e0 + 1 >= cnt) eb.y = 0.f;
      if (e0 + 2 >= cnt) eb.z = 0.f;
      if (e0 + 3 >= cnt) eb.w = 0.f;
    }
    st4(A.ebar + pbase + e0, eb);
  }
  // worker lines, one worker after the other: its L1 partial is committed per warp
  for (int k0 = 0; k0 < K; k0 += WS_B) {
   // WS_B workers' rows fetched together (nothing written in between that they could alias), then one worker at a time
   float4 mq[WS_B], dq[WS_B];
#pragma unroll
   for (int u = 0; u < WS_B; ++u) {
     const bool in = any && k0 + u < K;
     mq[u] = in ? ld4(A.m + (long long)(k0 + u) * P.dpad + pbase + e0) : make_float4(0.f, 0.f, 0.f, 0.f);
     dq[u] = (in && ESRC == ESRC_LAZY_SIGN) ? ld4(A.D + (long long)(k0 + u) * P.dpad + pbase + e0) : make_float4(0.f, 0.f, 0.f, 0.f);
   }
#pragma unroll
   for (int u = 0; u < WS_B; ++u) {
    const int k = k0 + u;
    if (k >= K) break;                               // (uniform)
    LaneAcc acc; lane_acc_init(acc);
    u32 w = 0u;
    if (any) {
      float* mp = A.m + (long long)k * P.dpad + pbase + e0;
      float* dp = A.D + (long long)k * P.dpad + pbase + e0;
      const float4 mk = mq[u];
      float4 E = eb;
      if (ESRC == ESRC_LAZY_SIGN) {
        const float4 dv = dq[u];
        const float sk = s_scale[k];
        E.x = prev_error<ESRC_LAZY_SIGN>(dv.x, sk, 0u); E.y = prev_error<ESRC_LAZY_SIGN>(dv.y, sk, 0u);
        E.z = prev_error<ESRC_LAZY_SIGN>(dv.z, sk, 0u); E.w = prev_error<ESRC_LAZY_SIGN>(dv.w, sk, 0u);
      }
      const float4 G = *reinterpret_cast<const float4*>(&s_g[k][e0]);
      float4 mn, dl;
      dl.x = worker_update<WD>(G.x, mk.x, E.x, xv.x, sp, mn.x);
      dl.y = worker_update<WD>(G.y, mk.y, E.y, xv.y, sp, mn.y);
      dl.z = worker_update<WD>(G.z, mk.z, E.z, xv.z, sp, mn.z);
      dl.w = worker_update<WD>(G.w, mk.w, E.w, xv.w, sp, mn.w);
      if (!full) {                                   // keep the padding of the rows zero
        if (e0 + 1 >= cnt) { mn.y = 0.f; dl.y = 0.f; }
        if (e0 + 2 >= cnt) { mn.z = 0.f; dl.z = 0.f; }
        if (e0 + 3 >= cnt) { mn.w = 0.f; dl.w = 0.f; }
      }
      st4(mp, mn);
      if (WRITE_D) st4(dp, dl);
      if (full) {
        lane_add4(acc, dl);
      } else {
        lane_add(acc, dl.x);
        if (e0 + 1 < cnt) lane_add(acc, dl.y);
        if (e0 + 2 < cnt) lane_add(acc, dl.z);
        if (e0 + 3 < cnt) lane_add(acc, dl.w);
      }
      w = (dl.x >= 0.0f ? 1u : 0u) | ((e0 + 1 < cnt && dl.y >= 0.0f) ? 2u : 0u) |
          ((e0 + 2 < cnt && dl.z >= 0.0f) ? 4u : 0u) | ((e0 + 3 < cnt && dl.w >= 0.0f) ? 8u : 0u);
    }
    // sign words: a warp covers 128 consecutive elements, four words (whole warp: lanes past the end add nothing)
    w <<= 4 * (lane & 7);
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    w |= __shfl_xor_sync(0xffffffffu, w, 2);
    w |= __shfl_xor_sync(0xffffffffu, w, 4);
    if ((lane & 7) == 0 && any) A.words[(long long)k * P.nwords + ((pbase + e0) >> 5)] = w;
    if (warp * 128 < cnt) warp_commit(acc, A.recs + (long long)k * P.T + ti.j, A.status);    // (warp-uniform)
   }
  }
}

}  // namespace sae
