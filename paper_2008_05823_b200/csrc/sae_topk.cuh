// Top-K threshold (Section 3.1): the exact k-th largest 31-bit magnitude key of every (row, tensor).
//
// The select itself is a three-level radix select (11 + 10 + 10 bits): level L histograms the digit of
// every key whose higher digits equal the prefix found so far, a select kernel then walks the histogram
// from the top.  What differs is where the keys come from:
//
// Fast path -- candidate window.  The threshold moves slowly from one step to the next, so the pass
// that produces the values (the worker pass for the workers' Delta^(k), the dense server pass for the
// server's Delta) also appends every key >= lo to a per-(row, tensor) candidate list, where lo lies a
// little below last step's threshold.  If the list did not overflow and holds at least k keys, the
// k-th largest key of the tensor is the k-th largest key of the list: the select reads the short list
// and makes no further pass over the data.
//
// Fallback -- the select reads the values themselves, only for the (row, tensor) pairs whose window
// failed (first step, a jump of the threshold, ties, zeros).  Both paths give the same exact key.
//
// One launch settles the common case (k_topk_select_window: one block per (row, tensor)): a list that holds the
// threshold is resolved by two histogram passes over it in shared memory -- the keys of a list lie in a narrow
// window above `lo`, so they are binned by their distance from `lo` and spread evenly over the bins -- and a
// pair whose window failed is resolved by the same block with the three-level radix select over its values
// when the tensor is small.  Only large tensors whose window failed go to the work list of the distributed
// three-level select (k_topk_worklist, then k_topk_hist / k_topk_select per level), whose launches find the
// list empty otherwise.
#pragma once
#include "sae_device.cuh"

namespace sae {

struct CandArgs {
  u32* keys;             // [rows][stride] candidate keys
  const long long* off;  // [T] start of tensor j's region inside a row
  const int* cap;        // [T] capacity of that region
  long long stride;      // keys per row
  u32* count;            // [rows][T] append cursors (may run past cap: that is the overflow signal)
  int T;
};

constexpr u32 NO_GUESS = 0xffffffffu;
constexpr int CAND_STAGE = 256;   // keys a warp stages in shared memory before one append to global memory

// Lower edge of the window for a previous threshold key: 2^SAE_TOPK_WINDOW_LOG2 key units below it, i.e.
// 2^(SAE_TOPK_WINDOW_LOG2 - 23) octaves (the default 18 is about 2 %).  With error feedback the entries
// that were not sent keep growing until they cross the threshold, so the density just below it is high
// (of the order of n / threshold): a wide window would overflow the candidate list.
#ifndef SAE_TOPK_WINDOW_LOG2
#define SAE_TOPK_WINDOW_LOG2 18
#endif
__device__ __forceinline__ u32 window_lo(u32 tau_prev) {
  if (tau_prev == 0u) return NO_GUESS;                 // no usable guess (first step, or an all-zero tail)
  return tau_prev > (1u << SAE_TOPK_WINDOW_LOG2) ? tau_prev - (1u << SAE_TOPK_WINDOW_LOG2) : 1u;
}

// Per-warp staging of candidate keys in shared memory; `n` is warp-uniform.
struct WarpStage {
  u32* buf;   // CAND_STAGE keys owned by this warp
  int n;
};

// Appends the staged keys of (row, j) to its global list: one atomic per flush.
__device__ __forceinline__ void stage_flush(WarpStage& st, const CandArgs& C, int row, int j) {
  if (st.n == 0) return;
  const int lane = threadIdx.x & 31;
  __syncwarp();
  u32 base = 0;
  if (lane == 0) base = atomicAdd(C.count + (long long)row * C.T + j, (u32)st.n);
  base = __shfl_sync(0xffffffffu, base, 0);
  const u32 cap = (u32)C.cap[j];
  u32* dst = C.keys + (long long)row * C.stride + C.off[j];
  for (int i = lane; i < st.n; i += 32)
    if (base + (u32)i < cap) dst[base + (u32)i] = st.buf[i];
  __syncwarp();
  st.n = 0;
}

// Stages the keys of one 128-element row (four per lane) that lie in the window.  The caller flushes
// whenever fewer than 128 free slots remain, so a whole row always fits.
__device__ __forceinline__ void stage_row4(WarpStage& st, u32 lo, u32 k0, u32 k1, u32 k2, u32 k3) {
  const u32 full = 0xffffffffu;
  const u32 b0 = __ballot_sync(full, k0 >= lo), b1 = __ballot_sync(full, k1 >= lo);
  const u32 b2 = __ballot_sync(full, k2 >= lo), b3 = __ballot_sync(full, k3 >= lo);
  if ((b0 | b1 | b2 | b3) == 0u) return;
  const u32 lt = (1u << (threadIdx.x & 31)) - 1u;
  const int o1 = __popc(b0), o2 = o1 + __popc(b1), o3 = o2 + __popc(b2);
  if (k0 >= lo) st.buf[st.n + __popc(b0 & lt)] = k0;
  if (k1 >= lo) st.buf[st.n + o1 + __popc(b1 & lt)] = k1;
  if (k2 >= lo) st.buf[st.n + o2 + __popc(b2 & lt)] = k2;
  if (k3 >= lo) st.buf[st.n + o3 + __popc(b3 & lt)] = k3;
  st.n += o3 + __popc(b3);
}

// one key per lane (scalar paths)
__device__ __forceinline__ void stage_row1(WarpStage& st, u32 lo, bool valid, u32 key) {
  const u32 b = __ballot_sync(0xffffffffu, valid && key >= lo);
  if (b == 0u) return;
  if (valid && key >= lo) st.buf[st.n + __popc(b & ((1u << (threadIdx.x & 31)) - 1u))] = key;
  st.n += __popc(b);
}

__device__ __forceinline__ u32 topk_count_of(int n, u32 num, u32 den) {
  unsigned long long kk = ((unsigned long long)n * num) / den;
  if (kk < 1) kk = 1;
  if (kk > (unsigned long long)n) kk = n;
  return (u32)kk;
}

// ---------------------------------------------------------------------------------------------------
struct SelectState {     // per (row, tensor)
  u32 prefix;            // digits found so far, right-aligned
  u32 rank;              // rank (1-based, from the top) still to find inside the prefix bucket
};

constexpr int HIST_BINS = 2048;

// Walks a histogram of `bins` (1024 or 2048) counters from the top: returns in *bin the bin that holds the
// rank-th entry and in *rank_in the rank inside it.  Block-wide; hist may be shared or global memory;
// the counters are cleared.  part/above: THREADS words of shared memory each.
__device__ __forceinline__ void walk_from_top(u32* hist, int bins, u32 rank, u32* part, u32* above, u32* out_bin,
                                              u32* out_rank) {
  const int tid = threadIdx.x;
  const int per = bins / THREADS;         // 8 or 4
  u32 c[8];
  u32 sum = 0;
  for (int q = 0; q < per; ++q) {
    const int b = bins - 1 - (tid * per + q);
    c[q] = hist[b];
    hist[b] = 0u;
    sum += c[q];
  }
  // exclusive prefix sum of the per-thread sums over the block: shuffle scan inside each warp, then the
  // warp totals
  const int lane = tid & 31, wrp = tid >> 5;
  u32 inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u32 v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  if (lane == 31) part[wrp] = inc;
  __syncthreads();
  if (tid == 0) {
    u32 run = 0;
    for (int t = 0; t < THREADS / 32; ++t) { above[t] = run; run += part[t]; }
  }
  __syncthreads();
  u32 run = above[wrp] + inc - sum;
  if (run < rank && rank <= run + sum) {
    for (int q = 0; q < per; ++q) {
      if (rank <= run + c[q]) {
        *out_bin = (u32)(bins - 1 - (tid * per + q));
        *out_rank = rank - run;
        break;
      }
      run += c[q];
    }
  }
  __syncthreads();
}

// Both paths feed the same per-(row, tensor) radix select.  Its input is a work list of items:
//   y <  0: data item x = tile * rows + row of a pair whose window failed (keys come from the values);
//   y >= 0: chunk y (CAND_CHUNK keys) of the candidate list of pair x = row * T + j.
constexpr int CAND_CHUNK = 4096;

// One thread per (row, tensor): decides whether the candidate window holds the threshold, queues the
// candidate chunks if so, raises the fallback flag otherwise, and resets the cursor.
__global__ void __launch_bounds__(THREADS) k_topk_decide(CandArgs C, int rows, const int* __restrict__ n, u32 num, u32 den,
                                                          const u32* __restrict__ tau_guess, u32* cand_n, u32* fallback,
                                                          u32* fallback_total, int2* work, u32* work_count) {
  const int rj = blockIdx.x * THREADS + threadIdx.x;
  if (rj >= rows * C.T) return;
  const int j = rj % C.T;
  const u32 cnt = C.count[rj];
  const u32 kk = topk_count_of(n[j], num, den);
  const bool ok = window_lo(tau_guess[rj]) != NO_GUESS && cnt <= (u32)C.cap[j] && cnt >= kk;
  C.count[rj] = 0u;
  cand_n[rj] = ok ? cnt : 0u;
  fallback[rj] = ok ? 0u : 1u;
  if (!ok) { atomicAdd(fallback_total, 1u); return; }
  const u32 chunks = (cnt + CAND_CHUNK - 1) / CAND_CHUNK;
  const u32 base = atomicAdd(work_count, chunks);
  for (u32 c = 0; c < chunks; ++c) work[base + c] = make_int2(rj, (int)c);
}

// Queues every (tile, row) data item whose (row, tensor) raised the fallback flag.
__global__ void __launch_bounds__(THREADS) k_topk_worklist(Plan P, int rows, const u32* __restrict__ fallback, int2* work,
                                                            u32* work_count) {
  const long long nitems = (long long)P.ntiles * rows;
  const long long mine = (long long)blockIdx.x * THREADS + threadIdx.x;
  if (mine >= nitems) return;
  const int tile = (int)(mine / rows);
  const int k = (int)(mine - (long long)tile * rows);
  if (fallback[(long long)k * P.T + P.tile_tensor[tile]]) work[atomicAdd(work_count, 1u)] = make_int2((int)mine, -1);
}

// The rows whose Top-K thresholds are wanted: stored ([rows][dpad] in buf), or -- when the worker pass did
// not store the model differences -- recomputed as fma(eta, m^(k), ebar), the operation that formed them.
struct DeltaSrc {
  const float* buf;
  const float* m;
  const float* ebar;
  float eta;
  int recompute;
};

__device__ __forceinline__ void hist_elem(u32 key, int level, u32 prefix, u32* hist) {
  if (level == 0) atomicAdd(hist + (key >> 20), 1u);
  else if (level == 1) { if ((key >> 20) == prefix) atomicAdd(hist + ((key >> 10) & 1023u), 1u); }
  else { if ((key >> 10) == prefix) atomicAdd(hist + (key & 1023u), 1u); }
}

// Level L histogram over the work list (a fixed grid of blocks strides over it).  Every item accumulates
// in shared memory first (the candidates of a pair nearly all share their leading digits, so direct
// global atomics would pile up on a few addresses) and adds its non-zero bins to the pair's histogram.
// hist is [rows][T][HIST_BINS]
__global__ void __launch_bounds__(THREADS) k_topk_hist(Plan P, CandArgs C, int rows, int level, DeltaSrc src,
                                                        const u32* __restrict__ cand_n, const SelectState* __restrict__ st,
                                                        u32* hist, const int2* __restrict__ work,
                                                        const u32* __restrict__ work_count) {
  __shared__ u32 sh[HIST_BINS];
  const int tid = threadIdx.x;
  const u32 nwork = *work_count;
  for (u32 q = blockIdx.x; q < nwork; q += gridDim.x) {
    const int2 w = work[q];
    int rj;
    const int bins = level == 0 ? HIST_BINS : 1024;
    for (int b = tid; b < bins; b += THREADS) sh[b] = 0u;
    __syncthreads();
    if (w.y < 0) {
      const int tile = w.x / rows;
      const int k = w.x - tile * rows;
      const TileInfo ti = tile_info(P, tile);
      rj = k * P.T + ti.j;
      const float* __restrict__ bp = (src.recompute ? src.m : src.buf) + (long long)k * P.dpad + ti.poff + ti.t0;
      const float* __restrict__ eb = src.ebar + ti.poff + ti.t0;     // read only when recomputing
      const u32 prefix = level ? st[rj].prefix : 0u;
      u32* target = sh;
      if (ti.cnt == TILE) {
#pragma unroll
        for (int it = 0; it < VEC_ITERS; ++it) {
          float4 v = ld4(bp + it * (THREADS * 4) + tid * 4);
          if (src.recompute) {
            const float4 e = ld4(eb + it * (THREADS * 4) + tid * 4);
            v.x = __fmaf_rn(src.eta, v.x, e.x); v.y = __fmaf_rn(src.eta, v.y, e.y);
            v.z = __fmaf_rn(src.eta, v.z, e.z); v.w = __fmaf_rn(src.eta, v.w, e.w);
          }
          hist_elem(mag_key(v.x), level, prefix, target);
          hist_elem(mag_key(v.y), level, prefix, target);
          hist_elem(mag_key(v.z), level, prefix, target);
          hist_elem(mag_key(v.w), level, prefix, target);
        }
      } else {
        for (int i = tid; i < ti.cnt; i += THREADS)
          hist_elem(mag_key(src.recompute ? __fmaf_rn(src.eta, bp[i], eb[i]) : bp[i]), level, prefix, target);
      }
    } else {
      rj = w.x;
      const int row = rj / C.T, j = rj - row * C.T;
      const u32* __restrict__ keys = C.keys + (long long)row * C.stride + C.off[j] + (long long)w.y * CAND_CHUNK;
      const int cnt = min((int)(cand_n[rj] - (u32)w.y * CAND_CHUNK), CAND_CHUNK);
      const u32 prefix = level ? st[rj].prefix : 0u;
      u32* target = sh;
      for (int i = tid; i < cnt; i += THREADS) hist_elem(keys[i], level, prefix, target);
    }
    __syncthreads();
    u32* gh = hist + (long long)rj * HIST_BINS;
    for (int b = tid; b < bins; b += THREADS) {
      const u32 c = sh[b];
      if (c) atomicAdd(gh + b, c);
    }
    __syncthreads();
  }
}

// One block per (row, tensor): find the bin holding the rank-th largest key, update prefix/rank, clear
// the histogram.  After level 2 the prefix is the threshold key itself (and the work list is released).
__global__ void __launch_bounds__(THREADS) k_topk_select(int T, int level, const int* __restrict__ n, u32 num, u32 den,
                                                          u32* hist, SelectState* st, u32* tau, u32* work_count,
                                                          const u32* __restrict__ fallback) {
  __shared__ u32 part[THREADS];
  __shared__ u32 above[THREADS];
  __shared__ u32 sh_bin, sh_rank;
  const int rj = blockIdx.x;              // row * T + j
  const int j = rj % T;
  if (level == 2 && rj == 0 && threadIdx.x == 0) *work_count = 0u;      // (nobody reads the list any more)
  if (!fallback[rj]) return;              // settled by k_topk_select_window: nothing was queued for this pair
  const u32 rank = (level == 0) ? topk_count_of(n[j], num, den) : st[rj].rank;
  const u32 old_prefix = (level == 0) ? 0u : st[rj].prefix;
  __syncthreads();
  walk_from_top(hist + (long long)rj * HIST_BINS, level == 0 ? HIST_BINS : 1024, rank, part, above, &sh_bin, &sh_rank);
  if (threadIdx.x == 0) {
    const u32 prefix = (level == 0) ? sh_bin : ((old_prefix << 10) | sh_bin);
    st[rj].prefix = prefix;
    st[rj].rank = sh_rank;
    if (level == 2) tau[rj] = prefix;
  }
}

// ---------------------------------------------------------------------------------------------------
// The whole select of one (row, tensor) in one block.
//
// Window path (the list did not overflow and holds at least k keys, so the k-th largest key of the tensor is
// the k-th largest key of the list): every key of the list is >= lo.  Pass 1 bins rel = key - lo in steps of
// 2^WIN_SHIFT over WIN_BINS bins and counts the keys above that range (the bulk of the selected entries: a
// heavy tail, counted per thread and reduced, not binned); the rank that is left is located from the top of
// the histogram.  Pass 2 bins the keys of that one bin by their low WIN_SHIFT bits, which gives the exact key.
// If the k-th largest key lies above the binned range (the threshold rose by more than the range in one step)
// the pair is treated like a failed window.
//
// Failed window: tensors of at most inline_max elements are settled here by the three-level radix select
// (11 + 10 + 10 bits) over their values, read by this block alone; larger ones raise their fallback flag for
// the distributed select that follows.
constexpr int WIN_SHIFT = 8;
constexpr int WIN_BINS = 2048;            // covers 2^19 key units above lo: twice the window below the old threshold

__global__ void __launch_bounds__(THREADS) k_topk_select_window(Plan P, CandArgs C, int rows, u32 num, u32 den,
                                                                 DeltaSrc src, const u32* tau_guess, u32* tau_out,
                                                                 u32* fallback, u32* fallback_total, int inline_max) {
  __shared__ u32 sh[HIST_BINS];
  __shared__ u32 part[THREADS];
  __shared__ u32 above[THREADS];
  __shared__ u32 sh_bin, sh_rank, sh_above;
  const int tid = threadIdx.x;
  const int rj = blockIdx.x;              // row * T + j
  const int row = rj / C.T, j = rj - row * C.T;
  const int n = P.n[j];
  const u32 kk = topk_count_of(n, num, den);
  const u32 cnt = C.count[rj];
  const u32 lo = window_lo(tau_guess[rj]);
  bool ok = lo != NO_GUESS && cnt <= (u32)C.cap[j] && cnt >= kk;
  for (int b = tid; b < HIST_BINS; b += THREADS) sh[b] = 0u;
  if (tid == 0) sh_above = 0u;
  __syncthreads();
  if (tid == 0) C.count[rj] = 0u;         // (every thread has read the cursor: the barrier above)
  if (ok) {
    const u32* __restrict__ keys = C.keys + (long long)row * C.stride + C.off[j];
    u32 mine = 0;
    for (u32 i = tid; i < cnt; i += THREADS) {
      const u32 rel = keys[i] - lo;
      if (rel >= ((u32)WIN_BINS << WIN_SHIFT)) ++mine;
      else atomicAdd(sh + (rel >> WIN_SHIFT), 1u);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((tid & 31) == 0 && mine) atomicAdd(&sh_above, mine);
    __syncthreads();
    const u32 over = sh_above;
    if (kk <= over) {
      ok = false;                         // (uniform: every thread reads the same count)
      __syncthreads();
      for (int b = tid; b < HIST_BINS; b += THREADS) sh[b] = 0u;
      __syncthreads();
    } else {
      walk_from_top(sh, WIN_BINS, kk - over, part, above, &sh_bin, &sh_rank);     // (clears the bins)
      const u32 bin = sh_bin, rank = sh_rank;
      for (u32 i = tid; i < cnt; i += THREADS) {
        const u32 rel = keys[i] - lo;
        if ((rel >> WIN_SHIFT) == bin) atomicAdd(sh + (rel & ((1u << WIN_SHIFT) - 1u)), 1u);
      }
      __syncthreads();
      walk_from_top(sh, 1024, rank, part, above, &sh_bin, &sh_rank);
      if (tid == 0) {
        tau_out[rj] = lo + (bin << WIN_SHIFT) + sh_bin;
        fallback[rj] = 0u;
      }
      return;
    }
  }
  // ---- the window failed ----
  if (tid == 0) atomicAdd(fallback_total, 1u);
  if (n > inline_max) {
    if (tid == 0) fallback[rj] = 1u;      // a large tensor: left to the distributed select
    return;
  }
  if (tid == 0) fallback[rj] = 0u;
  const float* __restrict__ bp = (src.recompute ? src.m : src.buf) + (long long)row * P.dpad + P.poff[j];
  const float* __restrict__ eb = src.ebar + P.poff[j];               // read only when recomputing
  u32 prefix = 0u, rank = kk;
  for (int level = 0; level < 3; ++level) {
    for (int i = tid; i < n; i += THREADS)
      hist_elem(mag_key(src.recompute ? __fmaf_rn(src.eta, bp[i], eb[i]) : bp[i]), level, prefix, sh);
    __syncthreads();
    walk_from_top(sh, level == 0 ? HIST_BINS : 1024, rank, part, above, &sh_bin, &sh_rank);
    prefix = (level == 0) ? sh_bin : ((prefix << 10) | sh_bin);
    rank = sh_rank;
    __syncthreads();                      // (sh_bin / sh_rank are rewritten by the next level)
  }
  if (tid == 0) tau_out[rj] = prefix;
}

}  // namespace sae
