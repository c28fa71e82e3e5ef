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
// when the tensor is small.  Only large tensors whose window failed queue their tiles on the work list of the
// distributed three-level select (k_topk_hist / k_topk_select per level), whose launches find the list empty
// otherwise.
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
  const int* wlog2;      // [T] log2 of the window's width in key units below last step's threshold; WINDOW_ALL:
                         // the tensor's region holds all of it, every non-zero key is a candidate
};

constexpr int WINDOW_ALL = 32;

constexpr u32 NO_GUESS = 0xffffffffu;
constexpr int CAND_STAGE = 256;   // keys a warp stages in shared memory before one append to global memory

// Lower edge of the window for a previous threshold key: 2^wlog2 key units below it, i.e. 2^(wlog2 - 23) octaves
// (SAE_TOPK_WINDOW_LOG2 = 18, about 2 %, for the large tensors).  With error feedback the entries that were not
// sent keep growing until they cross the threshold, so the density just below it is high (of the order of
// n / threshold): a wide window would overflow the candidate list of a large tensor.  A small tensor's threshold
// -- the k-th largest of few values, k = 1 .. a few hundred -- moves by far more than 2 % from step to step, and
// its region has room to spare (8 k + 1024 keys): its window is up to 8 times wider, and a tensor that fits its
// region whole collects every non-zero key, with or without a guess.
#ifndef SAE_TOPK_WINDOW_LOG2
#define SAE_TOPK_WINDOW_LOG2 18
#endif
__device__ __forceinline__ u32 window_lo(u32 tau_prev, int wlog2) {
  if (wlog2 >= WINDOW_ALL) return 1u;
  if (tau_prev == 0u) return NO_GUESS;                 // no usable guess (first step, or an all-zero tail)
  return tau_prev > (1u << wlog2) ? tau_prev - (1u << wlog2) : 1u;
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
template <int NT = THREADS>
__device__ __forceinline__ void walk_from_top(u32* hist, int bins, u32 rank, u32* part, u32* above, u32* out_bin,
                                              u32* out_rank) {
  const int tid = threadIdx.x;
  const int per = bins / NT;              // 8 or 4 (256 threads), 2 or 1 (1024 threads)
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
    for (int t = 0; t < NT / 32; ++t) { above[t] = run; run += part[t]; }
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
// what the one-launch select left to the distributed select for a pair (its `fallback` word)
constexpr u32 FB_NONE = 0u;       // settled
constexpr u32 FB_VALUES = 1u;     // the window failed on a large tensor: radix select over its values
constexpr u32 FB_LIST = 2u;       // a long candidate list that holds the threshold: radix select over its chunks

// The rows whose Top-K thresholds are wanted: stored ([rows][dpad] in buf), or -- when the worker pass did
// not store the model differences -- recomputed as fma(eta, m^(k), ebar), the operation that formed them.
struct DeltaSrc {
  const float* buf;
  const float* m;
  const float* ebar;
  float eta;
  int recompute;
};

// ++hist[bin] for the lanes with `take` set, one atomic per distinct bin of the warp: the keys of a tensor share
// their leading digits, so plain per-lane atomics would pile up on a few addresses.  Whole warps only.
__device__ __forceinline__ void hist_add_aggregated(u32* hist, u32 bin, bool take) {
  if (!__any_sync(0xffffffffu, take)) return;
  const u32 peers = __match_any_sync(0xffffffffu, take ? bin : 0xffffffffu);
  if (take && (threadIdx.x & 31) == (u32)(__ffs(peers) - 1)) atomicAdd(hist + bin, (u32)__popc(peers));
}

// digit of `key` at a level of the 11 + 10 + 10 radix select, and whether the key lies in the prefix bucket
__device__ __forceinline__ bool radix_digit(u32 key, int level, u32 prefix, u32* digit) {
  if (level == 0) { *digit = key >> 20; return true; }
  if (level == 1) { *digit = (key >> 10) & 1023u; return (key >> 20) == prefix; }
  *digit = key & 1023u;
  return (key >> 10) == prefix;
}

// one key per lane into the level's histogram (`valid` masks lanes past the end).  Plain shared-memory atomics:
// in the distributed select, where a block handles 4096 keys at a time, aggregating equal digits across the
// warp first costs more than the pile-up it avoids (measured: histogram launches 18 -> 30 us).
__device__ __forceinline__ void hist_elem(u32 key, int level, u32 prefix, u32* hist, bool valid = true) {
  u32 digit;
  const bool in = radix_digit(key, level, prefix, &digit);
  if (valid && in) atomicAdd(hist + digit, 1u);
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
        for (int i = tid; i - tid < ti.cnt; i += THREADS) {
          const bool valid = i < ti.cnt;
          const float v = valid ? (src.recompute ? __fmaf_rn(src.eta, bp[i], eb[i]) : bp[i]) : 0.0f;
          hist_elem(mag_key(v), level, prefix, target, valid);
        }
      }
    } else {
      rj = w.x;
      const int row = rj / C.T, j = rj - row * C.T;
      const u32* __restrict__ keys = C.keys + (long long)row * C.stride + C.off[j] + (long long)w.y * CAND_CHUNK;
      const int cnt = min((int)(cand_n[rj] - (u32)w.y * CAND_CHUNK), CAND_CHUNK);
      const u32 prefix = level ? st[rj].prefix : 0u;
      u32* target = sh;
      for (int i = tid; i - tid < cnt; i += THREADS) hist_elem(i < cnt ? keys[i] : 0u, level, prefix, target, i < cnt);
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
// The whole select of one (row, tensor) in one block -- except for the tensors with long candidate regions when
// the distributed select follows anyway: their lists are queued for it chunk by chunk.
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
// (11 + 10 + 10 bits) over their values, read by this block alone; larger ones raise their fallback flag and queue
// their tiles for the distributed select that follows.
constexpr int WIN_BINS = 2048;            // covers 2^19 key units above lo: twice the window below the old threshold
constexpr int SEL_U = 4;                  // loads a thread keeps in flight while it walks a list or a tensor
constexpr int SEL_LONG_REGION = 65536;    // candidate regions above this many keys count as long (see topk_thresholds)
#ifndef SAE_TOPK_INLINE_MAX
#define SAE_TOPK_INLINE_MAX 2048
#endif

// Calls f(key, valid) for every key of a candidate list, the whole block in step (every thread makes the same
// number of calls, so f may use warp-collective operations).  The list is read with 16-byte loads, SEL_U of them
// in flight per thread: a block walks its list alone, and what bounds it is the number of round trips to L2.
template <int NT, class F>
__device__ __forceinline__ void for_each_key(const u32* __restrict__ keys, u32 cnt, F f) {
  const uint4* __restrict__ k4 = reinterpret_cast<const uint4*>(keys);    // (regions start on 16-byte boundaries)
  const u32 n4 = (cnt + 3u) >> 2;
  for (u32 b = 0; b < n4; b += NT * SEL_U) {
    uint4 q[SEL_U];
#pragma unroll
    for (int u = 0; u < SEL_U; ++u) {
      const u32 idx = b + u * NT + threadIdx.x;
      q[u] = idx < n4 ? k4[idx] : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < SEL_U; ++u) {
      const u32 i = (b + u * NT + threadIdx.x) * 4u;
      f(q[u].x, i < cnt); f(q[u].y, i + 1u < cnt); f(q[u].z, i + 2u < cnt); f(q[u].w, i + 3u < cnt);
    }
  }
}

template <int NT>
__global__ void __launch_bounds__(NT) k_topk_select_window(Plan P, CandArgs C, const int* __restrict__ jlist, int nj,
                                                            u32 num, u32 den, DeltaSrc src, const u32* tau_guess,
                                                            u32* tau_out, u32* fallback, u32* fallback_total,
                                                            int inline_max, int chain_min_cap, u32* cand_n, int2* work,
                                                            u32* work_count, int rows) {
  __shared__ u32 sh[HIST_BINS];
  __shared__ u32 part[NT / 32];
  __shared__ u32 above[NT / 32];
  __shared__ u32 sh_bin, sh_rank, sh_above;
  const int tid = threadIdx.x;
  const int row = blockIdx.x / nj, j = jlist[blockIdx.x - row * nj];     // this launch's tensors: jlist[0 .. nj)
  const int rj = row * C.T + j;
  const int n = P.n[j];
  const u32 kk = topk_count_of(n, num, den);
  const u32 cnt = C.count[rj];
  const int wl = C.wlog2[j];
  const bool all = wl >= WINDOW_ALL;      // the list holds every non-zero key of the tensor
  const int shift = all ? 0 : wl - 10;    // bin width of pass 1: 1024 bins span the window below the old threshold
  const u32 lo = window_lo(tau_guess[rj], wl);
  const bool ok = lo != NO_GUESS && cnt <= (u32)C.cap[j] && cnt >= kk;
  for (int b = tid; b < HIST_BINS; b += NT) sh[b] = 0u;
  if (tid == 0) sh_above = 0u;
  __syncthreads();
  if (tid == 0) C.count[rj] = 0u;         // (every thread has read the cursor: the barrier above)
  if (ok && C.cap[j] > chain_min_cap) {
    // A long list: one block would be bound by its shared-memory atomics (tens of microseconds for 10^5 keys).
    // Its chunks go to the work list of the distributed select, which spreads them over the device.
    if (tid == 0) {
      cand_n[rj] = cnt;
      fallback[rj] = FB_LIST;
      const u32 chunks = (cnt + CAND_CHUNK - 1) / CAND_CHUNK;
      const u32 base = atomicAdd(work_count, chunks);
      for (u32 c = 0; c < chunks; ++c) work[base + c] = make_int2(rj, (int)c);
    }
    return;
  }
  if (ok) {
    const u32* __restrict__ keys = C.keys + (long long)row * C.stride + C.off[j];
    const u32 RANGE = all ? 0u : ((u32)WIN_BINS << shift);
    u32 mine = 0;
    if (!all)
      for_each_key<NT>(keys, cnt, [&](u32 key, bool valid) {
        const u32 rel = key - lo;
        if (valid) {
          if (rel >= RANGE) ++mine;
          else atomicAdd(sh + (rel >> shift), 1u);
        }
      });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((tid & 31) == 0 && mine) atomicAdd(&sh_above, mine);
    __syncthreads();
    const u32 over = all ? cnt : sh_above;   // (uniform: every thread reads the same count)
    if (kk > over) {
      walk_from_top<NT>(sh, WIN_BINS, kk - over, part, above, &sh_bin, &sh_rank);     // (clears the bins)
      const u32 bin = sh_bin, rank = sh_rank;
      for_each_key<NT>(keys, cnt, [&](u32 key, bool valid) {
        const u32 rel = key - lo;
        if (valid && (rel >> shift) == bin) atomicAdd(sh + (rel & ((1u << shift) - 1u)), 1u);
      });
      __syncthreads();
      walk_from_top<NT>(sh, shift > 10 ? HIST_BINS : 1024, rank, part, above, &sh_bin, &sh_rank);
      if (tid == 0) {
        tau_out[rj] = lo + (bin << shift) + sh_bin;
        fallback[rj] = FB_NONE;
      }
      return;
    }
    // The threshold rose past the binned range: it is the kk-th largest of the list's keys above the range
    // (a heavy tail spread over many octaves).  Three radix levels over those keys, still from the list.
    __syncthreads();
    for (int b = tid; b < HIST_BINS; b += NT) sh[b] = 0u;
    __syncthreads();
    u32 prefix = 0u, rank = kk;
    for (int level = 0; level < 3; ++level) {
      for_each_key<NT>(keys, cnt, [&](u32 key, bool valid) {
        u32 digit;
        const bool in = radix_digit(key, level, prefix, &digit);
        hist_add_aggregated(sh, digit, valid && key - lo >= RANGE && in);
      });
      __syncthreads();
      walk_from_top<NT>(sh, level == 0 ? HIST_BINS : 1024, rank, part, above, &sh_bin, &sh_rank);
      prefix = (level == 0) ? sh_bin : ((prefix << 10) | sh_bin);
      rank = sh_rank;
      __syncthreads();                    // (sh_bin / sh_rank are rewritten by the next level)
    }
    if (tid == 0) { tau_out[rj] = prefix; fallback[rj] = FB_NONE; }
    return;
  }
  // ---- the window failed ----
  if (tid == 0) atomicAdd(fallback_total, 1u);
  if (n > inline_max) {                       // a large tensor: its tiles to the distributed select
    const int tiles = (n + TILE - 1) / TILE;
    if (tid == 0) {
      fallback[rj] = FB_VALUES;
      sh_bin = atomicAdd(work_count, (u32)tiles);
    }
    __syncthreads();
    const u32 base = sh_bin;
    const int first = P.first_tile[j];
    for (int t = tid; t < tiles; t += NT) work[base + t] = make_int2((first + t) * rows + row, -1);
    return;
  }
  if (tid == 0) fallback[rj] = FB_NONE;
  const float* __restrict__ bp = (src.recompute ? src.m : src.buf) + (long long)row * P.dpad + P.poff[j];
  const float* __restrict__ eb = src.ebar + P.poff[j];               // read only when recomputing
  u32 prefix = 0u, rank = kk;
  for (int level = 0; level < 3; ++level) {
    // (tensors start on 128-byte boundaries in the padded layout and their padding is zero: 16-byte loads may run
    // up to three elements past n, and those are masked)
    const int n4 = (n + 3) >> 2;
    for (int b0 = 0; b0 < n4; b0 += NT * SEL_U) {
      float4 vq[SEL_U], eq[SEL_U];
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) {
        const int idx = b0 + u * NT + tid;
        vq[u] = idx < n4 ? ld4(bp + 4 * idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        eq[u] = (src.recompute && idx < n4) ? ld4(eb + 4 * idx) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < SEL_U; ++u) {
        const int i = 4 * (b0 + u * NT + tid);
        const float v[4] = {vq[u].x, vq[u].y, vq[u].z, vq[u].w}, e[4] = {eq[u].x, eq[u].y, eq[u].z, eq[u].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const u32 key = mag_key(src.recompute ? __fmaf_rn(src.eta, v[c], e[c]) : v[c]);
          u32 digit;
          const bool in = radix_digit(key, level, prefix, &digit);
          hist_add_aggregated(sh, digit, i + c < n && in);
        }
      }
    }
    __syncthreads();
    walk_from_top<NT>(sh, level == 0 ? HIST_BINS : 1024, rank, part, above, &sh_bin, &sh_rank);
    prefix = (level == 0) ? sh_bin : ((prefix << 10) | sh_bin);
    rank = sh_rank;
    __syncthreads();                      // (sh_bin / sh_rank are rewritten by the next level)
  }
  if (tid == 0) tau_out[rj] = prefix;
}

}  // namespace sae
