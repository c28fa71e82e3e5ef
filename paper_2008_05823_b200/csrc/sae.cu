// Host side of libsae: configuration checks, the segment/tile planner, state allocation and the
// per-iteration launch sequence of Algorithm 1.  Declarations and argument contracts: include/sae.h.
#include "../../include/sae.h"
#include "sae_kernels.cuh"
#include "sae_worker_tma.cuh"
#include "sae_worker_fused.cuh"
#include "sae_worker_small.cuh"
#include "sae_shard_topk.cuh"

#include <cuda.h>
#include <cudaTypedefs.h>
#include <nvtx3/nvToolsExt.h>      // header-only: ranges cost nothing unless a profiler has injected itself
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <unistd.h>
#include <new>
#include <vector>

// folded Top-K forms: the workers' threshold select on a second stream beside the server pass and its select
// small problems: the short-chain worker pass instead of the persistent ones
#ifndef SAE_SMALL_WORKER
#define SAE_SMALL_WORKER 1
#endif
#ifndef SAE_TOPK_PARALLEL_SELECT
#define SAE_TOPK_PARALLEL_SELECT 1
#endif
// scaled sign, p = 1: from this many workers on, the server pass of a step is folded into the next worker pass
#ifndef SAE_SIGN_FOLD_MIN_K
#define SAE_SIGN_FOLD_MIN_K 16
#endif

using namespace sae;

namespace {

thread_local int g_init_cuda_error = 0;

enum Slot { S_WORKER = 0, S_SERVER, S_APPLY, S_TOPK_HIST, S_TOPK_SELECT, S_EXPORT, S_IMPORT, S_MASK, S_FINALIZE, S_COUNT };
const char* const kSlotNames[SAE_NUM_KERNELS] = {"worker_pass", "server_aggregate", "apply_update", "topk_hist",
                                                 "topk_select", "export", "import", "mask_words",
                                                 "finalize_scales", "", "", ""};

struct EventPair { int slot; cudaEvent_t a, b; };

struct StepGraphKey { int esrc, last, avg_after, srv_pending, rot, comm, tail, fresh, reader; const float* grads; float lr, eta_prev; };
struct StepGraph { StepGraphKey key; cudaGraphExec_t exec; int kernels, esrc_after, last_after, pending_after, rot_after, tail_after, fresh_after; uint64_t stamp; };

}  // namespace

struct sae_handle {
  sae_config cfg;
  std::vector<int64_t> sizes;
  Plan P;
  int device;
  cudaStream_t stream;
  // tables
  int *d_tile_tensor, *d_first_tile, *d_n;
  long long *d_off, *d_poff;
  // state
  float *x, *e_srv, *ebar, *m, *D;
  CUtensorMap tm_m;      // momentum rows [K][dpad] as a tensor map (folded-averaging worker pass)
  CUtensorMap tm_D;      // stored model differences [K][dpad] (folded Top-K tail with stored differences)
  int fused_gen_ok;      // Top-K, p != 1, K = 8 or 16: the tail of a non-averaging step is folded into the next worker pass
  u32 *words, *words_srv, *mask_srv;
  float *scale[2], *scale_srv;
  u32 *tau[2], *tau_srv;
  L1Record *recs, *recs_srv;
  // inline_fin: the worker records alternate between two buffers with the step parity and the server records
  // rotate through this step's, the previous step's (still needed while its server lines are pending) and
  // the one the server pass clears for the next step -- four buffers rather than three, so that the rotation
  // has a period that divides the usual gradient-ring lengths and few distinct step graphs exist
  L1Record *recs_alt, *recs_srv_alt, *recs_srv_alt2, *recs_srv_alt3;
  int rot;
  int srv_pending;         // the last step's server lines (e = Delta - C(Delta), x -= C(Delta)) are still owed:
                           // e_srv holds Delta, the server records hold its L1 sum; the next server pass
                           // (or flush_server, before anything reads x or e) carries them out
  int inline_fin;          // small problem: the server pass forms the worker scales itself (one launch fewer)
  int small_worker;        // ... and the worker pass is the short-chain kernel (k_worker_small)
  u32 *hist;
  SelectState* sel;
  // Top-K candidate windows: key lists, per-tensor region offsets / capacities, cursors, fallback flags
  u32 *cand_keys, *cand_keys_srv, *cand_count, *cand_count_srv, *fb, *fb_srv, *fb_total;
  long long* d_cand_off;
  int* d_cand_cap;
  int* d_sel_list;       // [T] the order in which the one-launch select takes the tensors
  int n_sel_long;        // how many of them (the first ones) have long candidate regions
  int n_sel_long_srv;    // the same for the server's row, which counts shorter regions as long (see topk_thresholds)
  int* d_wlog2;          // [T] width of each tensor's candidate window (log2 of key units; WINDOW_ALL: whole tensor)
  int2* work;            // work list of the radix select: data items and candidate chunks
  u32* work_count;
  u32* cand_n;           // [K][T] candidates captured for this step's select
  // A second set of select scratch for the server's one row, a second stream and two events: in the folded
  // Top-K forms the workers' threshold select (needs only the worker pass) runs beside the parameter-sized
  // server pass and the server's own select (fork after the worker pass, join at the end of the step).
  u32 *hist_srv, *work_count_srv, *cand_n_srv;
  SelectState* sel_srv;
  int2* work_srv;
  cudaStream_t aux, aux2[2];            // aux2: for the second launch of a select (workers' [0], server's [1])
  cudaEvent_t ev_fork, ev_join, ev_fork2[2], ev_join2[2];
  long long cand_stride;
  u32* status;
  u32* status_host;      // pinned
  WaitCfg wc;            // how long device waits poll before they give up (and the test-only dropped copy)
  float* staging;        // sae_step_host
  float* out_stage;      // sae_get_params_host
  double* mismatch;      // sae_get_mismatch
  int64_t t;
  int esrc;              // how e^(k) is held now (ESRC_*)
  int fused_ok;          // p = 1, scaled sign, K a power of two <= 32: averaging is folded into the next worker pass
  float eta_prev;        // learning rate of the last step (needed while the average is pending)
  int last;              // which of scale[2]/tau[2] holds the last step's values
  int last_cuda_error;
  int persistent_blocks;  // #SMs x blocks per SM of the persistent worker pass
  int num_sms;
  int mu0;                 // momentum 0 and p != 1: no momentum rows (m^(k) is the step's gradient term, not state)
  int topk_nod;            // Top-K with p = 1: model differences never stored, two uniform-error buffers
  float* ebar_alt;
  int64_t launches;
  long long max_n;         // largest tensor
  // sharded operation: this handle owns workers k0 .. k0+P.K-1 of K_total; the server lines run on every shard
  int shard, k0, K_total;
  Plan P_all;                       // the plan with K = K_total (server pass, averaging)
  int attached;                     // workers whose message rows are known
  int mid_step;                     // sae_step_begin done, sae_step_end due
  int local_steps;                  // H: iteration t communicates iff (t+1) mod H == 0 (1: every iteration)
  // Top-K, p = 1, K = 8 or 16, no weight decay: the tail of a step (worker-axis aggregation, averaged error,
  // server lines) is left to the worker pass of the next step, which reads the same momentum rows anyway
  int fused_topk_ok;
  int tail_pending;                 // the last step stopped after its threshold select (scaled sign: after its scales)
  int reader;                       // the caller has been reading x / e between steps: a p = 1 scaled-sign step then
                                    // stops after its scales whatever K is, and the getter closes it in one pass
  int recs_srv_fresh;               // a server pass has added to the server's L1 records since they were last finalized
  float* ssum;                      // [dpad] ordered worker-axis sum of the selected entries (folded form)
  int avg_external;                 // the averaging sum is all-reduced by the caller instead of pulled in k order
  int avg_owed;                     // ... and is owed before the next sae_step_begin
  float lr_pending;
  std::vector<const u32*> h_word_rows;
  std::vector<const float*> h_scale_rows[2], h_d_rows;
  const u32** d_word_rows;
  const float** d_scale_rows[2];
  const float** d_d_rows;
  // sharded Top-K: the local workers' messages (lists of selected entries) and the tables over all workers
  unsigned long long* msg_entries;  // [K_loc][cand_stride]
  u32* msg_count;                   // [K_loc][T]
  float* agg_acc;                   // [dpad] scratch of the ordered sparse sum, zero between uses
  std::vector<const unsigned long long*> h_entry_rows;
  std::vector<const u32*> h_count_rows, h_tau_rows[2];
  const unsigned long long** d_entry_rows;
  const u32** d_count_rows;
  const u32** d_tau_rows[2];
  std::vector<void*> ipc_opened;    // mappings of other processes' buffers, closed by sae_destroy
  // cached step graphs
  int graphs_enabled, graph_misses, graph_pause;
  uint64_t graph_clock;
  std::vector<StepGraph> graphs;
  // profiling
  int profiling;
  std::vector<EventPair> pending;
  std::vector<cudaEvent_t> pool;
  double ms[SAE_NUM_KERNELS];
  int64_t cnt[SAE_NUM_KERNELS];
};

namespace {

struct DeviceGuard {
  int prev;
  bool ok;
  explicit DeviceGuard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    ok = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

#define SAE_CUDA(h, call)                                  \
  do {                                                     \
    cudaError_t e_ = (call);                               \
    if (e_ != cudaSuccess) {                               \
      (h)->last_cuda_error = (int)e_;                      \
      cudaGetLastError();                                  \
      return e_ == cudaErrorMemoryAllocation ? SAE_ERR_NOMEM : SAE_ERR_CUDA; \
    }                                                      \
  } while (0)

cudaEvent_t take_event(sae_handle* h) {
  if (!h->pool.empty()) { cudaEvent_t e = h->pool.back(); h->pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// One per kernel launch: counts it, brackets it with events while per-kernel timing is on, and opens an NVTX
// range named after the kernel's role ("worker_pass", "server_aggregate", ...) for timeline tools.
struct LaunchScope {
  sae_handle* h; int slot; cudaEvent_t a, b;
  LaunchScope(sae_handle* h_, int slot_) : h(h_), slot(slot_), a(nullptr), b(nullptr) {
    nvtxRangePushA(kSlotNames[slot]);
    if (h->profiling) { a = take_event(h); b = take_event(h); cudaEventRecord(a, h->stream); }
  }
  ~LaunchScope() {
    h->launches++;
    if (h->profiling) { cudaEventRecord(b, h->stream); h->pending.push_back({slot, a, b}); }
    nvtxRangePop();
  }
};

struct ApiRange {       // an NVTX range around a whole entry point
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
};

#define LAUNCH(h, slot, kern, grid, ...)                                   \
  do {                                                                     \
    LaunchScope ls_(h, slot);                                              \
    kern<<<(unsigned)(grid), THREADS, 0, (h)->stream>>>(__VA_ARGS__);      \
  } while (0)

// The dense server pass reads through a shared-memory ring above the 48 KB that need no opt-in.
#define LAUNCH_DENSE(h, kern, grid, ...)                                                                   \
  do {                                                                                                     \
    static thread_local int configured_device_ = -1;                                                       \
    if (configured_device_ != (h)->device) {                                                               \
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDenseSmem);            \
      configured_device_ = (h)->device;                                                                    \
    }                                                                                                      \
    LaunchScope ls_(h, S_SERVER);                                                                          \
    kern<<<(unsigned)(grid), THREADS, kDenseSmem, (h)->stream>>>(__VA_ARGS__);                             \
  } while (0)

// for functions without a status of their own: a failed call is picked up by the step's check_launch below
// (the runtime keeps the last error)
#define SAE_CUDA_VOID(h, call) do { (void)(h); (void)(call); } while (0)

int check_launch(sae_handle* h) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { h->last_cuda_error = (int)e; return SAE_ERR_CUDA; }
  return SAE_OK;
}

// SAE_DEBUG_FAIL_ALLOC=<n> (testing only, read by sae_init): the n-th device allocation of that sae_init
// (0-based) reports cudaErrorMemoryAllocation without calling cudaMalloc, so that the clean-up path of a failed
// initialisation can be exercised without exhausting a shared GPU's memory.
thread_local long g_fail_alloc_at = -1, g_alloc_index = 0;

template <class T>
cudaError_t dalloc(T** p, size_t count) {
  *p = nullptr;
  if (count == 0) count = 1;
  if (g_fail_alloc_at >= 0 && g_alloc_index++ == g_fail_alloc_at) return cudaErrorMemoryAllocation;
  return cudaMalloc((void**)p, count * sizeof(T));
}

void free_all(sae_handle* h) {
  void* ptrs[] = {h->d_tile_tensor, h->d_first_tile, h->d_n, h->d_off, h->d_poff, h->x, h->e_srv, h->ebar, h->ebar_alt, h->m, h->D,
                  h->words, h->words_srv, h->mask_srv, h->scale[0], h->scale[1], h->scale_srv, h->tau[0], h->tau[1],
                  h->tau_srv, h->recs, h->recs_alt, h->recs_srv, h->recs_srv_alt, h->recs_srv_alt2, h->recs_srv_alt3, h->hist, h->sel, h->status, h->staging, h->out_stage, h->mismatch,
                  h->cand_keys, h->cand_keys_srv, h->cand_count, h->cand_count_srv, h->fb, h->fb_srv, h->fb_total,
                  h->d_cand_off, h->d_cand_cap, h->d_wlog2, h->d_sel_list, h->work, h->work_count, h->cand_n, h->ssum};
  for (void* p : ptrs) if (p) cudaFree(p);
  void* srv_sel[] = {h->hist_srv, h->work_count_srv, h->cand_n_srv, h->sel_srv, h->work_srv};
  for (void* p : srv_sel) if (p) cudaFree(p);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  if (h->aux) cudaStreamDestroy(h->aux);
  for (int i = 0; i < 2; ++i) {
    if (h->ev_fork2[i]) cudaEventDestroy(h->ev_fork2[i]);
    if (h->ev_join2[i]) cudaEventDestroy(h->ev_join2[i]);
    if (h->aux2[i]) cudaStreamDestroy(h->aux2[i]);
  }
  void* tabs[] = {(void*)h->d_word_rows, (void*)h->d_scale_rows[0], (void*)h->d_scale_rows[1], (void*)h->d_d_rows,
                  (void*)h->d_entry_rows, (void*)h->d_count_rows, (void*)h->d_tau_rows[0], (void*)h->d_tau_rows[1],
                  (void*)h->msg_entries, (void*)h->msg_count, (void*)h->agg_acc};
  for (void* p : tabs) if (p) cudaFree(p);
  for (void* p : h->ipc_opened) cudaIpcCloseMemHandle(p);
  if (h->status_host) cudaFreeHost(h->status_host);
  for (auto& g : h->graphs) cudaGraphExecDestroy(g.exec);
  for (auto& ep : h->pending) { cudaEventDestroy(ep.a); cudaEventDestroy(ep.b); }
  for (auto e : h->pool) cudaEventDestroy(e);
}

// ---- Top-K threshold of every (row, tensor) of buf[rows][dpad] ---------------------------------------
// Candidate-window refine first; the three-level radix select then runs only where the window failed.
void topk_thresholds(sae_handle* h, const DeltaSrc& src, int rows, const CandArgs& cand, const u32* tau_guess,
                     u32* tau_out, u32* fb, u32* fb_total) {
  const Plan& P = h->P;
  const int pairs = rows * P.T;
  // the server's select has scratch of its own where a step may run it beside the workers' select
  const bool own = (fb == h->fb_srv) && h->hist_srv != nullptr;
  u32* hist = own ? h->hist_srv : h->hist;
  SelectState* sel = own ? h->sel_srv : h->sel;
  int2* work = own ? h->work_srv : h->work;
  u32* work_count = own ? h->work_count_srv : h->work_count;
  u32* cand_n = own ? h->cand_n_srv : h->cand_n;
  // One launch settles every pair whose candidate list holds the threshold, and small tensors whose window
  // failed; the server's single row is settled there entirely.  For the workers, large tensors whose window
  // failed (all of them at the first step) go through the distributed three-level select, whose launches
  // find an empty work list otherwise.
  // (A server row with a tensor of more than 2^20 elements keeps the distributed select as well: one block
  // would take too long over it.)
  const bool distributed = fb != h->fb_srv || h->max_n > (1ll << 20);
  const int inline_max = distributed ? SAE_TOPK_INLINE_MAX : 0x7fffffff;
  // Tensors with long candidate regions (the first n_sel_long of the list, longest first).  A single block
  // that walks a list of 10^5 keys is bound by its shared-memory atomics (60-120 us), the distributed select
  // spreads the same keys over the device but costs three levels of launches with real work in them.  What
  // pays, measured on config 3 (ms per step, p = 1 / p = 20; the select chains of the previous form 0.637 / 0.898):
  //   * the server's one row: its lists are short of their regions (its Delta is the mean of sparse messages);
  //     a block of 1024 threads per long list settles all of them in 12 us;
  //   * the workers with p = 1 (the lists stay short of their regions): blocks of 1024 threads, 0.599 / -- (the
  //     longest regions' chunks to the distributed select instead: 0.614);
  //   * the workers with stored differences (no averaging every step: the unsent entries pile up below the
  //     threshold and the lists are several times longer): every long list's chunks go to the distributed select,
  //     -- / 0.890 (blocks of 1024 threads: 0.927).
  // "Long" is a region of more than 65 536 keys (tensors above 0.8 M elements at 1 %): with the two launches side
  // by side the narrow blocks take the mid-sized lists at no cost to the critical path (16 384 as the limit:
  // 0.597 / 0.885; 65 536: 0.594 / 0.877; 131 072: 0.597 / 0.881).
  const bool server_row = fb == h->fb_srv;
  const bool long_inline = server_row || h->topk_nod || !distributed;
#ifndef SAE_SRV_LONG_REGION
#define SAE_SRV_LONG_REGION 16384
#endif
  // (the server's select sits at the end of the step's longest chain, behind the server pass: there the mid-sized
  // lists are worth wide blocks of their own -- 12 us beside 12 instead of 12 beside 24)
  const int n_long = long_inline ? (server_row ? h->n_sel_long_srv : h->n_sel_long) : 0;
  const int chunk_above = long_inline ? 0x7fffffff : SEL_LONG_REGION;
#ifndef SAE_SEL_TWO_STREAMS
#define SAE_SEL_TWO_STREAMS 1
#endif
  // The two launches take different lists: side by side where a second stream is at hand (the wide blocks leave
  // half of every SM's thread slots free, the narrow ones fill them) -- not while kernels are timed one by one.
  const int si = server_row ? 1 : 0;
  const bool two = SAE_SEL_TWO_STREAMS && n_long > 0 && P.T > n_long && h->aux2[si] != nullptr && !h->profiling;
  cudaStream_t short_stream = h->stream;
  if (two) {
    SAE_CUDA_VOID(h, cudaEventRecord(h->ev_fork2[si], h->stream));
    SAE_CUDA_VOID(h, cudaStreamWaitEvent(h->aux2[si], h->ev_fork2[si], 0));
    short_stream = h->aux2[si];
  }
  if (n_long > 0) {
    LaunchScope ls(h, S_TOPK_SELECT);
    k_topk_select_window<1024><<<(unsigned)(rows * n_long), 1024, 0, h->stream>>>(
        P, cand, h->d_sel_list, n_long, h->cfg.topk_num, h->cfg.topk_den, src, tau_guess, tau_out, fb, fb_total,
        inline_max, chunk_above, cand_n, work, work_count, rows);
  }
  if (P.T > n_long) {
    LaunchScope ls(h, S_TOPK_SELECT);
    k_topk_select_window<THREADS><<<(unsigned)(rows * (P.T - n_long)), THREADS, 0, short_stream>>>(
        P, cand, h->d_sel_list + n_long, P.T - n_long, h->cfg.topk_num, h->cfg.topk_den, src, tau_guess, tau_out, fb,
        fb_total, inline_max, chunk_above, cand_n, work, work_count, rows);
  }
  if (two) {
    SAE_CUDA_VOID(h, cudaEventRecord(h->ev_join2[si], h->aux2[si]));
    SAE_CUDA_VOID(h, cudaStreamWaitEvent(h->stream, h->ev_join2[si], 0));
  }
  if (!distributed) return;
  const long long hist_grid = 8LL * h->persistent_blocks;
  for (int level = 0; level < 3; ++level) {
    LAUNCH(h, S_TOPK_HIST, k_topk_hist, hist_grid, P, cand, rows, level, src, cand_n, sel, hist, work, work_count);
    LAUNCH(h, S_TOPK_SELECT, k_topk_select, pairs, P.T, level, h->d_n, h->cfg.topk_num, h->cfg.topk_den, hist, sel,
           tau_out, work_count, fb);
  }
}

DeltaSrc stored_rows(const float* buf) {
  DeltaSrc s; s.buf = buf; s.m = nullptr; s.ebar = nullptr; s.eta = 0.0f; s.recompute = 0;
  return s;
}

// The uniform local error as the next step will read it.  Top-K with p = 1 alternates between two buffers
// (the server pass reads the old one while writing the new one, and the getters of the last step's
// selection still need the old one); index `last` flips every step, like the scale and threshold buffers.
float* ebar_now(sae_handle* h) { return (h->topk_nod && h->last) ? h->ebar_alt : h->ebar; }
float* ebar_other(sae_handle* h) { return (h->topk_nod && !h->last) ? h->ebar_alt : h->ebar; }

CandArgs cand_args(sae_handle* h, bool server) {
  CandArgs c;
  c.keys = server ? h->cand_keys_srv : h->cand_keys;
  c.off = h->d_cand_off; c.cap = h->d_cand_cap; c.stride = h->cand_stride;
  c.count = server ? h->cand_count_srv : h->cand_count;
  c.T = h->P.T;
  c.wlog2 = h->d_wlog2;
  return c;
}

// The server lines a step left pending, carried out now (getters, checkpoints, steps that need x or e).
#ifndef SAE_LAZY_SERVER
#define SAE_LAZY_SERVER 1        // 0: every step runs its own apply kernel
#endif
// Top-K, folded form: carries out the tail the last step left to the next worker pass -- the dense server
// pass over the momentum rows (worker-axis aggregation, averaged error, any older pending server lines) and
// the server's threshold select -- the way a step that does not fold would have done it itself.  The step has
// already flipped `last`: its thresholds are tau[last], the uniform error it started from is ebar_other, the
// new one goes to ebar_now.  The server lines of that step are then pending like after any other step.
int flush_tail(sae_handle* h) {
  if (!h->tail_pending) return SAE_OK;
  const Plan& P = h->P;
  const bool dc = h->cfg.server_compress != 0;
  ServerArgs sa;
  memset(&sa, 0, sizeof(sa));
  sa.wc = h->wc;
  if (h->cfg.compressor == SAE_COMPRESSOR_SIGN) {
    // Scaled sign, p = 1: the open tail is the whole server pass of the last step, and the average of the local
    // errors is pending with it.  One pass over the K momentum rows does both: it re-forms every message
    // C(Delta^(k)) = +-s_k from Delta^(k) = fma(eta, m^(k), ebar) (the bits the worker pass packed), adds them
    // and the errors Delta^(k) - C(Delta^(k)) up in k order, and writes the server's Delta, its L1 partials and
    // sign words and the averaged error -- which thereby becomes the plain uniform error of the next step.
    if (h->esrc != ESRC_PENDING_AVG) return SAE_ERR_INVALID_ARG;
    const bool pending = h->srv_pending != 0;
    LAUNCH(h, S_FINALIZE, k_finalize_scales, (P.T + THREADS - 1) / THREADS, 0, P.T, h->d_n, h->recs, h->scale[h->last],
           h->recs_srv, (pending && dc && h->recs_srv_fresh) ? h->scale_srv : nullptr);
    sa.e_srv = h->e_srv; sa.scale_cur = h->scale[h->last]; sa.words_srv = h->words_srv; sa.recs_srv = h->recs_srv;
    sa.status = h->status; sa.x = h->x; sa.scale_srv_prev = h->scale_srv; sa.emit_srv = dc ? 1 : 0;
    sa.m = h->m; sa.ebar_in = h->ebar; sa.ebar = h->ebar; sa.eta = h->eta_prev;
    const int lsrv = pending ? (dc ? 3 : 1) : 0;
    if (lsrv == 0) LAUNCH_DENSE(h, (k_server_dense<1, true, true, 0>), P.ntiles, P, sa);
    else if (lsrv == 1) LAUNCH_DENSE(h, (k_server_dense<1, true, true, 1>), P.ntiles, P, sa);
    else LAUNCH_DENSE(h, (k_server_dense<1, true, true, 3>), P.ntiles, P, sa);
    h->recs_srv_fresh = 1;
    h->srv_pending = 1;
    h->tail_pending = 0;
    h->esrc = ESRC_UNIFORM;
    return check_launch(h);
  }
  sa.e_srv = h->e_srv; sa.tau_cur = h->tau[h->last]; sa.status = h->status;
  sa.cand_srv = cand_args(h, true); sa.tau_srv_prev = h->tau_srv; sa.emit_srv = dc ? 1 : 0;
  sa.m = h->m; sa.ebar_in = ebar_other(h); sa.ebar = ebar_now(h); sa.eta = h->eta_prev; sa.D = h->D;
  sa.x = h->x; sa.mask_srv = h->mask_srv;
  const int lsrv = h->srv_pending ? (dc ? 2 : 1) : 0;
  if (h->topk_nod) {
    if (lsrv == 0) LAUNCH_DENSE(h, (k_server_dense<2, true, true, 0>), P.ntiles, P, sa);
    else if (lsrv == 1) LAUNCH_DENSE(h, (k_server_dense<2, true, true, 1>), P.ntiles, P, sa);
    else LAUNCH_DENSE(h, (k_server_dense<2, true, true, 2>), P.ntiles, P, sa);
  } else {                                     // stored differences, a step whose pre-step does not average
    if (lsrv == 0) LAUNCH_DENSE(h, (k_server_dense<2, false, false, 0>), P.ntiles, P, sa);
    else if (lsrv == 1) LAUNCH_DENSE(h, (k_server_dense<2, false, false, 1>), P.ntiles, P, sa);
    else LAUNCH_DENSE(h, (k_server_dense<2, false, false, 2>), P.ntiles, P, sa);
  }
  if (dc) topk_thresholds(h, stored_rows(h->e_srv), 1, sa.cand_srv, h->tau_srv, h->tau_srv, h->fb_srv, h->fb_total + 1);
  h->srv_pending = 1;
  h->tail_pending = 0;
  return check_launch(h);
}

template <int COMP, int SRV>
void launch_apply_out(sae_handle* h, int out_kind, const ApplyArgs& aa) {
  if (out_kind == 0) LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_NONE>), h->P.ntiles, h->P, aa);
  else if (out_kind == 1) LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_NONE, 1>), h->P.ntiles, h->P, aa);
  else LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_NONE, 2>), h->P.ntiles, h->P, aa);
}

// out_kind 1 / 2: the apply kernel also writes the re-updated parameters / the step-ahead point x - ebar
// (uniform local errors) to `out`, caller layout, so that a getter needs no export pass of its own.
int flush_server(sae_handle* h, int out_kind = 0, float* out = nullptr) {
  { int rct = flush_tail(h); if (rct != SAE_OK) return rct; }
  if (!h->srv_pending) return SAE_OK;
  ApplyArgs aa;
  memset(&aa, 0, sizeof(aa));
  aa.out = out; aa.ebar_out = ebar_now(h);
  aa.e_srv = h->e_srv; aa.x = h->x; aa.ebar = h->ebar; aa.scale_srv = h->scale_srv; aa.recs_srv = h->recs_srv;
  if (h->inline_fin) {      // the last step accumulated into the buffer before the current rotation index
    L1Record* rs[4] = {h->recs_srv, h->recs_srv_alt, h->recs_srv_alt2, h->recs_srv_alt3};
    aa.recs_srv = rs[(h->rot + 3) % 4];
  }
  aa.tau_srv = h->tau_srv; aa.mask_srv = h->mask_srv;
  const bool dcs = h->cfg.server_compress != 0;
  if (h->cfg.compressor == SAE_COMPRESSOR_TOPK) {
    if (dcs) launch_apply_out<2, 2>(h, out_kind, aa); else launch_apply_out<2, 0>(h, out_kind, aa);
  } else if (dcs) launch_apply_out<1, 1>(h, out_kind, aa);
  else launch_apply_out<1, 0>(h, out_kind, aa);
  h->srv_pending = 0;
  return check_launch(h);
}

template <int ESRC, bool SIGN, bool WRITE_D, bool WD, bool TOPK, bool MU0 = false>
void launch_worker_wd(sae_handle* h, const StepParams& sp, const WorkerArgs& wa) {
  constexpr size_t kWorkerSmem = sizeof(WtSmemT<wt_stages(WRITE_D)>) + 128;
  static thread_local int configured_device = -1;     // opt in to > 48 KB of dynamic shared memory once
  if (configured_device != h->device) {
    cudaFuncSetAttribute(k_worker_tma<ESRC, SIGN, WRITE_D, WD, TOPK, MU0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)kWorkerSmem);
    configured_device = h->device;
  }
  const long long nitems = (long long)h->P.ntiles * h->P.K;
  // As many persistent blocks as the GPU holds, rounded down to a multiple of K when possible: block b
  // then always works for worker b mod K, which lets its warps carry L1 partials across items.
  long long grid = h->persistent_blocks;
  if (h->P.K <= grid) grid -= grid % h->P.K;
  if (nitems < grid) grid = nitems;
  LaunchScope ls(h, S_WORKER);
  k_worker_tma<ESRC, SIGN, WRITE_D, WD, TOPK, MU0><<<(unsigned)grid, WT_THREADS, kWorkerSmem, h->stream>>>(h->P, sp, wa, nitems);
}

template <int ESRC, bool SIGN, bool WRITE_D, bool TOPK = false>
void launch_worker(sae_handle* h, const StepParams& sp, const WorkerArgs& wa) {
  if constexpr (WRITE_D) {
    if (h->mu0) {          // no momentum rows (only steps that store the model differences run in this mode)
      if (sp.wd) launch_worker_wd<ESRC, SIGN, true, true, TOPK, true>(h, sp, wa);
      else launch_worker_wd<ESRC, SIGN, true, false, TOPK, true>(h, sp, wa);
      return;
    }
  }
  if (h->mu0) return;      // unreachable: the callers below keep WRITE_D set when there is no momentum buffer
  if (sp.wd) launch_worker_wd<ESRC, SIGN, WRITE_D, true, TOPK>(h, sp, wa);
  else launch_worker_wd<ESRC, SIGN, WRITE_D, false, TOPK>(h, sp, wa);
}

// The short-chain worker pass of small problems: a block per quarter tile, all workers.
template <int ESRC, bool WRITE_D>
void launch_small(sae_handle* h, const StepParams& sp, const WorkerArgs& wa, float eta_prev) {
  SmallArgs a;
  memset(&a, 0, sizeof(a));
  a.g = wa.g; a.m = wa.m; a.D = wa.D; a.ebar = const_cast<float*>(wa.ebar); a.x = wa.x; a.scale_prev = wa.scale_prev;
  a.words = wa.words; a.recs = wa.recs; a.status = wa.status; a.eta_prev = eta_prev;
  if (sp.wd && h->srv_pending) {
    // weight decay: the previous step's server lines are carried out by this pass before it reads x
    L1Record* rs[4] = {h->recs_srv, h->recs_srv_alt, h->recs_srv_alt2, h->recs_srv_alt3};
    a.lsrv = 1; a.dc = h->cfg.server_compress ? 1 : 0; a.e_srv = h->e_srv; a.x_rw = h->x;
    a.recs_srv_prev = rs[(h->rot + 3) % 4]; a.scale_srv = h->scale_srv;
    h->srv_pending = 0;
  }
  const size_t smem = (size_t)h->P.K * WS_ELEMS * sizeof(float);
  const long long grid = (long long)h->P.ntiles * WS_SUB;
  static thread_local int configured_device = -1;     // opt in to > 48 KB of dynamic shared memory once
  if (configured_device != h->device) {
    cudaFuncSetAttribute(k_worker_small<ESRC, WRITE_D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)(WS_MAXK * WS_ELEMS * sizeof(float)));
    cudaFuncSetAttribute(k_worker_small<ESRC, WRITE_D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         (int)(WS_MAXK * WS_ELEMS * sizeof(float)));
    configured_device = h->device;
  }
  LaunchScope ls(h, S_WORKER);
  if (sp.wd) k_worker_small<ESRC, WRITE_D, true><<<(unsigned)grid, THREADS, smem, h->stream>>>(h->P, sp, a);
  else k_worker_small<ESRC, WRITE_D, false><<<(unsigned)grid, THREADS, smem, h->stream>>>(h->P, sp, a);
}

template <int COMP, int SRV>
void launch_apply(sae_handle* h, int avg, const ApplyArgs& aa) {
  if (avg == AVG_NONE) LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_NONE>), h->P.ntiles, h->P, aa);
  else if (avg == AVG_FROM_D) LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_FROM_D>), h->P.ntiles, h->P, aa);
  else LAUNCH(h, S_APPLY, (k_apply<COMP, SRV, AVG_RECOMPUTE>), h->P.ntiles, h->P, aa);
}


// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time dependency on libcuda).
PFN_cuTensorMapEncodeTiled tensor_map_encoder() {
  static PFN_cuTensorMapEncodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (PFN_cuTensorMapEncodeTiled)p;
  }
  return fn;
}

// Row-major fp32 matrix [rows][inner] with the given row pitch, fetched in boxes of fw_box(rows) x fw_kh(rows).
bool make_row_map(CUtensorMap* map, const float* base, long long inner, int rows, long long pitch_elems) {
  PFN_cuTensorMapEncodeTiled enc = tensor_map_encoder();
  if (!enc || (reinterpret_cast<uintptr_t>(base) & 15) || ((pitch_elems * 4) & 15)) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 4};
  cuuint32_t box[2] = {(cuuint32_t)fw_box(rows), (cuuint32_t)fw_kh(rows)};
  cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int K, bool WD, int MODE = 0>
void launch_fused_kw(sae_handle* h, const StepParams& sp, const FusedArgs& fa, const CUtensorMap& tm_g) {
  constexpr size_t kFusedSmem = sizeof(FwSmemT<K, MODE>) + 128;
  static_assert(kFusedSmem <= 227 * 1024, "the ring must fit the shared memory of one block");
  static thread_local int configured_device = -1;
  if (configured_device != h->device) {
    cudaFuncSetAttribute(k_worker_fused<K, WD, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFusedSmem);
    configured_device = h->device;
  }
  typedef FwGeom<K, MODE> G;
  const long long nitems = (long long)h->P.ntiles * G::SUB;
  long long grid = h->persistent_blocks / SAE_WT_BLOCKS_PER_SM;      // one block per SM
  if (nitems < grid) grid = nitems;
  // Runs of one plan tile per block when the tensors are short (block-wise compression: a few tiles each) and
  // there is enough work to keep every block busy that way; long tensors stream best with the ranges dealt
  // out one by one (runs cost 4-5 % there).
  const bool short_tensors = h->P.ntiles < 4LL * h->P.T;
  int chunk_log2 = 0;
  if (short_tensors && nitems >= 8 * grid * G::SUB)
    while ((1 << chunk_log2) < G::SUB) ++chunk_log2;
  LaunchScope ls(h, S_WORKER);
  k_worker_fused<K, WD, MODE><<<(unsigned)grid, FW_THREADS, kFusedSmem, h->stream>>>(h->P, sp, fa, nitems, chunk_log2, h->tm_m, tm_g,
                                                                                      MODE == 2 ? h->tm_D : h->tm_m);
}

template <int K>
void launch_fused_k(sae_handle* h, const StepParams& sp, const FusedArgs& fa, const CUtensorMap& tm_g) {
  if (sp.wd) launch_fused_kw<K, true>(h, sp, fa, tm_g); else launch_fused_kw<K, false>(h, sp, fa, tm_g);
}

void launch_fused(sae_handle* h, const StepParams& sp, FusedArgs fa, int mode = 0) {
  // the gradients live in the caller's buffer: encode their tensor map for this step (host-only work)
  CUtensorMap tm_g;
  memset(&tm_g, 0, sizeof(tm_g));
  fa.g_tma_ok = make_row_map(&tm_g, fa.g, h->P.d, h->P.K, h->P.d) ? 1 : 0;
  if (mode == 1) {                     // (K = 8 or 16, no weight decay: checked by the caller)
    if (h->P.K == 8) launch_fused_kw<8, false, 1>(h, sp, fa, tm_g);
    else launch_fused_kw<16, false, 1>(h, sp, fa, tm_g);
    return;
  }
  if (mode == 2) {
    if (h->P.K == 8) launch_fused_kw<8, false, 2>(h, sp, fa, tm_g);
    else launch_fused_kw<16, false, 2>(h, sp, fa, tm_g);
    return;
  }
  fa.ebar_out = fa.ebar;
  switch (h->P.K) {
    case 1: launch_fused_k<1>(h, sp, fa, tm_g); break;
    case 2: launch_fused_k<2>(h, sp, fa, tm_g); break;
    case 4: launch_fused_k<4>(h, sp, fa, tm_g); break;
    case 8: launch_fused_k<8>(h, sp, fa, tm_g); break;
    case 16: launch_fused_k<16>(h, sp, fa, tm_g); break;
    default: launch_fused_k<32>(h, sp, fa, tm_g); break;
  }
}

// Does iteration t = h->t send the model differences?  (Every iteration unless local steps are set.)
bool communicates(const sae_handle* h) { return h->local_steps <= 1 || (h->t + 1) % h->local_steps == 0; }

int do_step_direct(sae_handle* h, const float* grads, float lr) {
  const sae_config& c = h->cfg;
  const Plan& P = h->P;
  const bool avg_after = c.avg_period > 0 && ((h->t + 2) % c.avg_period == 0);
  const int cur = 1 - h->last;
  const bool dc = c.server_compress != 0;
  StepParams sp;
  sp.mu = c.momentum; sp.eta = lr; sp.lambda = c.weight_decay;
  sp.saef = (c.mode == SAE_MODE_SAEF); sp.wd = (c.weight_decay != 0.0f);
  WorkerArgs wa;
  wa.wc = h->wc;
  wa.g = grads; wa.m = h->m; wa.D = h->D; wa.ebar = ebar_now(h); wa.x = h->x;
  wa.scale_prev = h->scale[h->last]; wa.tau_prev = h->tau[h->last];
  wa.words = h->words; wa.scale_cur = h->scale[cur]; wa.recs = h->recs; wa.status = h->status;
  wa.cand = cand_args(h, false);
  ServerArgs sa;
  memset(&sa, 0, sizeof(sa));
  sa.wc = h->wc;
  sa.e_srv = h->e_srv; sa.words = h->words; sa.scale_cur = h->scale[cur]; sa.D = h->D; sa.tau_cur = h->tau[cur];
  // inline_fin: rotating record buffers (see the handle)
  L1Record* rs3[4] = {h->recs_srv, h->recs_srv_alt, h->recs_srv_alt2, h->recs_srv_alt3};
  L1Record* const recs_now = (h->inline_fin && cur) ? h->recs_alt : h->recs;
  L1Record* const recs_other = (h->inline_fin && !cur) ? h->recs_alt : h->recs;
  L1Record* const recs_srv_now = h->inline_fin ? rs3[h->rot] : h->recs_srv;
  wa.recs = recs_now;
  sa.words_srv = h->words_srv; sa.scale_srv = h->scale_srv; sa.recs_srv = recs_srv_now; sa.status = h->status;
  sa.word_rows = nullptr; sa.scale_rows = nullptr; sa.recs = recs_now; sa.scale_out = h->scale[cur];
  sa.recs_clear = recs_other; sa.recs_srv_clear = rs3[(h->rot + 1) % 4]; sa.recs_srv_prev = rs3[(h->rot + 3) % 4];
  sa.cand_srv = cand_args(h, true); sa.tau_srv_prev = h->tau_srv; sa.emit_srv = dc ? 1 : 0; sa.ebar = ebar_now(h);
  sa.m = h->m; sa.ebar_in = ebar_now(h); sa.eta = lr;
  ApplyArgs aa;
  memset(&aa, 0, sizeof(aa));
  aa.e_srv = h->e_srv; aa.x = h->x; aa.ebar = ebar_now(h); aa.m = h->m; aa.D = h->D;
  aa.scale_cur = h->scale[cur]; aa.scale_srv = h->scale_srv; aa.recs_srv = recs_srv_now; aa.tau_cur = h->tau[cur];
  aa.tau_srv = h->tau_srv;
  aa.mask_srv = h->mask_srv; aa.eta = lr;

  if (!communicates(h)) {
    // Local iteration (Section 2: the model difference is communicated every H iterations): the worker lines
    // only.  The model difference keeps accumulating in D^(k), which from now on stands for e^(k) as it is.
    switch (h->esrc) {
      case ESRC_UNIFORM: launch_worker<ESRC_UNIFORM, false, true>(h, sp, wa); break;
      case ESRC_LAZY_SIGN: launch_worker<ESRC_LAZY_SIGN, false, true>(h, sp, wa); break;
      case ESRC_LAZY_TOPK: launch_worker<ESRC_LAZY_TOPK, false, true>(h, sp, wa); break;
      case ESRC_LOCAL_D: launch_worker<ESRC_LOCAL_D, false, true>(h, sp, wa); break;
      default: return SAE_ERR_INVALID_ARG;
    }
    h->esrc = ESRC_LOCAL_D;
    h->eta_prev = lr;
    h->t += 1;
    return check_launch(h);
  }
  if (c.compressor == SAE_COMPRESSOR_SIGN) {
    // an open tail that the next worker pass cannot take over (no sum vector, or this step does not fold): close it
    if (h->tail_pending && (h->ssum == nullptr || sp.wd)) { int rct = flush_tail(h); if (rct != SAE_OK) return rct; }
    // The model differences need not be stored when the previous error was uniform and the next
    // pre-step averages: the averaging pass recomputes them from m and ebar with the same fused op.
    const bool pending_in = h->esrc == ESRC_PENDING_AVG;
    const bool write_d = h->mu0 || !((h->esrc == ESRC_UNIFORM || pending_in) && avg_after);
    if (write_d && !h->D) return SAE_ERR_INVALID_ARG;
    // p = 1: the average is not formed here but at the head of the next worker pass
    // (the persistent folded pass takes power-of-two worker counts; the small-problem worker pass any)
    const bool defer_avg = avg_after && !write_d && (h->fused_ok || (h->small_worker && c.avg_period == 1));
    // The server lines of this step can be left to the next step's server pass when nothing in between
    // needs x or e: no weight decay (the worker pass reads x), no averaging in the apply kernel.
    // (small problems with weight decay: the lines wait as well, for the next worker pass, which carries them out)
    const bool lazy_ok = SAE_LAZY_SERVER && (!sp.wd || (h->small_worker && h->local_steps <= 1));
    // Folded form (p = 1 steady state, large problems): the whole server pass of this step stays open -- the
    // next step's worker pass re-forms every message C(Delta^(k)) in its averager warps anyway and adds them up
    // in k order on the way; a streaming server pass then only reads that sum.
    // (Worth the more the more workers: the unpacking server pass costs K additions per parameter, the streaming
    // one and the extra vector the worker pass writes do not depend on K -- config 4, 32 workers: 7.82 -> 7.62 ms
    // per step; config 2, 16 workers: 0.945 -> 0.939, the worker pass 0.821 -> 0.842 and the server pass
    // 0.122 -> 0.098; below 16 workers the unpacking pass is the cheaper one.)
    // The same open form, at any K, for a caller that reads the state between steps: the getter closes the step
    // in one pass over the momentum rows (flush_tail), which leaves the plain uniform error behind.
    const bool fold_sign = defer_avg && lazy_ok && !h->inline_fin && h->local_steps <= 1 &&
                           (h->ssum != nullptr || h->reader);
    if (h->tail_pending && !(pending_in && fold_sign && h->ssum != nullptr)) return SAE_ERR_INVALID_ARG;
    if (pending_in) {
      FusedArgs fa;
      memset(&fa, 0, sizeof(fa));
      fa.wc = h->wc;
      fa.g = grads; fa.m = h->m; fa.ebar = ebar_now(h); fa.x = h->x; fa.scale_prev = h->scale[h->last];
      fa.words = h->words; fa.recs = recs_now; fa.status = h->status; fa.eta_prev = h->eta_prev; fa.g_tma_ok = 0;
      fa.ssum = h->tail_pending ? h->ssum : nullptr;
      if (h->small_worker) launch_small<ESRC_PENDING_AVG, false>(h, sp, wa, h->eta_prev);
      else launch_fused(h, sp, fa);
    } else if (h->esrc == ESRC_UNIFORM) {
      if (h->small_worker) {
        if (write_d) launch_small<ESRC_UNIFORM, true>(h, sp, wa, 0.0f); else launch_small<ESRC_UNIFORM, false>(h, sp, wa, 0.0f);
      } else if (write_d) launch_worker<ESRC_UNIFORM, true, true>(h, sp, wa);
      else launch_worker<ESRC_UNIFORM, true, false>(h, sp, wa);
    } else if (h->esrc == ESRC_LOCAL_D) {
      launch_worker<ESRC_LOCAL_D, true, true>(h, sp, wa);
    } else if (h->small_worker) {
      launch_small<ESRC_LAZY_SIGN, true>(h, sp, wa, 0.0f);
    } else {
      launch_worker<ESRC_LAZY_SIGN, true, true>(h, sp, wa);
    }
    if (h->srv_pending && !lazy_ok) { int rcf = flush_server(h); if (rcf != SAE_OK) return rcf; }
    const bool pending = h->srv_pending != 0;
    if (!h->inline_fin) {
      LAUNCH(h, S_FINALIZE, k_finalize_scales, (P.K * P.T + P.T + THREADS - 1) / THREADS, P.K, P.T, h->d_n, h->recs,
             h->scale[cur], h->recs_srv, (pending && dc && h->recs_srv_fresh) ? h->scale_srv : nullptr);
      h->recs_srv_fresh = 0;
    }
    sa.x = h->x; sa.scale_srv_prev = h->scale_srv;
    // consecutive tiles per block: enough blocks to fill the device several times over, at most 8 tiles each
    const int tpb = std::max(1, std::min(8, P.ntiles / (h->num_sms * 16)));
    const int nblk = (P.ntiles + tpb - 1) / tpb;
    if (h->tail_pending) {                        // the previous step's server pass, from the sum
      sa.ssum = h->ssum;
      if (pending) {
        if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, false, false, true, true>), nblk, P, sa, tpb);
        else LAUNCH(h, S_SERVER, (k_server_sign<false, false, false, true, true>), nblk, P, sa, tpb);
      } else if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, false, false, false, true>), nblk, P, sa, tpb);
      else LAUNCH(h, S_SERVER, (k_server_sign<false, false, false, false, true>), nblk, P, sa, tpb);
      h->recs_srv_fresh = 1;
      h->srv_pending = 1;                         // its server lines wait for the next server pass
      h->tail_pending = 0;
    }
    if (fold_sign) {                              // this step's own server pass stays open
      h->tail_pending = 1;
      h->esrc = ESRC_PENDING_AVG;
      h->last = cur; h->eta_prev = lr; h->t += 1;
      return check_launch(h);
    }
    h->recs_srv_fresh = 1;                        // (the server pass below adds to the records)
    if (h->inline_fin) {
      if (pending) {
        if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, false, true, true>), nblk, P, sa, tpb);
        else LAUNCH(h, S_SERVER, (k_server_sign<false, false, true, true>), nblk, P, sa, tpb);
      } else if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, false, true>), nblk, P, sa, tpb);
      else LAUNCH(h, S_SERVER, (k_server_sign<false, false, true>), nblk, P, sa, tpb);
      h->rot = (h->rot + 1) % 4;
    } else if (pending) {
      if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, false, false, true>), nblk, P, sa, tpb);
      else LAUNCH(h, S_SERVER, (k_server_sign<false, false, false, true>), nblk, P, sa, tpb);
    } else if (dc) LAUNCH(h, S_SERVER, k_server_sign<true>, nblk, P, sa, tpb);
    else LAUNCH(h, S_SERVER, k_server_sign<false>, nblk, P, sa, tpb);
    const int avg = (avg_after && !defer_avg) ? (write_d ? AVG_FROM_D : AVG_RECOMPUTE) : AVG_NONE;
    if (lazy_ok && avg == AVG_NONE) {
      h->srv_pending = 1;                       // this step's server lines wait for the next server pass
    } else {
      h->srv_pending = 0;
      if (dc) launch_apply<1, 1>(h, avg, aa); else launch_apply<1, 0>(h, avg, aa);
    }
    h->esrc = defer_avg ? ESRC_PENDING_AVG : (avg_after ? ESRC_UNIFORM : ESRC_LAZY_SIGN);
  } else if (c.compressor == SAE_COMPRESSOR_TOPK) {
    // p = 1 (previous error uniform, pre-step averages, every step): the model differences are not stored;
    // whoever needs them after the worker pass recomputes them from m and the old uniform error
    const bool nod = h->topk_nod;
    if (nod && !(h->esrc == ESRC_UNIFORM && avg_after)) return SAE_ERR_INVALID_ARG;
    if (!nod && !h->D) return SAE_ERR_INVALID_ARG;
    // the server lines wait for the next dense server pass unless the worker pass needs x (weight decay)
    const bool lazy_ok = SAE_LAZY_SERVER && !sp.wd;
    if (h->srv_pending && !lazy_ok) { int rcf = flush_server(h); if (rcf != SAE_OK) return rcf; }
    int lsrv = h->srv_pending ? (dc ? 2 : 1) : 0;
    sa.x = h->x; sa.mask_srv = h->mask_srv;
    DeltaSrc src = stored_rows(h->D);
    if (nod) { src.m = h->m; src.ebar = ebar_now(h); src.eta = lr; src.recompute = 1; }
    // Folded form: this step stops after its threshold select; the rest (aggregation, averaged error, server
    // lines) is done by the next step's worker pass and a parameter-sized server pass behind it.
    // With stored differences (p != 1) the same holds for the steps whose pre-step does not average: the next
    // worker pass reads the stored rows anyway (it forms e^(k) = D - C(D) from them).
    const bool fold = lazy_ok && h->local_steps <= 1 &&
                      (nod ? h->fused_topk_ok != 0 : (h->fused_gen_ok && !avg_after));
    bool worker_done = false;
    if (h->tail_pending) {
      if (!lazy_ok || (!nod && h->esrc != ESRC_LAZY_TOPK)) return SAE_ERR_INVALID_ARG;
      FusedArgs fa;
      memset(&fa, 0, sizeof(fa));
      fa.wc = h->wc;
      fa.g = grads; fa.m = h->m; fa.ebar = ebar_other(h); fa.ebar_out = ebar_now(h); fa.x = h->x; fa.D = h->D;
      fa.tau_prev = h->tau[h->last]; fa.ssum = h->ssum; fa.cand = wa.cand; fa.status = h->status;
      fa.eta_prev = h->eta_prev;
      launch_fused(h, sp, fa, nod ? 1 : 2);
      // The workers' select needs only the worker pass; the server pass and the server's select need only the
      // sum it wrote.  Two chains of small dependent launches: run them side by side (not while kernels are
      // being timed one by one).
      const bool side = h->aux != nullptr && !h->profiling;
      if (side) {
        cudaStream_t main_stream = h->stream;
        SAE_CUDA(h, cudaEventRecord(h->ev_fork, main_stream));
        SAE_CUDA(h, cudaStreamWaitEvent(h->aux, h->ev_fork, 0));
        h->stream = h->aux;
        topk_thresholds(h, src, P.K, wa.cand, h->tau[h->last], h->tau[cur], h->fb, h->fb_total);
        h->stream = main_stream;
        SAE_CUDA(h, cudaEventRecord(h->ev_join, h->aux));
      } else {
        topk_thresholds(h, src, P.K, wa.cand, h->tau[h->last], h->tau[cur], h->fb, h->fb_total);
      }
      sa.ssum = h->ssum;
      if (lsrv == 0) LAUNCH_DENSE(h, (k_server_dense<2, false, false, 0, true>), P.ntiles, P, sa);
      else if (lsrv == 1) LAUNCH_DENSE(h, (k_server_dense<2, false, false, 1, true>), P.ntiles, P, sa);
      else LAUNCH_DENSE(h, (k_server_dense<2, false, false, 2, true>), P.ntiles, P, sa);
      if (dc) topk_thresholds(h, stored_rows(h->e_srv), 1, sa.cand_srv, h->tau_srv, h->tau_srv, h->fb_srv, h->fb_total + 1);
      if (side) SAE_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_join, 0));
      h->srv_pending = 1;                    // the previous step's server lines now wait for the next server pass
      h->tail_pending = 0;
      lsrv = dc ? 2 : 1;
      worker_done = true;
    }
    if (!worker_done) {
      if (nod) launch_worker<ESRC_UNIFORM, false, false, true>(h, sp, wa);
      else if (h->esrc == ESRC_UNIFORM) launch_worker<ESRC_UNIFORM, false, true, true>(h, sp, wa);
      else if (h->esrc == ESRC_LOCAL_D) launch_worker<ESRC_LOCAL_D, false, true, true>(h, sp, wa);
      else launch_worker<ESRC_LAZY_TOPK, false, true, true>(h, sp, wa);
      topk_thresholds(h, src, P.K, wa.cand, h->tau[h->last], h->tau[cur], h->fb, h->fb_total);
    }
    if (fold) {                              // this step's own tail stays open for the next worker pass
      h->tail_pending = 1;
      h->esrc = avg_after ? ESRC_UNIFORM : ESRC_LAZY_TOPK;
      h->last = cur; h->eta_prev = lr; h->t += 1;
      return check_launch(h);
    }
    // the averaged error (if the pre-step averages) comes out of the same pass over D as the server's sum
    if (nod) sa.ebar = ebar_other(h);          // becomes the current one when `last` flips below
#define SAE_DENSE(AVGF, RECF)                                                                              \
    do {                                                                                                   \
      if (lsrv == 0) LAUNCH_DENSE(h, (k_server_dense<2, AVGF, RECF, 0>), P.ntiles, P, sa);                 \
      else if (lsrv == 1) LAUNCH_DENSE(h, (k_server_dense<2, AVGF, RECF, 1>), P.ntiles, P, sa);            \
      else LAUNCH_DENSE(h, (k_server_dense<2, AVGF, RECF, 2>), P.ntiles, P, sa);                           \
    } while (0)
    if (nod) SAE_DENSE(true, true);
    else if (avg_after) SAE_DENSE(true, false);
    else SAE_DENSE(false, false);
#undef SAE_DENSE
    if (dc) topk_thresholds(h, stored_rows(h->e_srv), 1, sa.cand_srv, h->tau_srv, h->tau_srv, h->fb_srv, h->fb_total + 1);
    if (lazy_ok) {
      h->srv_pending = 1;
    } else {
      h->srv_pending = 0;
      if (dc) launch_apply<2, 2>(h, AVG_NONE, aa); else launch_apply<2, 0>(h, AVG_NONE, aa);
    }
    h->esrc = avg_after ? ESRC_UNIFORM : ESRC_LAZY_TOPK;
  } else {
    // identity: every error stays exactly zero, so e^(k) is the (all-zero) uniform vector forever
    if (h->esrc == ESRC_LOCAL_D) launch_worker<ESRC_LOCAL_D, false, true>(h, sp, wa);
    else launch_worker<ESRC_UNIFORM, false, true>(h, sp, wa);
    LAUNCH_DENSE(h, (k_server_dense<0, false>), P.ntiles, P, sa);
    launch_apply<0, 0>(h, AVG_NONE, aa);
    h->esrc = ESRC_UNIFORM;
  }
  h->last = cur;
  h->eta_prev = lr;
  h->t += 1;
  return check_launch(h);
}

// One step through a cached CUDA graph.  The launch sequence of a step depends only on the handle's
// small state (how the error is held, which scale buffer is current, whether the pre-step averages),
// the gradient pointer and the learning rate; a step with a key seen before is replayed with a single
// cudaGraphLaunch, which takes the per-kernel launch cost off the host (small workloads are bound by it).
int do_step(sae_handle* h, const float* grads, float lr) {
  if (h->esrc == ESRC_PENDING_AVG) h->reader = 0;       // nobody looked at the state since the last step
  bool usable = h->graphs_enabled && !h->profiling && h->stream != nullptr && h->stream != cudaStreamLegacy &&
                h->stream != cudaStreamPerThread;
  if (usable) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(h->stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
      cudaGetLastError();
      usable = false;          // the caller is capturing this stream: our launches simply join that capture
    }
  }
  if (!usable) return do_step_direct(h, grads, lr);

  StepGraphKey key;
  key.esrc = h->esrc; key.last = h->last; key.srv_pending = h->srv_pending; key.rot = h->rot;
  key.comm = communicates(h) ? 1 : 0; key.tail = h->tail_pending; key.fresh = h->recs_srv_fresh; key.reader = h->reader;
  key.avg_after = (h->cfg.avg_period > 0 && ((h->t + 2) % h->cfg.avg_period == 0)) ? 1 : 0;
  key.grads = grads; key.lr = lr; key.eta_prev = h->eta_prev;     // every value a captured kernel argument depends on
  for (size_t q = 0; q < h->graphs.size(); ++q) {
    StepGraph& e = h->graphs[q];
    if (e.key.esrc == key.esrc && e.key.last == key.last && e.key.avg_after == key.avg_after &&
        e.key.srv_pending == key.srv_pending && e.key.rot == key.rot && e.key.comm == key.comm && e.key.tail == key.tail && e.key.fresh == key.fresh && e.key.reader == key.reader && e.key.grads == key.grads && e.key.lr == key.lr && e.key.eta_prev == key.eta_prev) {
      SAE_CUDA(h, cudaGraphLaunch(e.exec, h->stream));
      h->launches += e.kernels;
      h->esrc = e.esrc_after; h->last = e.last_after; h->srv_pending = e.pending_after; h->rot = e.rot_after;
      h->tail_pending = e.tail_after; h->recs_srv_fresh = e.fresh_after;
      h->eta_prev = lr; h->t += 1;
      e.stamp = ++h->graph_clock;
      h->graph_misses = 0;
      return SAE_OK;
    }
  }
  // Not seen before.  Capturing costs far more than a direct step, so a key is only captured when it can come
  // back: the learning rate must have held still for a step (lr == the previous step's).  A schedule that
  // changes lr every step (warm-up, cosine) therefore runs direct steps without paying for captures, and
  // graphs come back by themselves once lr settles.  A run of captures that never hit pauses capturing for a
  // while instead of switching it off for good.
  const bool lr_settled = h->t == 0 || lr == h->eta_prev;
  if (h->graph_pause > 0) { --h->graph_pause; return do_step_direct(h, grads, lr); }
  if (!lr_settled) return do_step_direct(h, grads, lr);
  if (++h->graph_misses > 64) { h->graph_misses = 0; h->graph_pause = 256; return do_step_direct(h, grads, lr); }
  // The capture below runs the host side of the step (which advances the handle's small state) without any
  // device work; if it fails, that state is put back and the step runs directly, so host and device agree.
  struct HostState { int64_t t, launches; int esrc, last, rot, srv_pending, tail_pending, recs_srv_fresh; float eta_prev; };
  const HostState before = {h->t, h->launches, h->esrc, h->last, h->rot, h->srv_pending, h->tail_pending,
                            h->recs_srv_fresh, h->eta_prev};
  auto restore = [&]() {
    h->t = before.t; h->launches = before.launches; h->esrc = before.esrc; h->last = before.last; h->rot = before.rot;
    h->srv_pending = before.srv_pending; h->tail_pending = before.tail_pending;
    h->recs_srv_fresh = before.recs_srv_fresh; h->eta_prev = before.eta_prev;
  };
  auto fall_back = [&](cudaError_t ce) {
    h->last_cuda_error = (int)ce; cudaGetLastError();
    restore();
    h->graph_pause = 256;
    return do_step_direct(h, grads, lr);
  };
  const int64_t launches0 = h->launches;
  {
    const cudaError_t cb = cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal);
    if (cb != cudaSuccess) return fall_back(cb);
  }
  int rc = do_step_direct(h, grads, lr);
  cudaGraph_t graph = nullptr;
  cudaError_t ce = cudaStreamEndCapture(h->stream, &graph);
  if (rc != SAE_OK || ce != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    if (rc != SAE_OK) {                             // the step itself was refused; nothing ran on the device
      if (ce != cudaSuccess) cudaGetLastError();
      restore();
      return rc;
    }
    return fall_back(ce != cudaSuccess ? ce : cudaErrorUnknown);
  }
  StepGraph e;
  e.key = key; e.exec = nullptr; e.kernels = (int)(h->launches - launches0);
  e.esrc_after = h->esrc; e.last_after = h->last; e.pending_after = h->srv_pending; e.rot_after = h->rot;
  e.tail_after = h->tail_pending; e.fresh_after = h->recs_srv_fresh;
  e.stamp = ++h->graph_clock;
  ce = cudaGraphInstantiate(&e.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ce != cudaSuccess) return fall_back(ce);
  ce = cudaGraphLaunch(e.exec, h->stream);
  if (ce != cudaSuccess) { cudaGraphExecDestroy(e.exec); return fall_back(ce); }
  if (h->graphs.size() >= 128) {               // evict the least recently used graph
    size_t victim = 0;
    for (size_t q = 1; q < h->graphs.size(); ++q) if (h->graphs[q].stamp < h->graphs[victim].stamp) victim = q;
    cudaGraphExecDestroy(h->graphs[victim].exec);
    h->graphs[victim] = e;
  } else {
    h->graphs.push_back(e);
  }
  return SAE_OK;
}

// The pending average of a p = 1 scaled-sign step whose server pass is already done, formed in place: the
// averaged error becomes the plain uniform error (what the next worker pass would have formed, same bits).
int close_pending_avg(sae_handle* h) {
  if (h->esrc != ESRC_PENDING_AVG) return SAE_OK;
  { int rct = flush_tail(h); if (rct != SAE_OK) return rct; }          // (an open tail closes the average with it)
  if (h->esrc != ESRC_PENDING_AVG) return SAE_OK;
  LAUNCH(h, S_EXPORT, k_materialize_avg, h->P.ntiles, h->P, h->m, h->ebar, h->scale[h->last], h->eta_prev, h->ebar);
  h->esrc = ESRC_UNIFORM;
  return check_launch(h);
}

ExportArgs export_args(sae_handle* h, int what, int k) {
  ExportArgs ea;
  ea.x = h->x; ea.e_srv = h->e_srv; ea.m = h->m; ea.D = h->D; ea.ebar = ebar_now(h);
  ea.scale_last = h->scale[h->last]; ea.tau_last = h->tau[h->last];
  ea.esrc = h->esrc; ea.what = what; ea.k = k; ea.saef = (h->cfg.mode == SAE_MODE_SAEF);
  return ea;
}

int export_vec(sae_handle* h, int what, int k, float* out) {
  if (what == EXP_M) {
    int rct = flush_tail(h);
    if (rct != SAE_OK) return rct;
  } else {
    h->reader = 1;                                       // x and e must be up to date, and will be asked for again
    const bool saef = h->cfg.mode == SAE_MODE_SAEF;
    const bool need_error = what == EXP_WERR || (what == EXP_STEP_AHEAD && saef);
    if (need_error) { int rca = close_pending_avg(h); if (rca != SAE_OK) return rca; }
    { int rct = flush_tail(h); if (rct != SAE_OK) return rct; }
    // the pending server lines and the answer in one pass where the answer is x, or x minus a uniform error
    int out_kind = 0;
    if (what == EXP_X || (what == EXP_STEP_AHEAD && !saef)) out_kind = 1;
    else if (what == EXP_STEP_AHEAD && h->esrc == ESRC_UNIFORM) out_kind = 2;
    if (h->srv_pending && out_kind != 0) return flush_server(h, out_kind, out);
    int rcf = flush_server(h);
    if (rcf != SAE_OK) return rcf;
  }
  const ExportArgs ea = export_args(h, what, k);
  LAUNCH(h, S_EXPORT, k_export, h->P.ntiles, h->P, ea, out);
  return check_launch(h);
}

// ---- checkpoint: every buffer a later step or getter depends on, in a fixed order ----
struct CkptHeader {
  uint64_t magic;
  int32_t K, T, compressor, server_compress, mode, avg_period;
  uint32_t topk_num, topk_den;
  float momentum, weight_decay;
  int64_t d, t;
  int32_t esrc, last;
  float eta_prev;
  int32_t worker_begin, num_workers_total;     // which workers of how many this handle owns (sharded operation)
  int32_t local_steps;                         // 0 in checkpoints written before local steps existed (= 1)
};
constexpr uint64_t kCkptMagic = 0x5341455F434B5032ull;   // "SAE_CKP2"

struct CkptSection { void* ptr; size_t bytes; };

std::vector<CkptSection> ckpt_sections(sae_handle* h) {
  const Plan& P = h->P;
  const size_t KT = (size_t)P.K * P.T, f = sizeof(float);
  const bool sign = h->cfg.compressor == SAE_COMPRESSOR_SIGN, topk = h->cfg.compressor == SAE_COMPRESSOR_TOPK;
  std::vector<CkptSection> v;
  v.push_back({h->x, (size_t)P.dpad * f}); v.push_back({h->e_srv, (size_t)P.dpad * f});
  v.push_back({h->ebar, (size_t)P.dpad * f});
  if (h->m) v.push_back({h->m, (size_t)P.K * P.dpad * f});
  if (h->D) v.push_back({h->D, (size_t)P.K * P.dpad * f});
  if (h->ebar_alt) v.push_back({h->ebar_alt, (size_t)P.dpad * f});
  if (sign) { v.push_back({h->words, (size_t)P.K * P.nwords * 4}); v.push_back({h->words_srv, (size_t)P.nwords * 4}); }
  if (topk) v.push_back({h->mask_srv, (size_t)P.nwords * 4});
  v.push_back({h->scale[0], KT * f}); v.push_back({h->scale[1], KT * f}); v.push_back({h->scale_srv, (size_t)P.T * f});
  v.push_back({h->tau[0], KT * 4}); v.push_back({h->tau[1], KT * 4}); v.push_back({h->tau_srv, (size_t)P.T * 4});
  return v;
}

size_t ckpt_bytes(sae_handle* h) {
  size_t total = 256;                       // header, padded
  for (const auto& s : ckpt_sections(h)) total += (s.bytes + 255) / 256 * 256;
  return total;
}

}  // namespace

extern "C" {

}  // extern "C"

namespace {

// sae_init and sae_init_shard: worker rows k0 .. k0+K_loc-1 of cfg->num_workers are held here
int init_impl(const sae_config* cfg, int k0, int K_loc, bool shard, const float* x0, sae_handle** out) {
  if (out) *out = nullptr;
  if (!cfg || !x0 || !out) return SAE_ERR_INVALID_ARG;
  if (cfg->abi_version != SAE_ABI_VERSION) return SAE_ERR_ABI;
  if (cfg->num_workers < 1 || cfg->num_workers > MAX_WORKERS || cfg->num_tensors < 1 || !cfg->tensor_sizes)
    return SAE_ERR_INVALID_ARG;
  if (cfg->compressor < 0 || cfg->compressor > 2 || (cfg->mode != 0 && cfg->mode != 1) ||
      (cfg->server_compress != 0 && cfg->server_compress != 1) || cfg->avg_period < 0)
    return SAE_ERR_INVALID_ARG;
  if (!(cfg->momentum >= 0.0f && cfg->momentum < 1.0f) || !(cfg->weight_decay >= 0.0f)) return SAE_ERR_INVALID_ARG;
  if (cfg->compressor == SAE_COMPRESSOR_TOPK && (cfg->topk_den == 0 || cfg->topk_num > cfg->topk_den))
    return SAE_ERR_INVALID_ARG;
  if (cfg->device < 0) return SAE_ERR_INVALID_ARG;
  if (k0 < 0 || K_loc < 1 || k0 + K_loc > cfg->num_workers) return SAE_ERR_INVALID_ARG;
  if (shard && cfg->compressor == SAE_COMPRESSOR_IDENTITY) return SAE_ERR_INVALID_ARG;
  const int T = cfg->num_tensors, K = K_loc;          // K: worker rows held by this handle
  long long d = 0, dpad = 0, ntiles = 0;
  for (int j = 0; j < T; ++j) {
    const int64_t n = cfg->tensor_sizes[j];
    if (n <= 0 || n > (1ll << 30)) return SAE_ERR_INVALID_ARG;
    d += n; dpad += (n + 31) / 32 * 32; ntiles += (n + TILE - 1) / TILE;
  }
  if (ntiles * K >= (1ll << 31) || ntiles >= (1ll << 31)) return SAE_ERR_INVALID_ARG;

  DeviceGuard guard(cfg->device);
  if (!guard.ok) { g_init_cuda_error = (int)cudaGetLastError(); return SAE_ERR_CUDA; }
  g_fail_alloc_at = -1; g_alloc_index = 0;
  if (const char* ev = getenv("SAE_DEBUG_FAIL_ALLOC")) { const long v = atol(ev); if (v >= 0) g_fail_alloc_at = v; }
  struct FailAllocOff { ~FailAllocOff() { g_fail_alloc_at = -1; } } fail_alloc_off;   // only this sae_init

  sae_handle* h = new (std::nothrow) sae_handle();
  if (!h) return SAE_ERR_NOMEM;
  h->cfg = *cfg;
  h->sizes.assign(cfg->tensor_sizes, cfg->tensor_sizes + T);
  h->cfg.tensor_sizes = h->sizes.data();
  h->max_n = 0;
  for (int j = 0; j < T; ++j) h->max_n = std::max<long long>(h->max_n, h->sizes[j]);
  h->device = cfg->device;
  h->stream = (cudaStream_t)cfg->stream;
  h->t = 0; h->esrc = ESRC_UNIFORM; h->last = 0; h->eta_prev = 0.0f; h->local_steps = 1;
  // Device waits give up after SAE_WAIT_LIMIT_US microseconds of polling (default: one second).
  // SAE_DEBUG_DROP_COPY=<item> (testing only) makes the producer of the worker / server passes announce the
  // copies of that work item without issuing them, so that the waits on it run out and SAE_ERR_TIMEOUT is raised.
  h->wc.limit_us = 0; h->wc.drop_item = 0;
  if (const char* ev = getenv("SAE_WAIT_LIMIT_US")) { const long v = atol(ev); if (v > 0 && v <= 60000000L) h->wc.limit_us = (u32)v; }
  if (const char* ev = getenv("SAE_DEBUG_DROP_COPY")) { const long v = atol(ev); if (v >= 0 && v < (1L << 31) - 1) h->wc.drop_item = (u32)v + 1u; }
  h->graphs_enabled = 1; h->graph_misses = 0; h->graph_pause = 0; h->graph_clock = 0;
  h->fused_ok = (!shard && cfg->compressor == SAE_COMPRESSOR_SIGN && cfg->avg_period == 1 && cfg->num_workers <= 32 &&
                 (cfg->num_workers & (cfg->num_workers - 1)) == 0) ? 1 : 0; h->last_cuda_error = 0; h->launches = 0; h->profiling = 0;
  h->shard = shard ? 1 : 0; h->k0 = k0; h->K_total = cfg->num_workers; h->attached = 0; h->mid_step = 0;
  for (int i = 0; i < SAE_NUM_KERNELS; ++i) { h->ms[i] = 0; h->cnt[i] = 0; }
  {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess || sms < 1) sms = 148;
    h->persistent_blocks = sms * SAE_WT_BLOCKS_PER_SM;
    h->num_sms = sms;
  }

  std::vector<int> tile_tensor((size_t)ntiles), first_tile(T), n32(T);
  std::vector<long long> off(T), poff(T);
  {
    long long o = 0, po = 0; int tl = 0;
    for (int j = 0; j < T; ++j) {
      const long long n = h->sizes[j];
      off[j] = o; poff[j] = po; first_tile[j] = tl; n32[j] = (int)n;
      const int tj = (int)((n + TILE - 1) / TILE);
      for (int q = 0; q < tj; ++q) tile_tensor[tl + q] = j;
      tl += tj; o += n; po += (n + 31) / 32 * 32;
    }
  }
  const bool sign = cfg->compressor == SAE_COMPRESSOR_SIGN, topk = cfg->compressor == SAE_COMPRESSOR_TOPK;
  h->topk_nod = (!shard && topk && cfg->avg_period == 1) ? 1 : 0;      // (a shard always stores its differences)
  h->mu0 = (cfg->momentum == 0.0f && cfg->avg_period != 1) ? 1 : 0;
  const bool need_D = shard || !((sign || topk) && cfg->avg_period == 1);
  const long long nwords = dpad / 32;
  const size_t KT = (size_t)K * T;

  int rc = SAE_OK;
  auto fail = [&](cudaError_t e) {
    h->last_cuda_error = (int)e; g_init_cuda_error = (int)e; cudaGetLastError();
    rc = (e == cudaErrorMemoryAllocation) ? SAE_ERR_NOMEM : SAE_ERR_CUDA;
  };
#define TRY(call) do { if (rc == SAE_OK) { cudaError_t e_ = (call); if (e_ != cudaSuccess) fail(e_); } } while (0)
#define ALLOC0(ptr, count) do { TRY(dalloc(&(ptr), (count))); \
    if (rc == SAE_OK) TRY(cudaMemsetAsync((ptr), 0, (size_t)((count) ? (count) : 1) * sizeof(*(ptr)), h->stream)); } while (0)
  ALLOC0(h->d_tile_tensor, (size_t)ntiles); ALLOC0(h->d_first_tile, T); ALLOC0(h->d_n, T);
  ALLOC0(h->d_off, T); ALLOC0(h->d_poff, T);
  ALLOC0(h->x, dpad); ALLOC0(h->e_srv, dpad); ALLOC0(h->ebar, dpad);
  if (!h->mu0) ALLOC0(h->m, (size_t)K * dpad);
  if (need_D) ALLOC0(h->D, (size_t)K * dpad);
  if (h->topk_nod) ALLOC0(h->ebar_alt, dpad);
  h->fused_topk_ok = (h->topk_nod && (K == 8 || K == 16) && dpad < (1ll << 31) && d < (1ll << 31)) ? 1 : 0;
  h->tail_pending = 0; h->recs_srv_fresh = 0; h->reader = 0;
  h->fused_gen_ok = (!shard && topk && cfg->avg_period != 1 && (K == 8 || K == 16) && dpad < (1ll << 31) &&
                     d < (1ll << 31)) ? 1 : 0;
  // (scaled sign: the folded server pass is for large problems, p = 1, K a power of two up to 32)
  const bool sign_fold = h->fused_ok && K >= SAE_SIGN_FOLD_MIN_K && (long long)K * dpad > (1ll << 24);
  if (h->fused_topk_ok || h->fused_gen_ok || sign_fold) ALLOC0(h->ssum, dpad);
  ALLOC0(h->words, sign ? (size_t)K * nwords : 0);
  ALLOC0(h->words_srv, sign ? nwords : 0);
  ALLOC0(h->mask_srv, topk ? nwords : 0);
  ALLOC0(h->scale[0], KT); ALLOC0(h->scale[1], KT); ALLOC0(h->scale_srv, T);
  ALLOC0(h->tau[0], KT); ALLOC0(h->tau[1], KT); ALLOC0(h->tau_srv, T);
  ALLOC0(h->recs, sign ? KT : 0); ALLOC0(h->recs_srv, sign ? T : 0);
  // latency-bound sizes (the whole K x d state fits L2 several times over): one launch fewer per step
  h->inline_fin = (sign && !shard && (long long)K * dpad <= (1ll << 24)) ? 1 : 0;
  h->small_worker = (SAE_SMALL_WORKER && h->inline_fin && K <= WS_MAXK && !h->mu0) ? 1 : 0;
  if (h->inline_fin) {
    ALLOC0(h->recs_srv_alt, T); ALLOC0(h->recs_srv_alt2, T); ALLOC0(h->recs_srv_alt3, T); ALLOC0(h->recs_alt, KT);
  }
  ALLOC0(h->hist, topk ? KT * HIST_BINS : 0);
  ALLOC0(h->sel, topk ? KT : 0);
  std::vector<long long> cand_off(T, 0);
  std::vector<int> cand_cap(T, 0), wlog2(T, SAE_TOPK_WINDOW_LOG2);
  h->cand_stride = 0;
  if (topk) {
    // room for 8 k_j + 1024 keys per (row, tensor): the window normally catches about 2 k_j
    for (int j = 0; j < T; ++j) {
      unsigned long long kk = ((unsigned long long)h->sizes[j] * cfg->topk_num) / cfg->topk_den;
      if (kk < 1) kk = 1;
      unsigned long long cap = 8 * kk + 1024;
      if (cap > (unsigned long long)h->sizes[j]) cap = (unsigned long long)h->sizes[j];
      cand_off[j] = h->cand_stride; cand_cap[j] = (int)cap;
      // window width: the whole tensor where the region holds it; else 2 % of the old threshold, up to 8 times
      // wider for small k (whose threshold moves more from step to step and whose region has room to spare)
      if (cap >= (unsigned long long)h->sizes[j] && h->sizes[j] <= 16384) wlog2[j] = WINDOW_ALL;   // (small tensors only:
                                        // with a large Top-K ratio every region holds its tensor, and listing all of K x d would not pay)
      else for (unsigned long long w = 2; w <= 8 && w * kk <= 1024; w *= 2) wlog2[j] += 1;
      h->cand_stride += (long long)((cap + 3) / 4 * 4);
    }
  }
  ALLOC0(h->cand_keys, topk ? (size_t)K * h->cand_stride : 0);
  ALLOC0(h->cand_keys_srv, topk ? (size_t)h->cand_stride : 0);
  ALLOC0(h->cand_count, topk ? KT : 0); ALLOC0(h->cand_count_srv, topk ? T : 0);
  ALLOC0(h->fb, topk ? KT : 0); ALLOC0(h->fb_srv, topk ? T : 0); ALLOC0(h->fb_total, 2);
  ALLOC0(h->d_cand_off, T); ALLOC0(h->d_cand_cap, T); ALLOC0(h->d_wlog2, T); ALLOC0(h->d_sel_list, T);
  std::vector<int> sel_list(T);
  for (int j = 0; j < T; ++j) sel_list[j] = j;
  // the order in which the one-launch select takes the tensors: longest candidate regions first, so that their
  // blocks start first and the short ones fill in behind them
  std::stable_sort(sel_list.begin(), sel_list.end(), [&](int a, int b) { return cand_cap[a] > cand_cap[b]; });
  h->n_sel_long = 0;
  for (int j = 0; j < T; ++j) if (cand_cap[j] > SEL_LONG_REGION) h->n_sel_long += 1;
  h->n_sel_long_srv = 0;
  for (int j = 0; j < T; ++j) if (cand_cap[j] > SAE_SRV_LONG_REGION) h->n_sel_long_srv += 1;
  ALLOC0(h->work, topk ? (size_t)ntiles * K + (size_t)K * (h->cand_stride / CAND_CHUNK + T) : 0);
  ALLOC0(h->work_count, 1); ALLOC0(h->cand_n, topk ? KT : 0);
#if SAE_TOPK_PARALLEL_SELECT
  if (h->fused_topk_ok || h->fused_gen_ok) {
    ALLOC0(h->hist_srv, (size_t)T * HIST_BINS); ALLOC0(h->sel_srv, T); ALLOC0(h->cand_n_srv, T); ALLOC0(h->work_count_srv, 1);
    ALLOC0(h->work_srv, (size_t)ntiles + (size_t)(h->cand_stride / CAND_CHUNK + T));
    TRY(cudaStreamCreateWithFlags(&h->aux, cudaStreamNonBlocking));
    TRY(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
    TRY(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
    for (int i = 0; i < 2; ++i) {
      TRY(cudaStreamCreateWithFlags(&h->aux2[i], cudaStreamNonBlocking));
      TRY(cudaEventCreateWithFlags(&h->ev_fork2[i], cudaEventDisableTiming));
      TRY(cudaEventCreateWithFlags(&h->ev_join2[i], cudaEventDisableTiming));
    }
  }
#endif
  ALLOC0(h->status, 1);
  TRY(cudaMallocHost((void**)&h->status_host, sizeof(u32)));
  TRY(cudaMemcpyAsync(h->d_tile_tensor, tile_tensor.data(), sizeof(int) * ntiles, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_first_tile, first_tile.data(), sizeof(int) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_n, n32.data(), sizeof(int) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_off, off.data(), sizeof(long long) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_poff, poff.data(), sizeof(long long) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_cand_off, cand_off.data(), sizeof(long long) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_cand_cap, cand_cap.data(), sizeof(int) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_wlog2, wlog2.data(), sizeof(int) * T, cudaMemcpyHostToDevice, h->stream));
  TRY(cudaMemcpyAsync(h->d_sel_list, sel_list.data(), sizeof(int) * T, cudaMemcpyHostToDevice, h->stream));
#undef ALLOC0
  if (rc == SAE_OK) {
    Plan& P = h->P;
    P.K = K; P.T = T; P.k_pow2 = ((K & (K - 1)) == 0) ? 1 : 0; P.inv_k = 1.0f / (float)K; P.ntiles = (int)ntiles; P.d = d; P.dpad = dpad; P.nwords = nwords;
    P.tile_tensor = h->d_tile_tensor; P.first_tile = h->d_first_tile; P.n = h->d_n; P.off = h->d_off; P.poff = h->d_poff;
    h->P_all = P;
    const int Kt = h->K_total;
    h->P_all.K = Kt; h->P_all.k_pow2 = ((Kt & (Kt - 1)) == 0) ? 1 : 0; h->P_all.inv_k = 1.0f / (float)Kt;
    LAUNCH(h, S_IMPORT, k_import, P.ntiles, P, x0, h->x);
    TRY(cudaGetLastError());
    TRY(cudaStreamSynchronize(h->stream));     // host tables above go out of scope
  }
#undef TRY
  if (rc == SAE_OK && h->fused_topk_ok && !make_row_map(&h->tm_m, h->m, dpad, K, dpad)) h->fused_topk_ok = 0;
  if (rc == SAE_OK && h->fused_gen_ok &&
      !(h->m && h->D && make_row_map(&h->tm_m, h->m, dpad, K, dpad) && make_row_map(&h->tm_D, h->D, dpad, K, dpad)))
    h->fused_gen_ok = 0;
  if (rc == SAE_OK && h->fused_ok) {
    // the folded-averaging pass needs a tensor map over the momentum rows and 32-bit TMA coordinates
    if (dpad >= (1ll << 31) || d >= (1ll << 31) || !make_row_map(&h->tm_m, h->m, dpad, K, dpad)) h->fused_ok = 0;
  }
  if (rc != SAE_OK) { free_all(h); delete h; return rc; }
  if (rc == SAE_OK && shard) {
    const size_t Kt = (size_t)h->K_total;
    h->h_word_rows.assign(Kt, nullptr); h->h_d_rows.assign(Kt, nullptr);
    h->h_scale_rows[0].assign(Kt, nullptr); h->h_scale_rows[1].assign(Kt, nullptr);
    cudaError_t e = dalloc(&h->d_word_rows, Kt);
    if (e == cudaSuccess) e = dalloc(&h->d_scale_rows[0], Kt);
    if (e == cudaSuccess) e = dalloc(&h->d_scale_rows[1], Kt);
    if (e == cudaSuccess) e = dalloc(&h->d_d_rows, Kt);
    if (topk) {
      h->h_entry_rows.assign(Kt, nullptr); h->h_count_rows.assign(Kt, nullptr);
      h->h_tau_rows[0].assign(Kt, nullptr); h->h_tau_rows[1].assign(Kt, nullptr);
      if (e == cudaSuccess) e = dalloc(&h->d_entry_rows, Kt);
      if (e == cudaSuccess) e = dalloc(&h->d_count_rows, Kt);
      if (e == cudaSuccess) e = dalloc(&h->d_tau_rows[0], Kt);
      if (e == cudaSuccess) e = dalloc(&h->d_tau_rows[1], Kt);
      if (e == cudaSuccess) e = dalloc(&h->msg_entries, (size_t)K * (size_t)h->cand_stride);
      if (e == cudaSuccess) e = dalloc(&h->msg_count, KT);
      if (e == cudaSuccess) e = dalloc(&h->agg_acc, (size_t)dpad);
      if (e == cudaSuccess) e = cudaMemsetAsync(h->msg_count, 0, KT * sizeof(u32), h->stream);
      if (e == cudaSuccess) e = cudaMemsetAsync(h->agg_acc, 0, (size_t)dpad * sizeof(float), h->stream);
      if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    }
    if (e != cudaSuccess) { h->last_cuda_error = (int)e; g_init_cuda_error = (int)e; cudaGetLastError(); rc = SAE_ERR_NOMEM; }
  }
  if (rc != SAE_OK) { free_all(h); delete h; return rc; }
  // Pre-step of iteration 0: all errors are zero, so averaging (if (0+1) mod p = 0) changes nothing.
  *out = h;
  return SAE_OK;
}

// ---- sharded operation ------------------------------------------------------------------------------
// What a shard publishes: where its workers' message rows (sign words, the two scale buffers) and stored
// model differences live.  Same process: the raw pointers; another process: CUDA IPC handles.
struct ShardBlob {
  uint64_t magic;
  int32_t pid, device, worker_begin, num_local, T, pad;
  int64_t nwords, dpad;
  int32_t compressor, pad2;
  int64_t cand_stride;
  void* raw[8];                       // words, scale[0], scale[1], D | Top-K: entries, counts, tau[0], tau[1]
  cudaIpcMemHandle_t ipc[8];
};
constexpr int kShardBufs = 8;
constexpr uint64_t kShardMagic = 0x5341455F53484432ull;   // "SAE_SHD2"
static_assert(sizeof(ShardBlob) <= SAE_SHARD_BLOB_BYTES, "blob must fit the documented size");

int shard_begin(sae_handle* h, const float* grads, float lr) {
  const sae_config& c = h->cfg;
  const Plan& P = h->P;
  const int cur = 1 - h->last;
  StepParams sp;
  sp.mu = c.momentum; sp.eta = lr; sp.lambda = c.weight_decay;
  sp.saef = (c.mode == SAE_MODE_SAEF); sp.wd = (c.weight_decay != 0.0f);
  WorkerArgs wa;
  wa.wc = h->wc;
  wa.g = grads; wa.m = h->m; wa.D = h->D; wa.ebar = h->ebar; wa.x = h->x;
  wa.scale_prev = h->scale[h->last]; wa.tau_prev = h->tau[h->last];
  wa.words = h->words; wa.scale_cur = h->scale[cur]; wa.recs = h->recs; wa.status = h->status;
  wa.cand = cand_args(h, false);
  if (c.compressor == SAE_COMPRESSOR_TOPK) {
    // worker lines, the local workers' thresholds, then their messages: the lists of selected entries
    SAE_CUDA(h, cudaMemsetAsync(h->msg_count, 0, sizeof(u32) * (size_t)P.K * P.T, h->stream));
    if (h->esrc == ESRC_UNIFORM) launch_worker<ESRC_UNIFORM, false, true, true>(h, sp, wa);
    else launch_worker<ESRC_LAZY_TOPK, false, true, true>(h, sp, wa);
    topk_thresholds(h, stored_rows(h->D), P.K, wa.cand, h->tau[h->last], h->tau[cur], h->fb, h->fb_total);
    SparseMsgArgs ma;
    ma.D = h->D; ma.tau = h->tau[cur]; ma.entries = h->msg_entries; ma.off = h->d_cand_off; ma.cap = h->d_cand_cap;
    ma.stride = h->cand_stride; ma.count = h->msg_count;
    LAUNCH(h, S_TOPK_SELECT, k_topk_compact, (long long)P.ntiles * P.K, P, ma);
    h->mid_step = 1; h->lr_pending = lr;
    return check_launch(h);
  }
  // the model differences are always stored: the averaging reads them from every owner
  if (h->esrc == ESRC_UNIFORM) launch_worker<ESRC_UNIFORM, true, true>(h, sp, wa);
  else launch_worker<ESRC_LAZY_SIGN, true, true>(h, sp, wa);
  LAUNCH(h, S_FINALIZE, k_finalize_scales, (P.K * P.T + P.T + THREADS - 1) / THREADS, P.K, P.T, h->d_n, h->recs,
         h->scale[cur], h->recs_srv, (float*)nullptr);
  h->mid_step = 1; h->lr_pending = lr;
  return check_launch(h);
}

int shard_end(sae_handle* h) {
  const sae_config& c = h->cfg;
  const Plan& PA = h->P_all;
  const int cur = 1 - h->last;
  const bool dc = c.server_compress != 0;
  const bool avg_after = c.avg_period > 0 && ((h->t + 2) % c.avg_period == 0);
  ServerArgs sa;
  memset(&sa, 0, sizeof(sa));
  sa.wc = h->wc;
  sa.e_srv = h->e_srv; sa.words_srv = h->words_srv; sa.scale_srv = h->scale_srv; sa.recs_srv = h->recs_srv;
  sa.status = h->status; sa.word_rows = h->d_word_rows; sa.scale_rows = h->d_scale_rows[cur];
  ApplyArgs aa;
  memset(&aa, 0, sizeof(aa));
  aa.e_srv = h->e_srv; aa.x = h->x; aa.ebar = h->ebar; aa.scale_srv = h->scale_srv; aa.recs_srv = h->recs_srv;
  aa.eta = h->lr_pending;
  if (c.compressor == SAE_COMPRESSOR_TOPK) {
    // the ordered worker-axis sum from every owner's list of selected entries, then the server lines
    SparseAggArgs ga;
    ga.e_srv = h->e_srv; ga.acc = h->agg_acc; ga.entry_rows = h->d_entry_rows; ga.count_rows = h->d_count_rows;
    ga.d_rows = h->d_d_rows; ga.tau_rows = h->d_tau_rows[cur]; ga.off = h->d_cand_off; ga.cap = h->d_cand_cap;
    {
      LaunchScope ls(h, S_SERVER);
      k_topk_sparse_aggregate<<<(unsigned)((PA.ntiles + AGG_TILES - 1) / AGG_TILES), AGG_THREADS, 0, h->stream>>>(PA, ga);
    }
    aa.tau_srv = h->tau_srv; aa.mask_srv = h->mask_srv;
    if (dc) {
      LAUNCH(h, S_SERVER, k_server_candidates, PA.ntiles, PA, h->e_srv, cand_args(h, true), h->tau_srv);
      topk_thresholds(h, stored_rows(h->e_srv), 1, cand_args(h, true), h->tau_srv, h->tau_srv, h->fb_srv, h->fb_total + 1);
      LAUNCH(h, S_APPLY, (k_apply<2, 2, AVG_NONE>), PA.ntiles, PA, aa);
    } else {
      LAUNCH(h, S_APPLY, (k_apply<2, 0, AVG_NONE>), PA.ntiles, PA, aa);
    }
    if (avg_after && !h->avg_external)
      LAUNCH(h, S_APPLY, (k_avg_pull<false, 2>), PA.ntiles, PA, h->d_d_rows, (const void* const*)h->d_tau_rows[cur], h->ebar);
    if (avg_after && h->avg_external) h->avg_owed = 1;
    h->esrc = (avg_after && !h->avg_external) ? ESRC_UNIFORM : ESRC_LAZY_TOPK;
    h->last = cur; h->eta_prev = h->lr_pending; h->t += 1; h->mid_step = 0;
    return check_launch(h);
  }
  const int tpb = std::max(1, std::min(8, PA.ntiles / (h->num_sms * 16)));
  const int nblk = (PA.ntiles + tpb - 1) / tpb;
  if (dc) LAUNCH(h, S_SERVER, (k_server_sign<true, true>), nblk, PA, sa, tpb);
  else LAUNCH(h, S_SERVER, (k_server_sign<false, true>), nblk, PA, sa, tpb);
  if (dc) LAUNCH(h, S_APPLY, (k_apply<1, 1, AVG_NONE>), PA.ntiles, PA, aa);
  else LAUNCH(h, S_APPLY, (k_apply<1, 0, AVG_NONE>), PA.ntiles, PA, aa);
  if (avg_after && !h->avg_external)
    LAUNCH(h, S_APPLY, (k_avg_pull<false, 1>), PA.ntiles, PA, h->d_d_rows, (const void* const*)h->d_scale_rows[cur], h->ebar);
  if (avg_after && h->avg_external) h->avg_owed = 1;     // the error stays "lazy" until sae_avg_set
  h->esrc = (avg_after && !h->avg_external) ? ESRC_UNIFORM : ESRC_LAZY_SIGN;
  h->last = cur; h->eta_prev = h->lr_pending; h->t += 1; h->mid_step = 0;
  return check_launch(h);
}

}  // namespace

extern "C" {

int sae_init(const sae_config* cfg, const float* x0, sae_handle** out) {
  if (out) *out = nullptr;
  if (!cfg) return SAE_ERR_INVALID_ARG;
  return init_impl(cfg, 0, cfg->num_workers, false, x0, out);
}

int sae_init_shard(const sae_config* cfg, int32_t worker_begin, int32_t num_local_workers, const float* x0,
                   sae_handle** out) {
  if (out) *out = nullptr;
  if (!cfg) return SAE_ERR_INVALID_ARG;
  return init_impl(cfg, worker_begin, num_local_workers, true, x0, out);
}

int sae_shard_export(sae_handle* h, void* blob_host, size_t bytes) {
  if (!h || !blob_host || bytes < SAE_SHARD_BLOB_BYTES || !h->shard) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  ShardBlob b;
  memset(&b, 0, sizeof(b));
  b.magic = kShardMagic; b.pid = (int32_t)getpid(); b.device = h->device; b.worker_begin = h->k0; b.num_local = h->P.K;
  b.T = h->P.T; b.nwords = h->P.nwords; b.dpad = h->P.dpad;
  b.compressor = h->cfg.compressor; b.cand_stride = h->cand_stride;
  b.raw[0] = h->words; b.raw[1] = h->scale[0]; b.raw[2] = h->scale[1]; b.raw[3] = h->D;
  if (h->cfg.compressor == SAE_COMPRESSOR_TOPK) {
    b.raw[4] = h->msg_entries; b.raw[5] = h->msg_count; b.raw[6] = h->tau[0]; b.raw[7] = h->tau[1];
  }
  for (int q = 0; q < kShardBufs; ++q)
    if (b.raw[q]) SAE_CUDA(h, cudaIpcGetMemHandle(&b.ipc[q], b.raw[q]));
  memset(blob_host, 0, SAE_SHARD_BLOB_BYTES);
  memcpy(blob_host, &b, sizeof(b));
  return SAE_OK;
}

int sae_shard_attach(sae_handle* h, const void* blob_host, size_t bytes) {
  if (!h || !blob_host || bytes < SAE_SHARD_BLOB_BYTES || !h->shard || h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  ShardBlob b;
  memcpy(&b, blob_host, sizeof(b));
  if (b.magic != kShardMagic || b.T != h->P.T || b.nwords != h->P.nwords || b.dpad != h->P.dpad || b.worker_begin < 0 ||
      b.num_local < 1 || b.worker_begin + b.num_local > h->K_total || b.compressor != h->cfg.compressor ||
      b.cand_stride != h->cand_stride)
    return SAE_ERR_INVALID_ARG;
  for (int q = 0; q < b.num_local; ++q)
    if (h->h_word_rows[(size_t)b.worker_begin + q]) return SAE_ERR_INVALID_ARG;      // rows already attached
  void* base[kShardBufs];
  if (b.pid == (int32_t)getpid()) {
    if (b.device != h->device) {
      // rows of another GPU driven by this process: they are only readable from here once peer access is on
      int can = 0;
      if (b.device < 0 || cudaDeviceCanAccessPeer(&can, h->device, b.device) != cudaSuccess || !can) {
        cudaGetLastError();
        return SAE_ERR_INVALID_ARG;
      }
      const cudaError_t pe = cudaDeviceEnablePeerAccess(b.device, 0);
      if (pe != cudaSuccess && pe != cudaErrorPeerAccessAlreadyEnabled) {
        h->last_cuda_error = (int)pe; cudaGetLastError();
        return SAE_ERR_CUDA;
      }
      cudaGetLastError();
    }
    for (int q = 0; q < kShardBufs; ++q) base[q] = b.raw[q];
  } else {
    for (int q = 0; q < kShardBufs; ++q) {
      base[q] = nullptr;
      if (!b.raw[q]) continue;
      SAE_CUDA(h, cudaIpcOpenMemHandle(&base[q], b.ipc[q], cudaIpcMemLazyEnablePeerAccess));
      h->ipc_opened.push_back(base[q]);
    }
  }
  const bool topk_rows = h->cfg.compressor == SAE_COMPRESSOR_TOPK;
  for (int q = 0; q < b.num_local; ++q) {
    const size_t k = (size_t)b.worker_begin + q;
    h->h_word_rows[k] = (const u32*)base[0] + (size_t)q * b.nwords;
    h->h_scale_rows[0][k] = (const float*)base[1] + (size_t)q * b.T;
    h->h_scale_rows[1][k] = (const float*)base[2] + (size_t)q * b.T;
    h->h_d_rows[k] = (const float*)base[3] + (size_t)q * b.dpad;
    if (topk_rows) {
      h->h_entry_rows[k] = (const unsigned long long*)base[4] + (size_t)q * (size_t)b.cand_stride;
      h->h_count_rows[k] = (const u32*)base[5] + (size_t)q * b.T;
      h->h_tau_rows[0][k] = (const u32*)base[6] + (size_t)q * b.T;
      h->h_tau_rows[1][k] = (const u32*)base[7] + (size_t)q * b.T;
    }
  }
  h->attached += b.num_local;
  if (h->attached == h->K_total) {
    const size_t Kt = (size_t)h->K_total;
    SAE_CUDA(h, cudaMemcpyAsync(h->d_word_rows, h->h_word_rows.data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
    SAE_CUDA(h, cudaMemcpyAsync(h->d_scale_rows[0], h->h_scale_rows[0].data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
    SAE_CUDA(h, cudaMemcpyAsync(h->d_scale_rows[1], h->h_scale_rows[1].data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
    SAE_CUDA(h, cudaMemcpyAsync(h->d_d_rows, h->h_d_rows.data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
    if (topk_rows) {
      SAE_CUDA(h, cudaMemcpyAsync(h->d_entry_rows, h->h_entry_rows.data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
      SAE_CUDA(h, cudaMemcpyAsync(h->d_count_rows, h->h_count_rows.data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
      SAE_CUDA(h, cudaMemcpyAsync(h->d_tau_rows[0], h->h_tau_rows[0].data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
      SAE_CUDA(h, cudaMemcpyAsync(h->d_tau_rows[1], h->h_tau_rows[1].data(), Kt * sizeof(void*), cudaMemcpyHostToDevice, h->stream));
    }
    SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  }
  return SAE_OK;
}

int sae_shard_detach(sae_handle* h) {
  if (!h || !h->shard || h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  for (void* p : h->ipc_opened) cudaIpcCloseMemHandle(p);
  h->ipc_opened.clear();
  for (auto& r : h->h_word_rows) r = nullptr;
  for (auto& r : h->h_d_rows) r = nullptr;
  for (auto& r : h->h_scale_rows[0]) r = nullptr;
  for (auto& r : h->h_scale_rows[1]) r = nullptr;
  for (auto& r : h->h_entry_rows) r = nullptr;
  for (auto& r : h->h_count_rows) r = nullptr;
  for (auto& r : h->h_tau_rows[0]) r = nullptr;
  for (auto& r : h->h_tau_rows[1]) r = nullptr;
  h->attached = 0;
  return SAE_OK;
}

int sae_set_local_steps(sae_handle* h, int32_t period) {
  if (!h || period < 1 || h->t != 0 || h->shard) return SAE_ERR_INVALID_ARG;
  if (period > 1 && (h->cfg.mode != SAE_MODE_SAEF || h->cfg.avg_period != 0)) return SAE_ERR_INVALID_ARG;
  h->local_steps = period;
  return SAE_OK;
}

int sae_shard_set_avg_mode(sae_handle* h, int32_t external_sum) {
  if (!h || !h->shard || h->mid_step || h->avg_owed) return SAE_ERR_INVALID_ARG;
  h->avg_external = external_sum ? 1 : 0;
  return SAE_OK;
}

int sae_avg_due(const sae_handle* h) { return (h && h->avg_owed) ? 1 : 0; }
int64_t sae_num_padded(const sae_handle* h) { return h ? h->P.dpad : -1; }

int sae_avg_local_sum(sae_handle* h, float* sum_padded) {
  if (!h || !sum_padded || !h->shard || !h->avg_owed || h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  // this shard's own rows, k in order: the table entries k0 .. k0+K-1 with the local plan (K = local workers)
  if (h->cfg.compressor == SAE_COMPRESSOR_TOPK)
    LAUNCH(h, S_APPLY, (k_avg_pull<true, 2>), h->P.ntiles, h->P, h->d_d_rows + h->k0,
           (const void* const*)(h->d_tau_rows[h->last] + h->k0), sum_padded);
  else
    LAUNCH(h, S_APPLY, (k_avg_pull<true, 1>), h->P.ntiles, h->P, h->d_d_rows + h->k0,
           (const void* const*)(h->d_scale_rows[h->last] + h->k0), sum_padded);
  return check_launch(h);
}

int sae_avg_set(sae_handle* h, const float* sum_padded) {
  if (!h || !sum_padded || !h->shard || !h->avg_owed || h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  LAUNCH(h, S_APPLY, k_avg_set, h->P_all.ntiles, h->P_all, sum_padded, h->ebar);
  h->esrc = ESRC_UNIFORM;
  h->avg_owed = 0;
  return check_launch(h);
}

int sae_step_begin(sae_handle* h, const float* grads_local, float lr) {
  ApiRange nvtx_range("sae_step_begin");
  if (!h || !grads_local || !(lr > 0.0f) || !(lr < 3.0e38f)) return SAE_ERR_INVALID_ARG;
  if (!h->shard || h->mid_step || h->avg_owed || h->attached != h->K_total) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  return shard_begin(h, grads_local, lr);
}

int sae_step_end(sae_handle* h) {
  ApiRange nvtx_range("sae_step_end");
  if (!h || !h->shard || !h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  return shard_end(h);
}

int sae_step(sae_handle* h, const float* grads, float lr) {
  ApiRange nvtx_range("sae_step");
  if (!h || !grads || !(lr > 0.0f) || !(lr < 3.0e38f) || h->shard) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  return do_step(h, grads, lr);
}

int sae_step_host(sae_handle* h, const float* grads_host, float lr) {
  ApiRange nvtx_range("sae_step_host");
  if (!h || !grads_host || !(lr > 0.0f) || !(lr < 3.0e38f) || h->shard) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  const size_t count = (size_t)h->P.K * (size_t)h->P.d;
  if (!h->staging) SAE_CUDA(h, dalloc(&h->staging, count));
  SAE_CUDA(h, cudaMemcpyAsync(h->staging, grads_host, count * sizeof(float), cudaMemcpyHostToDevice, h->stream));
  return do_step(h, h->staging, lr);
}

int sae_get_params(sae_handle* h, float* out) {
  ApiRange nvtx_range("sae_get_params");
  if (!h || !out) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  return export_vec(h, EXP_X, 0, out);
}

int sae_get_params_host(sae_handle* h, float* out_host) {
  if (!h || !out_host) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  // Export into a library-owned caller-layout buffer (allocated by the first call), then one
  // contiguous device-to-host copy.
  if (!h->out_stage) SAE_CUDA(h, dalloc(&h->out_stage, (size_t)h->P.d));
  int rc = export_vec(h, EXP_X, 0, h->out_stage);
  if (rc != SAE_OK) return rc;
  SAE_CUDA(h, cudaMemcpyAsync(out_host, h->out_stage, sizeof(float) * h->P.d, cudaMemcpyDeviceToHost, h->stream));
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  return SAE_OK;
}

int sae_get_step_ahead(sae_handle* h, int32_t worker, float* out) {
  ApiRange nvtx_range("sae_get_step_ahead");
  if (!h || !out || worker < 0 || worker >= h->P.K) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  return export_vec(h, EXP_STEP_AHEAD, worker, out);
}

int sae_get_state(sae_handle* h, int32_t which, int32_t worker, void* out, size_t bytes) {
  if (!h || !out) return SAE_ERR_INVALID_ARG;
  const Plan& P = h->P;
  const bool per_worker = which == SAE_STATE_MOMENTUM || which == SAE_STATE_WORKER_ERROR ||
                          which == SAE_STATE_WORKER_SCALES || which == SAE_STATE_WORKER_WORDS ||
                          which == SAE_STATE_WORKER_TAU || which == SAE_STATE_WORKER_MASK;
  if (per_worker && (worker < 0 || worker >= P.K)) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  { int rct = flush_tail(h); if (rct != SAE_OK) return rct; }
  if (which == SAE_STATE_SERVER_SCALES || which == SAE_STATE_SERVER_MASK) {
    int rcf = flush_server(h);
    if (rcf != SAE_OK) return rcf;
  }
  const bool sign = h->cfg.compressor == SAE_COMPRESSOR_SIGN, topk = h->cfg.compressor == SAE_COMPRESSOR_TOPK;
  const size_t vec = sizeof(float) * (size_t)P.d, tb = sizeof(float) * (size_t)P.T, wb = sizeof(u32) * (size_t)P.nwords;
  const void* src = nullptr; size_t need = 0;
  switch (which) {
    case SAE_STATE_MOMENTUM:
      if (bytes < vec || !h->m) return SAE_ERR_INVALID_ARG;       // (mu = 0: m^(k) is not kept)
      return export_vec(h, EXP_M, worker, (float*)out);
    case SAE_STATE_WORKER_ERROR: if (bytes < vec) return SAE_ERR_INVALID_ARG; return export_vec(h, EXP_WERR, worker, (float*)out);
    case SAE_STATE_SERVER_ERROR: if (bytes < vec) return SAE_ERR_INVALID_ARG; return export_vec(h, EXP_ESRV, 0, (float*)out);
    case SAE_STATE_WORKER_SCALES: if (!sign) return SAE_ERR_INVALID_ARG; src = h->scale[h->last] + (size_t)worker * P.T; need = tb; break;
    case SAE_STATE_SERVER_SCALES: if (!sign) return SAE_ERR_INVALID_ARG; src = h->scale_srv; need = tb; break;
    case SAE_STATE_WORKER_WORDS: if (!sign) return SAE_ERR_INVALID_ARG; src = h->words + (size_t)worker * P.nwords; need = wb; break;
    case SAE_STATE_SERVER_WORDS: if (!sign) return SAE_ERR_INVALID_ARG; src = h->words_srv; need = wb; break;
    case SAE_STATE_WORKER_TAU: if (!topk) return SAE_ERR_INVALID_ARG; src = h->tau[h->last] + (size_t)worker * P.T; need = tb; break;
    case SAE_STATE_SERVER_TAU: if (!topk) return SAE_ERR_INVALID_ARG; src = h->tau_srv; need = tb; break;
    case SAE_STATE_SERVER_MASK: if (!topk) return SAE_ERR_INVALID_ARG; src = h->mask_srv; need = wb; break;
    case SAE_STATE_TOPK_FALLBACKS: if (!topk) return SAE_ERR_INVALID_ARG; src = h->fb_total; need = 2 * sizeof(u32); break;
    case SAE_STATE_WORKER_MASK:
      if (!topk || bytes < wb) return SAE_ERR_INVALID_ARG;
      {
        DeltaSrc src = stored_rows(h->D ? h->D + (size_t)worker * P.dpad : nullptr);
        if (h->topk_nod) {     // the last step's differences: its learning rate, the uniform error it started from
          src.m = h->m + (size_t)worker * P.dpad; src.ebar = ebar_other(h); src.eta = h->eta_prev; src.recompute = 1;
        }
        LAUNCH(h, S_MASK, k_mask_words, P.ntiles, P, src, h->tau[h->last] + (size_t)worker * P.T, (u32*)out);
      }
      return check_launch(h);
    default: return SAE_ERR_INVALID_ARG;
  }
  if (bytes < need) return SAE_ERR_INVALID_ARG;
  SAE_CUDA(h, cudaMemcpyAsync(out, src, need, cudaMemcpyDeviceToDevice, h->stream));
  return SAE_OK;
}

int64_t sae_state_bytes(sae_handle* h) { return h ? (int64_t)ckpt_bytes(h) : -1; }

int sae_save_state(sae_handle* h, void* out, size_t bytes) {
  if (!h || !out || bytes < ckpt_bytes(h) || h->mid_step || h->avg_owed) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  { int rcf = flush_server(h); if (rcf != SAE_OK) return rcf; }
  CkptHeader hd;
  memset(&hd, 0, sizeof(hd));
  hd.magic = kCkptMagic; hd.K = h->P.K; hd.T = h->P.T; hd.compressor = h->cfg.compressor;
  hd.server_compress = h->cfg.server_compress; hd.mode = h->cfg.mode; hd.avg_period = h->cfg.avg_period;
  hd.topk_num = h->cfg.topk_num; hd.topk_den = h->cfg.topk_den; hd.momentum = h->cfg.momentum;
  hd.weight_decay = h->cfg.weight_decay; hd.d = h->P.d; hd.t = h->t; hd.esrc = h->esrc; hd.last = h->last;
  hd.eta_prev = h->eta_prev; hd.worker_begin = h->k0; hd.num_workers_total = h->K_total;
  hd.local_steps = h->local_steps;
  SAE_CUDA(h, cudaMemcpyAsync(out, &hd, sizeof(hd), cudaMemcpyHostToDevice, h->stream));
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));        // hd lives on this stack frame
  char* q = (char*)out + 256;
  for (const auto& s : ckpt_sections(h)) {
    SAE_CUDA(h, cudaMemcpyAsync(q, s.ptr, s.bytes, cudaMemcpyDeviceToDevice, h->stream));
    q += (s.bytes + 255) / 256 * 256;
  }
  return SAE_OK;
}

int sae_load_state(sae_handle* h, const void* in, size_t bytes) {
  if (!h || !in || bytes < ckpt_bytes(h) || h->mid_step) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  CkptHeader hd;
  SAE_CUDA(h, cudaMemcpyAsync(&hd, in, sizeof(hd), cudaMemcpyDeviceToHost, h->stream));
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  const sae_config& c = h->cfg;
  if (hd.magic != kCkptMagic || hd.K != h->P.K || hd.T != h->P.T || hd.d != h->P.d || hd.compressor != c.compressor ||
      hd.server_compress != c.server_compress || hd.mode != c.mode || hd.avg_period != c.avg_period ||
      hd.topk_num != c.topk_num || hd.topk_den != c.topk_den || hd.momentum != c.momentum ||
      hd.weight_decay != c.weight_decay || hd.worker_begin != h->k0 || hd.num_workers_total != h->K_total ||
      std::max(hd.local_steps, 1) != h->local_steps)
    return SAE_ERR_INVALID_ARG;                         // a checkpoint of a different configuration
  if (hd.esrc == ESRC_PENDING_AVG && !h->fused_ok && !(h->small_worker && c.avg_period == 1)) return SAE_ERR_INVALID_ARG;
  const char* q = (const char*)in + 256;
  for (const auto& s : ckpt_sections(h)) {
    SAE_CUDA(h, cudaMemcpyAsync(s.ptr, q, s.bytes, cudaMemcpyDeviceToDevice, h->stream));
    q += (s.bytes + 255) / 256 * 256;
  }
  h->t = hd.t; h->esrc = hd.esrc; h->last = hd.last; h->eta_prev = hd.eta_prev;
  h->srv_pending = 0;        // a checkpoint is taken with the server lines carried out
  h->tail_pending = 0; h->recs_srv_fresh = 0;
  if (h->inline_fin) {       // the L1 records are transient, but nothing else clears them before the next step
    SAE_CUDA(h, cudaMemsetAsync(h->recs, 0, sizeof(L1Record) * (size_t)h->P.K * h->P.T, h->stream));
    SAE_CUDA(h, cudaMemsetAsync(h->recs_srv, 0, sizeof(L1Record) * (size_t)h->P.T, h->stream));
    SAE_CUDA(h, cudaMemsetAsync(h->recs_srv_alt, 0, sizeof(L1Record) * (size_t)h->P.T, h->stream));
    SAE_CUDA(h, cudaMemsetAsync(h->recs_srv_alt2, 0, sizeof(L1Record) * (size_t)h->P.T, h->stream));
    SAE_CUDA(h, cudaMemsetAsync(h->recs_srv_alt3, 0, sizeof(L1Record) * (size_t)h->P.T, h->stream));
    SAE_CUDA(h, cudaMemsetAsync(h->recs_alt, 0, sizeof(L1Record) * (size_t)h->P.K * h->P.T, h->stream));
    h->rot = 0;
  }
  return SAE_OK;
}

int sae_get_mismatch(sae_handle* h, double* out_host) {
  if (!h || !out_host || h->shard) return SAE_ERR_INVALID_ARG;     // needs every worker's error in one place
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  { int rcf = flush_server(h); if (rcf != SAE_OK) return rcf; }
  if (!h->mismatch) SAE_CUDA(h, dalloc(&h->mismatch, 2));
  SAE_CUDA(h, cudaMemsetAsync(h->mismatch, 0, 2 * sizeof(double), h->stream));
  { int rca = close_pending_avg(h); if (rca != SAE_OK) return rca; }
  const ExportArgs ea = export_args(h, EXP_WERR, 0);
  LAUNCH(h, S_EXPORT, k_mismatch, h->P.ntiles, h->P, ea, h->mismatch);
  int rc = check_launch(h);
  if (rc != SAE_OK) return rc;
  SAE_CUDA(h, cudaMemcpyAsync(out_host, h->mismatch, 2 * sizeof(double), cudaMemcpyDeviceToHost, h->stream));
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  return SAE_OK;
}

int64_t sae_iteration(const sae_handle* h) { return h ? h->t : -1; }
int64_t sae_num_params(const sae_handle* h) { return h ? h->P.d : -1; }
int64_t sae_num_words(const sae_handle* h) { return h ? h->P.nwords : -1; }

int sae_sync(sae_handle* h) {
  if (!h) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  SAE_CUDA(h, cudaMemcpyAsync(h->status_host, h->status, sizeof(u32), cudaMemcpyDeviceToHost, h->stream));
  SAE_CUDA(h, cudaMemsetAsync(h->status, 0, sizeof(u32), h->stream));
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  const u32 st = *h->status_host;
  if (st & STATUS_TIMEOUT) return SAE_ERR_TIMEOUT;
  if (st & STATUS_RANGE) return SAE_ERR_RANGE;
  return SAE_OK;
}

int sae_set_profiling(sae_handle* h, int32_t enabled) {
  if (!h) return SAE_ERR_INVALID_ARG;
  h->profiling = enabled ? 1 : 0;
  return SAE_OK;
}

int sae_get_kernel_times(sae_handle* h, float* ms_host, int64_t* launches_host) {
  if (!h || !ms_host || !launches_host) return SAE_ERR_INVALID_ARG;
  DeviceGuard guard(h->device);
  if (!guard.ok) return SAE_ERR_CUDA;
  SAE_CUDA(h, cudaStreamSynchronize(h->stream));
  for (auto& ep : h->pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ep.a, ep.b) == cudaSuccess) { h->ms[ep.slot] += ms; h->cnt[ep.slot] += 1; }
    h->pool.push_back(ep.a); h->pool.push_back(ep.b);
  }
  h->pending.clear();
  for (int i = 0; i < SAE_NUM_KERNELS; ++i) {
    ms_host[i] = (float)h->ms[i]; launches_host[i] = h->cnt[i];
    h->ms[i] = 0; h->cnt[i] = 0;
  }
  return SAE_OK;
}

const char* sae_kernel_name(int32_t slot) {
  if (slot < 0 || slot >= SAE_NUM_KERNELS) return "";
  return kSlotNames[slot];
}

int64_t sae_kernel_launches(const sae_handle* h) { return h ? h->launches : -1; }

void sae_destroy(sae_handle* h) {
  if (!h) return;
  DeviceGuard guard(h->device);
  if (guard.ok) cudaStreamSynchronize(h->stream);
  free_all(h);
  delete h;
}

const char* sae_strerror(int status) {
  switch (status) {
    case SAE_OK: return "ok";
    case SAE_ERR_INVALID_ARG: return "invalid argument";
    case SAE_ERR_NOMEM: return "out of memory";
    case SAE_ERR_CUDA: return "CUDA runtime error";
    case SAE_ERR_RANGE: return "model difference non-finite or out of range (|v| >= 2^32)";
    case SAE_ERR_TIMEOUT: return "device wait timed out";
    case SAE_ERR_ABI: return "ABI version mismatch";
    case SAE_ERR_TOO_LARGE: return "input exceeds the fixed scratch capacity of the no-allocation entry point";
    default: return "unknown status";
  }
}

int sae_last_cuda_error(const sae_handle* h) { return h ? h->last_cuda_error : g_init_cuda_error; }

}  // extern "C"
