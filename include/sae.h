/*
 * sae.h -- C ABI of the Step-Ahead Error Feedback hot path (sm_100a CUDA library, libsae.so).
 *
 * One handle holds the whole state of Algorithm 1 ("Distributed Momentum SGD with Double-Way
 * Compression") for K data-parallel workers simulated as a batch axis on ONE GPU (or, in sharded
 * operation, the rows of some of the workers: see sae_init_shard): parameters x,
 * server error e, per-worker momentum m^(k) and per-worker error e^(k).  The caller supplies the
 * stochastic gradients; the library performs every other line of the algorithm in CUDA kernels.
 *
 * Conventions
 *  - All pointers are DEVICE pointers unless the name ends in _host.  The library never takes
 *    ownership of a caller buffer; it owns its state and scratch (allocated in sae_init only).
 *  - "Caller layout" of a parameter-shaped vector: the T tensors concatenated in list order with no
 *    padding, d = sum_j n_j floats.  Gradients are [K][d] row-major in that layout.
 *  - All work is enqueued on the stream given in the configuration and is asynchronous with respect
 *    to the host unless stated otherwise.  A handle must not be used from two host threads at once.
 *  - Arithmetic is IEEE fp32, round-to-nearest, denormals kept, with the fused operations fixed:
 *    m = fma(mu, m, g'), Delta = fma(eta, m, e), g' = fma(lambda, xh, g); everything else is one
 *    separately rounded operation; worker-axis sums run k = 0..K-1 from 0 and are divided by (float)K.
 *  - Every function returns SAE_OK (0) or a negative sae_status.  No exceptions, no global state.
 *    Errors detected on the device (non-finite or out-of-range values) are sticky and are reported
 *    by the next sae_sync call.
 */
#ifndef SAE_H_
#define SAE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SAE_ABI_VERSION 1u

typedef enum {
  SAE_OK = 0,
  SAE_ERR_INVALID_ARG = -1, /* null pointer, K < 1, n_j <= 0, mu outside [0,1), lr <= 0, bad enum, ... */
  SAE_ERR_NOMEM = -2,       /* device or host allocation failed                                          */
  SAE_ERR_CUDA = -3,        /* a CUDA runtime call failed; sae_last_cuda_error gives the code            */
  SAE_ERR_RANGE = -4,       /* a model difference was non-finite or had magnitude >= 2^32 (device check) */
  SAE_ERR_TIMEOUT = -5,     /* a bounded device-side wait (on a shared-memory barrier) expired           */
  SAE_ERR_ABI = -6,         /* abi_version mismatch                                                      */
  SAE_ERR_TOO_LARGE = -7    /* input larger than the fixed scratch of sae_sign_compress_noalloc          */
} sae_status;

/* Compressor C(.) of Algorithm 1, applied per tensor (Section 5: "layer-wise"). */
#define SAE_COMPRESSOR_IDENTITY 0 /* C(v) = v: full-precision distributed momentum SGD (Section 2)       */
#define SAE_COMPRESSOR_SIGN 1     /* Eq. 2: C(v) = (||v||_1 / n) sign(v), sent as 1 scale + 1 bit/element */
#define SAE_COMPRESSOR_TOPK 2     /* Section 3.1: keep the k largest magnitudes, zero the rest           */

#define SAE_MODE_EF 0   /* Algorithm 1, "Local Error Feedback" branch: gradient evaluated at x_t          */
#define SAE_MODE_SAEF 1 /* Algorithm 1, "Step Ahead Error Feedback" branch: at x_t - e_t^(k)              */

typedef struct sae_handle sae_handle; /* opaque, library-owned */

typedef struct {
  uint32_t abi_version;        /* must be SAE_ABI_VERSION                                               */
  int32_t num_workers;         /* K of Algorithm 1, 1..1024                                             */
  int32_t num_tensors;         /* T >= 1 compression segments                                           */
  const int64_t *tensor_sizes; /* HOST pointer, T entries, 0 < n_j <= 2^30; copied by sae_init          */
  int32_t compressor;          /* SAE_COMPRESSOR_*                                                      */
  int32_t server_compress;     /* 1: double-way compression (server applies C, keeps its error e);
                                  0: single-way (server sends Delta uncompressed, e stays 0) (Section 5) */
  int32_t mode;                /* SAE_MODE_*                                                            */
  int32_t avg_period;          /* p >= 1: worker errors are averaged in the pre-step of every iteration
                                  t with (t+1) mod p = 0 (Algorithm 1, Section 3.2); 0 = never (p = inf) */
  float momentum;              /* mu in [0,1).  mu = 0 (the SGD / SignSGD variants) with avg_period != 1:
                                  m^(k) equals the step's gradient term and is not kept -- no momentum
                                  rows are allocated, read or written, SAE_STATE_MOMENTUM is refused, and
                                  a -0 gradient term counts as +0 (fma(0, m, -0) would keep the sign of m) */
  float weight_decay;          /* lambda >= 0: coupled L2, lambda * (point where the gradient is
                                  evaluated) is added to the gradient                                    */
  uint32_t topk_num, topk_den; /* Top-K keeps k_j = max(1, floor(n_j*num/den)) entries per tensor; all
                                  entries tying the k_j-th magnitude are kept, exact zeros never are     */
  int32_t device;              /* CUDA device ordinal                                                   */
  void *stream;                /* cudaStream_t (NULL = default stream)                                  */
} sae_config;

/*
 * Algorithm 1, "Initialize": x = x0, m^(k) = 0, e^(k) = 0, e = 0, t = 0, then the pre-step of
 * iteration 0.  x0: device, d floats, caller layout, copied.  Allocates all state and scratch.
 * *out receives the handle.  Host-synchronous.
 */
int sae_init(const sae_config *cfg, const float *x0, sae_handle **out);

/*
 * One iteration t of Algorithm 1 (worker lines, server lines, re-update) followed by the pre-step
 * (error averaging when due) of iteration t+1:
 *   xh = x - e^(k) (SAEF) or x (EF);  m^(k) = mu m^(k) + (g^(k) + lambda xh);  Delta^(k) = e^(k) + lr m^(k);
 *   e^(k) = Delta^(k) - C(Delta^(k));  Delta = e + (1/K) sum_k C(Delta^(k));  e = Delta - C(Delta);
 *   x = x - C(Delta).
 * grads: device, [K][d] floats, caller layout, read-only, must stay valid until the step has run.
 * lr: eta_t > 0.  Enqueues kernels only; allocates no device memory.
 * On a stream other than the default stream the kernels of a step are captured once per distinct
 * (state, grads pointer, lr) into a CUDA graph and later steps with the same key replay it with one
 * graph launch (the host cost of a step drops from one launch per kernel to one launch); if the
 * caller is itself capturing the stream, the kernels simply join that capture.
 * Top-K with the folded tail (8 or 16 workers, no weight decay): part of a step -- the workers' threshold
 * select -- runs on a second stream the handle owns (created by sae_init), forked from the handle's stream
 * after the worker pass and joined to it again before the call returns, so all of a step's work stays
 * ordered on the handle's stream as the caller sees it (inside a capture: two branches of the same graph).
 */
int sae_step(sae_handle *h, const float *grads, float lr);

/*
 * Same step with the gradients in HOST memory (pinned memory gives an asynchronous copy): copies
 * them to a library-owned device staging buffer on the handle's stream, then runs the step.  The
 * staging buffer (K*d floats) is allocated by the first call.
 */
int sae_step_host(sae_handle *h, const float *grads_host, float lr);

/*
 * Local steps (Section 2: Algorithm 1 "can be easily extended to local SGD, where the local model
 * difference will be communicated every several (>1) iterations"; the paper does not spell the extension
 * out, this is the reading built here).  With period H, iteration t communicates iff (t+1) mod H = 0 and is
 * then exactly sae_step above.  On the other iterations only the worker lines run:
 *   xh = x - e^(k);  m^(k) = mu m^(k) + (g^(k) + lambda xh);  e^(k) = e^(k) + lr m^(k)
 * i.e. the model difference stays with the worker and keeps accumulating in the place of its error;
 * nothing is compressed or sent, x and the server error do not change.  sae_get_step_ahead(k) = x - e^(k)
 * is then worker k's local model one step ahead, the point of its next gradient, and
 * SAE_STATE_WORKER_ERROR returns that running difference.  A local iteration is one pass over g, m^(k)
 * and the stored difference (20 bytes per worker-element) and no server pass.
 * period >= 1 (1 = Algorithm 1 as printed).  Only before the first step, in SAE_MODE_SAEF, with
 * avg_period = 0 and not on a shard; otherwise SAE_ERR_INVALID_ARG.  Checkpoints carry the period and
 * load only into a handle set to the same one.
 */
int sae_set_local_steps(sae_handle *h, int32_t period);

/* Algorithm 1, "Output": x_t into out (device, d floats, caller layout). */
int sae_get_params(sae_handle *h, float *out);
/* Same into HOST memory (through a library-owned device buffer allocated by the first call);
 * synchronises the stream before returning. */
int sae_get_params_host(sae_handle *h, float *out_host);

/*
 * The point where worker k must evaluate its next gradient: x_t - e_t^(k) in SAEF mode ("One step
 * ahead"), x_t in EF mode.  out: device, d floats, caller layout.
 */
int sae_get_step_ahead(sae_handle *h, int32_t worker, float *out);

/* State and last-message getters (parity checks, checkpointing). `out` is a DEVICE buffer of at least
 * `bytes` bytes; the call fails with SAE_ERR_INVALID_ARG if that is too small.  Parameter-shaped
 * results are in caller layout. */
#define SAE_STATE_MOMENTUM 0      /* m^(k): d floats                                                    */
#define SAE_STATE_WORKER_ERROR 1  /* e^(k) after the last pre-step: d floats                            */
#define SAE_STATE_SERVER_ERROR 2  /* e: d floats (worker ignored)                                       */
#define SAE_STATE_WORKER_SCALES 3 /* scaled sign: ||Delta^(k)||_1/n_j of the last step, T floats        */
#define SAE_STATE_SERVER_SCALES 4 /* same for the server's Delta, T floats                              */
#define SAE_STATE_WORKER_WORDS 5  /* sign words of C(Delta^(k)) of the last step (format below)         */
#define SAE_STATE_SERVER_WORDS 6  /* sign words of C(Delta) of the last step                            */
#define SAE_STATE_WORKER_TAU 7    /* Top-K: bit pattern of the k_j-th largest |Delta^(k)|, T uint32     */
#define SAE_STATE_SERVER_TAU 8    /* same for the server, T uint32                                      */
#define SAE_STATE_WORKER_MASK 9   /* Top-K: selected set of the last step as bit words (format below)   */
#define SAE_STATE_SERVER_MASK 10  /* same for the server                                                */
#define SAE_STATE_TOPK_FALLBACKS 11 /* Top-K diagnostics, 2 uint32: how many (worker, tensor) pairs and how
                                     many server tensors so far needed the full radix select because the
                                     candidate window around the previous threshold did not hold it    */
int sae_get_state(sae_handle *h, int32_t which, int32_t worker, void *out, size_t bytes);
/*
 * Bit-word format (sign message and Top-K mask): per tensor ceil(n_j/32) little-endian uint32 words,
 * bit i of word w <-> element 32w+i of that tensor; sign: 1 <-> Delta_i >= 0 (code +scale), mask:
 * 1 <-> selected; padding bits 0; the tensors' word arrays concatenated in list order.
 */

/*
 * Checkpoint / resume.  sae_save_state copies everything later steps and getters depend on (x, e, m^(k),
 * the held form of e^(k), last scales / thresholds / messages, t, the last learning rate) into `out`
 * (DEVICE buffer of at least sae_state_bytes(h) bytes; stream-ordered except for a short synchronisation).
 * sae_load_state restores it into a handle created with the SAME configuration (anything else is
 * SAE_ERR_INVALID_ARG); the run then continues bit for bit as the saved one would have.
 */
int64_t sae_state_bytes(sae_handle *h);
int sae_save_state(sae_handle *h, void *out, size_t bytes);
int sae_load_state(sae_handle *h, const void *in, size_t bytes);

/*
 * Gradient-mismatch bounds of Section 3 (Fig. 3, right; the factors L^2 and the sigma^2 term are left out),
 * for the current errors, with ebar = (1/K) sum_k e^(k):
 *   out_host[0] = || e + ebar ||^2                         -- local error feedback
 *   out_host[1] = (1/K) sum_k || e + ebar - e^(k) ||^2      -- step ahead
 * accumulated in fp64 on the device.  out_host: HOST, 2 doubles.  Synchronises the stream.
 */
int sae_get_mismatch(sae_handle *h, double *out_host);

/* Number of iterations performed so far (t). */
int64_t sae_iteration(const sae_handle *h);
/* d = sum n_j, and the number of bit words per worker, sum_j ceil(n_j/32). */
int64_t sae_num_params(const sae_handle *h);
int64_t sae_num_words(const sae_handle *h);

/* Waits for the stream; returns and clears the sticky device status (SAE_OK or SAE_ERR_RANGE...).
 *
 * SAE_ERR_TIMEOUT: the worker and server passes move tiles into shared memory with asynchronous bulk copies
 * and wait for them on shared-memory barriers.  Every such wait is bounded in time: a warp that has polled
 * for longer than the handle's limit raises the status and the kernel returns (after the copying warp has
 * waited, under the same limit, for the copies it still had in flight) -- it never traps and never spins
 * without a bound.  The limit is one second unless the environment variable SAE_WAIT_LIMIT_US (microseconds,
 * 1 .. 60 000 000, read by sae_init) sets another; a kernel in which a copy was lost therefore ends within
 * about twice the limit.  After SAE_ERR_TIMEOUT the handle's state is that of a half-finished step: destroy it
 * (or restore a checkpoint); the CUDA context and other handles are unaffected. */
int sae_sync(sae_handle *h);

/*
 * Per-kernel timing.  With profiling enabled every kernel launch of sae_step is bracketed by CUDA
 * events on the handle's stream.  sae_get_kernel_times synchronises, then writes for each of the
 * SAE_NUM_KERNELS kernel slots the accumulated milliseconds and launch count since the last reset
 * and resets them.  Slot names: sae_kernel_name(slot).
 */
#define SAE_NUM_KERNELS 12
int sae_set_profiling(sae_handle *h, int32_t enabled);
int sae_get_kernel_times(sae_handle *h, float *ms_host, int64_t *launches_host);
const char *sae_kernel_name(int32_t slot);
/* Total kernels launched by this handle so far. */
int64_t sae_kernel_launches(const sae_handle *h);

/*
 * Sharded operation: the K workers of Algorithm 1 spread over several handles ("shards": one per GPU /
 * process), scaled-sign or Top-K compressor.  A shard owns workers worker_begin .. worker_begin+num_local_workers-1:
 * their momentum, error and message rows live in its memory.  The server lines ("Server: receive ...,
 * send C(Delta)") are replicated: every shard keeps x and the server error e and computes the same bits,
 * because it reads all K messages (1 scale per tensor + 1 bit per element per worker, Eq. 2) in k order.
 * The exchange of Algorithm 1 ("send C(Delta^(k)) to the server") is not a separate copy: the server pass
 * reads every worker's sign words and scales in place from the owner's memory through a table of row
 * pointers -- plain loads, over NVLink when the owner is another GPU -- so gather and aggregation are one
 * kernel.  Error averaging (pre-step, every p iterations) likewise reads the owners' stored model
 * differences in place.
 *
 *   sae_init_shard    cfg->num_workers is K of the whole job; otherwise as sae_init (the identity compressor
 *                     is not sharded).  Worker indices of the getters are LOCAL (0 .. num_local-1).
 *                     Top-K: a worker's message is the list of its selected (index, value) entries (Section
 *                     3.1), compacted by its owner once the thresholds are known; every shard adds all K lists
 *                     in k order, reading them in place (an unselected entry contributes an exact zero, so the
 *                     ordered sum over the selecting workers is the full ordered sum).
 *   sae_shard_export  writes SAE_SHARD_BLOB_BYTES bytes (HOST) describing where this shard's rows live: raw
 *                     pointers for handles of the same process, CUDA IPC handles for other processes.
 *   sae_shard_attach  makes the rows of one exported blob (any shard's, including this handle's own) known
 *                     to this handle.  Every handle must attach the blobs of all shards before stepping.
 *                     Buffers of another process are mapped with cudaIpcOpenMemHandle (peer access enabled
 *                     lazily) and unmapped by sae_shard_detach or sae_destroy.  Rows of the same process on
 *                     ANOTHER device are taken by their raw pointers after peer access from this handle's
 *                     device to theirs has been switched on here (cudaDeviceEnablePeerAccess; already on counts
 *                     as success); if the two devices cannot reach each other the blob is refused with
 *                     SAE_ERR_INVALID_ARG and nothing is attached, so no kernel ever reads an unmapped row.
 *   sae_shard_detach  forgets every attached row and unmaps other processes' buffers (waits for the stream
 *                     first).  An owner must not be destroyed while another process still maps its rows:
 *                     detach everywhere, synchronise the ranks, then destroy.
 *   sae_step_begin    worker lines of iteration t for the local workers: grads_local is [num_local][d].
 *   sae_step_end      server lines, re-update and the pre-step of iteration t+1.
 *
 * Error averaging by all-reduce (the communication the paper names for it, Section 3.2: "ring all-reduce").
 * sae_shard_set_avg_mode(h, 1) replaces the in-place pull of all K x d stored differences by a sum the
 * caller all-reduces: when sae_avg_due(h) is 1 after sae_step_end, call sae_avg_local_sum(h, buf) (buf:
 * device, sae_num_padded(h) floats; receives sum_k e^(k) over this shard's workers, k in order, in the
 * library's padded layout), all-reduce buf over the shards with SUM, then sae_avg_set(h, buf) on every
 * shard (ebar = buf / K).  This moves 2 d floats per shard instead of K d, but the order of the all-reduce's
 * additions is the library's, not k = 0..K-1: the averaged error then agrees with Algorithm 1 to fp32
 * rounding, not bit for bit (with one shard it is exact).  sae_step_begin is refused while the sum is owed.
 *
 * Errors: SAE_ERR_INVALID_ARG for a null pointer, the identity compressor, a worker range outside
 * 0..K-1, a blob that is too short / foreign / describes another parameter list / names rows that are already
 * attached, sae_step_begin before every worker's rows are attached or while a step is open, sae_step_end
 * without an open step, sae_shard_attach / sae_shard_detach / checkpoint calls while a step is open;
 * SAE_ERR_CUDA when mapping a peer's buffer fails (sae_last_cuda_error has the code).  Device-detected
 * errors (RANGE, TIMEOUT) are sticky and reported by sae_sync, as for sae_step.
 *
 * Ordering is the caller's duty (a host barrier after synchronising the streams, or a collective that is
 * stream-ordered on every shard): every shard's sae_step_begin work must be complete before any shard's
 * sae_step_end work starts (the messages are read remotely), and every shard's sae_step_end work before
 * any shard's next sae_step_begin (which overwrites them).  Shards of one process on one stream need
 * nothing: stream order already gives both.  sae_step and sae_step_host refuse a sharded handle.
 */
#define SAE_SHARD_BLOB_BYTES 1024
int sae_init_shard(const sae_config *cfg, int32_t worker_begin, int32_t num_local_workers, const float *x0,
                   sae_handle **out);
int sae_shard_export(sae_handle *h, void *blob_host, size_t bytes);
int sae_shard_attach(sae_handle *h, const void *blob_host, size_t bytes);
int sae_shard_detach(sae_handle *h);
int sae_step_begin(sae_handle *h, const float *grads_local, float lr);
int sae_step_end(sae_handle *h);
int sae_shard_set_avg_mode(sae_handle *h, int32_t external_sum);
int sae_avg_due(const sae_handle *h);
int64_t sae_num_padded(const sae_handle *h);
int sae_avg_local_sum(sae_handle *h, float *sum_padded);
int sae_avg_set(sae_handle *h, const float *sum_padded);

/* Frees everything the handle owns (synchronises first). NULL is allowed. */
void sae_destroy(sae_handle *h);

const char *sae_strerror(int status);
/* cudaError_t of the most recent failed CUDA call made on behalf of this handle (0 if none);
 * with h == NULL, of the most recent failed sae_init. */
int sae_last_cuda_error(const sae_handle *h);

/*
 * (The paper has no counterpart for this entry point; it exists for a class of callers, not for a
 * step of Algorithm 1.)
 *
 * The scaled-sign compressor of ONE tensor without any allocation, for callers that cannot call
 * cudaMalloc: code running inside another framework's memory pool or under a fixed device-memory
 * budget, plug-ins that are handed only their input and output buffers, and latency-critical loops in
 * which an allocation (which may synchronise the whole device) is not acceptable.  Every other entry
 * point of this library works on a handle whose state and scratch sae_init allocates.
 *
 * Computes C(v) of Eq. 2 for v[0..n): the exact L1 scale (same definition and same bits as the
 * worker pass: sum of floor(|v_i| 2^64) as an integer, truncated to 53 bits, divided by n) into
 * *scale, and the sign words (bit i of word w <-> v[32w+i] >= 0, padding bits 0) into
 * words[0..ceil(n/32)).  range_flag (may be NULL) receives 1 if some |v_i| was non-finite or >= 2^32,
 * else 0.  v, words, scale, range_flag: DEVICE pointers owned by the caller; the work is enqueued on
 * `stream` (cudaStream_t, NULL = default stream) of the CURRENT device and is asynchronous.
 *
 * The per-tile partial sums live in a fixed array inside the library image (128 KiB + 256 B of
 * device memory on every GPU that loads the library, held until the process exits), so:
 *  - n must not exceed sae_noalloc_max_elements() = 33 554 432; larger inputs are rejected with
 *    SAE_ERR_TOO_LARGE and nothing is launched (n < 1 or a NULL pointer: SAE_ERR_INVALID_ARG);
 *  - the first call on each device looks up the array's device address (no allocation); make that
 *    first call before starting any stream capture;
 *  - all calls share the one array: two calls whose kernels may overlap on the GPU (different
 *    streams, or different host threads) race on it -- serialise them.  The array keeps the previous
 *    call's contents; the call itself clears the counter and flag it relies on.
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 */
int sae_sign_compress_noalloc(const float *v, int64_t n, uint32_t *words, float *scale, int32_t *range_flag,
                              void *stream);
int64_t sae_noalloc_max_elements(void);

#ifdef __cplusplus
}
#endif
#endif /* SAE_H_ */
