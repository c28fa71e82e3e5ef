// CPU oracle for one iteration of "Distributed Momentum SGD with Double-Way Compression"
// (Algorithm 1 of the Step-Ahead Error Feedback paper), with the scaled-sign compressor (Eq. 2),
// the Top-K sparsifier (Section 3.1, "How related to compression?") and the identity compressor.
//
// THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, sequential restatement of the algorithm in the
// paper's order and notation, used only by the tests, by the smoke check and by the benchmark's
// CPU-baseline leg.  It shares no code with the CUDA library and the product never calls it.
//
// Two instantiations:
//   * float  -- the arithmetic the CUDA path computes in; every operation is pinned:
//               fma(a,b,c) is one fused, correctly rounded operation, everything else is a single
//               separately rounded IEEE operation (build with -ffp-contract=off).  The scaled-sign
//               scale is defined through an exact integer sum (see l1_fixed below) so that it does
//               not depend on summation order.
//   * double -- the same steps in fp64 with a plain sequential L1 sum; used to check the paper's
//               identities (Eq. 3 / Appendix A) to ~1e-12.
//
// Readings of the paper that nothing in it can confirm ("parity unpinned" for the sign(0) and Top-K
// conventions, they are fixed here and in the CUDA path alike):
//   * sign(0): the 1-bit code has no zero, so v >= 0 maps to +scale (hence +-0 -> +scale);
//   * weight decay: coupled L2, lambda * (point where the gradient is evaluated) added to the gradient
//     (a reading; the arithmetic itself is pinned to a library SGD optimiser with weight decay);
//   * Top-K: k = max(1, floor(n*num/den)); every entry whose magnitude ties the k-th largest is kept,
//     exact zeros are never selected.
//   * local steps (Section 2 names the extension to local SGD, where a worker sends its model difference only
//     once in several iterations, without spelling it out): with period H, iteration t communicates iff
//     (t+1) mod H = 0; on the other iterations a worker only does its own lines, and its model difference
//     keeps accumulating in the place of its error: e^(k) <- Delta^(k) = e^(k) + eta m^(k), nothing is sent,
//     x and the server error stay.  The gradient point x - e^(k) of the step-ahead branch is then the
//     worker's local model one step ahead.  Step-ahead branch without error averaging only.
//
// Threads: `threads` > 1 only distributes independent units (whole (worker, tensor) pairs for the
// compressor, single elements for the elementwise loops); each unit is still computed sequentially,
// so results are bit-identical for any thread count.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>
#include <functional>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef unsigned __int128 u128;

namespace {

enum { C_IDENTITY = 0, C_SIGN = 1, C_TOPK = 2 };
enum { MODE_EF = 0, MODE_SAEF = 1 };

inline float  fma_r(float a, float b, float c)    { return std::fmaf(a, b, c); }
inline double fma_r(double a, double b, double c) { return std::fma(a, b, c); }

// ---- Eq. 2, float: exact L1 --------------------------------------------------------------------
// S = sum_i floor(|v_i| * 2^64) as an exact unsigned 128-bit integer.  |v| = M * 2^(ex-24) with M a
// 24-bit integer (frexp), so |v| * 2^64 = M * 2^(ex+40): a shift of M.  Entries that are not finite
// or have |v| >= 2^32 are outside the representable range and raise `range`.
inline u128 floor_fixed64(float a) {   // a finite, 0 <= a < 2^32
  if (a == 0.0f) return 0;
  int ex;
  float f = std::frexp(a, &ex);               // a = f * 2^ex, f in [0.5, 1)
  uint32_t M = (uint32_t)std::ldexp(f, 24);   // exact: f has at most 24 significant bits
  int sh = ex + 40;
  if (sh >= 0) return (u128)M << sh;
  if (sh <= -32) return 0;
  return (u128)(M >> (-sh));
}

inline u128 l1_fixed(const float* v, int64_t n, bool* range) {
  u128 S = 0;
  for (int64_t i = 0; i < n; ++i) {
    float a = std::fabs(v[i]);
    if (!(a < 4294967296.0f)) { *range = true; continue; }
    S += floor_fixed64(a);
  }
  return S;
}

// scale = ||v||_1 / n (Eq. 2): the exact sum truncated to its top 53 bits (so that it is a double
// without rounding), one double division, an exact scaling by 2^-64, one rounding to float.
inline float scale_from_fixed(u128 S, int64_t n) {
  if (S == 0) return 0.0f;
  int p = 127;
  while (!((S >> p) & 1)) --p;
  if (p > 52) { int sh = p - 52; S = (S >> sh) << sh; }
  double Dd = (double)S;
  return (float)((Dd / (double)n) * 0x1p-64);
}

inline float sign_scale(const float* v, int64_t n, bool* range) {
  return scale_from_fixed(l1_fixed(v, n, range), n);
}
inline double sign_scale(const double* v, int64_t n, bool* range) {
  long double S = 0;
  for (int64_t i = 0; i < n; ++i) { if (!std::isfinite(v[i])) *range = true; S += std::fabs((long double)v[i]); }
  return (double)(S / (long double)n);
}

// ---- Top-K keys: the bit pattern of |v| orders finite magnitudes ---------------------------------
inline uint64_t mag_key(float v)  { uint32_t b; std::memcpy(&b, &v, 4); return b & 0x7fffffffu; }
inline uint64_t mag_key(double v) { uint64_t b; std::memcpy(&b, &v, 8); return b & 0x7fffffffffffffffull; }

inline int64_t topk_count(int64_t n, uint32_t num, uint32_t den) {
  int64_t kk = (int64_t)(((u128)n * num) / den);
  if (kk < 1) kk = 1;
  if (kk > n) kk = n;
  return kk;
}

template <class R>
uint64_t topk_threshold(const R* v, int64_t n, int64_t kk) {
  std::vector<uint64_t> keys(n);
  for (int64_t i = 0; i < n; ++i) keys[i] = mag_key(v[i]);
  std::nth_element(keys.begin(), keys.begin() + (kk - 1), keys.end(), std::greater<uint64_t>());
  return keys[kk - 1];
}

// ---- the compressor C(.) applied to one tensor ----------------------------------------------------
template <class R>
void compress(int compressor, const R* v, int64_t n, uint32_t num, uint32_t den, R* c, R* scale_out,
              uint64_t* tau_out, bool* range) {
  if (compressor == C_IDENTITY) {
    for (int64_t i = 0; i < n; ++i) c[i] = v[i];
  } else if (compressor == C_SIGN) {
    R s = sign_scale(v, n, range);
    *scale_out = s;
    for (int64_t i = 0; i < n; ++i) c[i] = (v[i] >= (R)0) ? s : -s;
  } else {
    uint64_t tau = topk_threshold(v, n, topk_count(n, num, den));
    *tau_out = tau;
    for (int64_t i = 0; i < n; ++i) {
      uint64_t key = mag_key(v[i]);
      c[i] = (key >= tau && key != 0) ? v[i] : (R)0;
    }
  }
}

template <class R>
struct Oracle {
  int K, T, compressor, server_compress, mode, avg_period, threads;
  int local_steps = 1;                      // H: communicate when (t+1) mod H == 0
  R mu, lambda;
  uint32_t num, den;
  std::vector<int64_t> n, off;
  int64_t d;
  int64_t t;
  bool range;
  std::vector<R> x, e_srv, Ds, cs;          // [d]
  std::vector<R> m, e, D, c;                // [K][d]
  std::vector<R> scale, scale_srv;          // [K][T], [T]
  std::vector<uint64_t> tau, tau_srv;       // [K][T], [T]

  // Algorithm 1, "Average local error" (inside the SAEF branch; honoured in EF mode too when asked).
  void pre_step() {
    if (avg_period > 0 && (t + 1) % avg_period == 0) {
      #pragma omp parallel for num_threads(threads)
      for (int64_t i = 0; i < d; ++i) {
        R acc = 0;
        for (int k = 0; k < K; ++k) acc = acc + e[(int64_t)k * d + i];
        R eb = acc / (R)K;
        for (int k = 0; k < K; ++k) e[(int64_t)k * d + i] = eb;
      }
    }
  }

  void step(const R* g, R eta) {
    // Worker-k: step-ahead point, local momentum, local model difference.
    #pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
    for (int k = 0; k < K; ++k) {
      for (int64_t i = 0; i < d; ++i) {
        int64_t q = (int64_t)k * d + i;
        R xh = (mode == MODE_SAEF) ? x[i] - e[q] : x[i];              // x_{t+1/2} = x_t - e_t  |  x_t
        R ge = (lambda != (R)0) ? fma_r(lambda, xh, g[q]) : g[q];     // gradient at xh (+ coupled L2)
        m[q] = fma_r(mu, m[q], ge);                                    // m_{t+1} = mu m_t + grad
        D[q] = fma_r(eta, m[q], e[q]);                                 // Delta = e_t + eta m_{t+1}
      }
    }
    if (local_steps > 1 && (t + 1) % local_steps != 0) {
      // not a communication iteration: the model difference stays with the worker and keeps growing
      e = D;
      t = t + 1;
      return;
    }
    // c^(k) = C(Delta^(k)) per tensor;  e^(k)_{t+1} = Delta^(k) - C(Delta^(k)).
    #pragma omp parallel for collapse(2) num_threads(threads) schedule(dynamic, 1)
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < T; ++j) {
        int64_t q = (int64_t)k * d + off[j];
        bool rg = false;
        compress<R>(compressor, &D[q], n[j], num, den, &c[q], &scale[(int64_t)k * T + j],
                    &tau[(int64_t)k * T + j], &rg);
        if (rg) {
          #pragma omp atomic write
          range = true;
        }
        for (int64_t i = 0; i < n[j]; ++i) e[q + i] = D[q + i] - c[q + i];
      }
    // Server: Delta = e + (1/K) sum_k C(Delta^(k)), k in order.
    #pragma omp parallel for num_threads(threads)
    for (int64_t i = 0; i < d; ++i) {
      R acc = 0;
      for (int k = 0; k < K; ++k) acc = acc + c[(int64_t)k * d + i];
      Ds[i] = e_srv[i] + acc / (R)K;
    }
    // Server compressor (double-way) or identity (single-way), per tensor.
    #pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
    for (int j = 0; j < T; ++j) {
      bool rg = false;
      compress<R>(server_compress ? compressor : C_IDENTITY, &Ds[off[j]], n[j], num, den, &cs[off[j]],
                  &scale_srv[j], &tau_srv[j], &rg);
      if (rg) {
        #pragma omp atomic write
        range = true;
      }
    }
    // e_{t+1} = Delta - C(Delta);  re-update x_{t+1} = x_t - C(Delta).
    #pragma omp parallel for num_threads(threads)
    for (int64_t i = 0; i < d; ++i) {
      e_srv[i] = Ds[i] - cs[i];
      x[i] = x[i] - cs[i];
    }
    t = t + 1;
    pre_step();
  }
};

template <class R>
Oracle<R>* create(int K, int T, const int64_t* sizes, int compressor, int server_compress, int mode,
                  int avg_period, double mu, double lambda, uint32_t num, uint32_t den, int threads,
                  const R* x0) {
  if (K < 1 || T < 1 || !sizes || compressor < 0 || compressor > 2 || avg_period < 0) return nullptr;
  if (compressor == C_TOPK && (den == 0 || num > den)) return nullptr;
  Oracle<R>* o = new Oracle<R>();
  o->K = K; o->T = T; o->compressor = compressor; o->server_compress = server_compress;
  o->mode = mode; o->avg_period = avg_period; o->threads = threads < 1 ? 1 : threads;
  o->mu = (R)mu; o->lambda = (R)lambda; o->num = num; o->den = den;
  o->n.assign(sizes, sizes + T);
  o->off.resize(T);
  int64_t d = 0;
  for (int j = 0; j < T; ++j) { if (sizes[j] < 1) { delete o; return nullptr; } o->off[j] = d; d += sizes[j]; }
  o->d = d; o->t = 0; o->range = false;
  o->x.assign(x0, x0 + d);
  o->e_srv.assign(d, 0); o->Ds.assign(d, 0); o->cs.assign(d, 0);
  o->m.assign((size_t)K * d, 0); o->e.assign((size_t)K * d, 0);
  o->D.assign((size_t)K * d, 0); o->c.assign((size_t)K * d, 0);
  o->scale.assign((size_t)K * T, 0); o->scale_srv.assign(T, 0);
  o->tau.assign((size_t)K * T, 0); o->tau_srv.assign(T, 0);
  o->pre_step();                               // pre-step of iteration 0
  return o;
}

// which: 0 x | 1 server error | 2 momentum[k] | 3 worker error[k] | 4 Delta[k] (last) | 5 C(Delta[k]) (last)
//        6 server Delta (last) | 7 C(server Delta) (last) | 8 worker scales[k] [T] | 9 server scales [T]
template <class R>
int get_real(Oracle<R>* o, int which, int k, R* out) {
  int64_t d = o->d;
  if (which >= 2 && which <= 5 && (k < 0 || k >= o->K)) return -1;
  if (which == 8 && (k < 0 || k >= o->K)) return -1;
  const R* src = nullptr; int64_t cnt = d;
  switch (which) {
    case 0: src = o->x.data(); break;
    case 1: src = o->e_srv.data(); break;
    case 2: src = &o->m[(int64_t)k * d]; break;
    case 3: src = &o->e[(int64_t)k * d]; break;
    case 4: src = &o->D[(int64_t)k * d]; break;
    case 5: src = &o->c[(int64_t)k * d]; break;
    case 6: src = o->Ds.data(); break;
    case 7: src = o->cs.data(); break;
    case 8: src = &o->scale[(int64_t)k * o->T]; cnt = o->T; break;
    case 9: src = o->scale_srv.data(); cnt = o->T; break;
    default: return -1;
  }
  std::memcpy(out, src, sizeof(R) * cnt);
  return 0;
}

}  // namespace

extern "C" {

#define SAO_API(SUF, R)                                                                              \
  void* sao_create_##SUF(int K, int T, const int64_t* sizes, int compressor, int server_compress,    \
                         int mode, int avg_period, double mu, double lambda, uint32_t num,           \
                         uint32_t den, int threads, const R* x0) {                                   \
    return create<R>(K, T, sizes, compressor, server_compress, mode, avg_period, mu, lambda, num,    \
                     den, threads, x0);                                                              \
  }                                                                                                  \
  void sao_destroy_##SUF(void* h) { delete (Oracle<R>*)h; }                                          \
  void sao_step_##SUF(void* h, const R* g, double eta) { ((Oracle<R>*)h)->step(g, (R)eta); }         \
  int sao_get_##SUF(void* h, int which, int k, R* out) { return get_real<R>((Oracle<R>*)h, which, k, out); } \
  int64_t sao_iteration_##SUF(void* h) { return ((Oracle<R>*)h)->t; }                                \
  /* local-step period H >= 1; only before the first step, step-ahead branch, no error averaging */   \
  int sao_set_local_steps_##SUF(void* h, int H) {                                                    \
    Oracle<R>* o = (Oracle<R>*)h;                                                                    \
    if (H < 1 || o->t != 0 || (H > 1 && (o->mode != MODE_SAEF || o->avg_period != 0))) return -1;    \
    o->local_steps = H;                                                                              \
    return 0;                                                                                        \
  }                                                                                                  \
  int sao_range_flag_##SUF(void* h) { return ((Oracle<R>*)h)->range ? 1 : 0; }                       \
  /* Top-K thresholds (keys) of the last step: k >= 0 worker k, k < 0 server; T entries. */          \
  void sao_get_tau_##SUF(void* h, int k, uint64_t* out) {                                            \
    Oracle<R>* o = (Oracle<R>*)h;                                                                    \
    const uint64_t* s = k < 0 ? o->tau_srv.data() : &o->tau[(int64_t)k * o->T];                      \
    std::memcpy(out, s, 8 * (size_t)o->T);                                                           \
  }                                                                                                  \
  /* the compressor alone, on one tensor */                                                          \
  int sao_compress_##SUF(int compressor, const R* v, int64_t n, uint32_t num, uint32_t den, R* c,    \
                         R* scale, uint64_t* tau) {                                                  \
    bool rg = false; R s = 0; uint64_t ta = 0;                                                       \
    compress<R>(compressor, v, n, num, den, c, &s, &ta, &rg);                                        \
    if (scale) *scale = s;                                                                           \
    if (tau) *tau = ta;                                                                              \
    return rg ? 1 : 0;                                                                               \
  }

SAO_API(f32, float)
SAO_API(f64, double)

// exact fixed-point L1 of a float vector: out[0] = low 64 bits, out[1] = high 64 bits. Returns the range flag.
int sao_l1_fixed_f32(const float* v, int64_t n, uint64_t* out) {
  bool rg = false;
  u128 S = l1_fixed(v, n, &rg);
  out[0] = (uint64_t)S; out[1] = (uint64_t)(S >> 64);
  return rg ? 1 : 0;
}

float sao_scale_from_fixed_f32(uint64_t lo, uint64_t hi, int64_t n) {
  return scale_from_fixed(((u128)hi << 64) | lo, n);
}

int64_t sao_topk_count(int64_t n, uint32_t num, uint32_t den) { return topk_count(n, num, den); }

// Sign message format: per tensor ceil(n_j/32) little-endian 32-bit words, bit i of word w <-> element
// 32w+i, 1 <-> v >= 0 (the +scale code), padding bits 0; tensors concatenated in list order.
int64_t sao_pack_signs_f32(const float* v, int T, const int64_t* sizes, uint32_t* words) {
  int64_t w0 = 0, q = 0;
  for (int j = 0; j < T; ++j) {
    int64_t nw = (sizes[j] + 31) / 32;
    for (int64_t w = 0; w < nw; ++w) words[w0 + w] = 0;
    for (int64_t i = 0; i < sizes[j]; ++i)
      if (v[q + i] >= 0.0f) words[w0 + i / 32] |= (1u << (i % 32));
    w0 += nw; q += sizes[j];
  }
  return w0;
}

int sao_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
