// Scalify oracle: TEST INFRASTRUCTURE, not product code.
//
// A plain, slow, obviously-correct CPU statement of the scaled operations of
// "Scalify: scale propagation for efficient low-precision LLM training"
// (arxiv 2407.17353).  Everything is computed in fp64 from the bit patterns
// of the operands; nothing here is shared with, or derived from, the CUDA
// library.  Only tests, the smoke check and the CPU-baseline leg of the
// benchmark may call it.
//
// Conventions
//   * A ScaledArray is (data, scale) with value = data * scale (Section 2).
//   * Scales are powers of two kept in fp32 (Section 2, E8M0 simulated in
//     float32) and every propagated scale is rounded DOWN to a power of two
//     (Section 3.2, last paragraph).
//   * Data bit patterns: OCP FP8 E4M3 (finite-only, max 448, NaN 0x7F),
//     OCP FP8 E5M2 (IEEE-like, max 57344), IEEE binary16, bfloat16, binary32.
//   * Encoding is round-to-nearest-even straight from the fp64 value to the
//     target format; FP8 overflow saturates to the largest finite value,
//     FP16/BF16/FP32 overflow gives infinity; subnormals are kept.
//
// dtype codes used on this C interface: 0 E4M3, 1 E5M2, 2 F16, 3 BF16, 4 F32.
// statistic codes: 0 none, 1 AMAX, 2 L2 (root mean square).
//
// Parity pins: every function below is pinned by tests/test_oracle_*.py
// (exhaustive codec round trips, comparison of the codecs with an independent
// library cast, brute force on tiny matrices, closed forms, invariants,
// finite differences, textbook Adam / LayerNorm; tests/test_oracle_support_ops.py pins
// the embedding / softmax / cross-entropy readings against torch in fp64;
// tests/test_oracle_mx.py pins the block-scale functions).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <cstdlib>
#include <vector>
#include <limits>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { E4M3 = 0, E5M2 = 1, F16 = 2, BF16 = 3, F32 = 4 };
enum { STAT_NONE = 0, STAT_AMAX = 1, STAT_L2 = 2 };

struct Fmt {
  int ebits;      // exponent field width
  int mbits;      // mantissa field width
  int bias;       // exponent bias
  bool ieee_top;  // true: all-ones exponent is inf/NaN; false (E4M3): only S.1111.111 is NaN
  bool saturate;  // overflow -> max finite instead of inf
};

const Fmt kFmt[4] = {
    {4, 3, 7, false, true},    // E4M3 (finite-only)
    {5, 2, 15, true, true},    // E5M2
    {5, 10, 15, true, false},  // F16
    {8, 7, 127, true, false},  // BF16
};

uint32_t load_bits(const void* p, int dtype, int64_t i) {
  if (dtype <= E5M2) return static_cast<const uint8_t*>(p)[i];
  if (dtype == F32) return static_cast<const uint32_t*>(p)[i];
  return static_cast<const uint16_t*>(p)[i];
}

void store_bits(void* p, int dtype, int64_t i, uint32_t b) {
  if (dtype <= E5M2) static_cast<uint8_t*>(p)[i] = static_cast<uint8_t>(b);
  else if (dtype == F32) static_cast<uint32_t*>(p)[i] = b;
  else static_cast<uint16_t*>(p)[i] = static_cast<uint16_t>(b);
}

// value of a bit pattern (Section 2: the data component is an ordinary float)
double decode(uint32_t bits, int dtype) {
  if (dtype == F32) {
    float f;
    std::memcpy(&f, &bits, 4);
    return static_cast<double>(f);
  }
  const Fmt& f = kFmt[dtype];
  const int total = 1 + f.ebits + f.mbits;
  const uint32_t sign = (bits >> (total - 1)) & 1u;
  const uint32_t e = (bits >> f.mbits) & ((1u << f.ebits) - 1u);
  const uint32_t m = bits & ((1u << f.mbits) - 1u);
  const uint32_t e_all = (1u << f.ebits) - 1u;
  const uint32_t m_all = (1u << f.mbits) - 1u;
  double v;
  if (f.ieee_top && e == e_all) {
    v = (m == 0) ? std::numeric_limits<double>::infinity()
                 : std::numeric_limits<double>::quiet_NaN();
  } else if (!f.ieee_top && e == e_all && m == m_all) {
    v = std::numeric_limits<double>::quiet_NaN();
  } else if (e == 0) {
    v = std::ldexp(static_cast<double>(m), 1 - f.bias - f.mbits);  // subnormal
  } else {
    v = std::ldexp(static_cast<double>((1u << f.mbits) + m), static_cast<int>(e) - f.bias - f.mbits);
  }
  return sign ? -v : v;
}

double max_finite(int dtype) {
  const Fmt& f = kFmt[dtype];
  const uint32_t e_all = (1u << f.ebits) - 1u;
  if (f.ieee_top) {
    // exponent field e_all-1, mantissa all ones
    return std::ldexp(static_cast<double>((2u << f.mbits) - 1u), static_cast<int>(e_all) - 1 - f.bias - f.mbits);
  }
  // E4M3: exponent field all ones, mantissa all ones minus one
  return std::ldexp(static_cast<double>((2u << f.mbits) - 2u), static_cast<int>(e_all) - f.bias - f.mbits);
}

// round-to-nearest-even encode of an fp64 value
uint32_t encode(double v, int dtype) {
  if (dtype == F32) {
    float f = static_cast<float>(v);  // IEEE double->float conversion, round to nearest even
    uint32_t b;
    std::memcpy(&b, &f, 4);
    if (std::isnan(v)) b = 0x7FC00000u;
    return b;
  }
  const Fmt& f = kFmt[dtype];
  const int total = 1 + f.ebits + f.mbits;
  const uint32_t e_all = (1u << f.ebits) - 1u;
  const uint32_t m_all = (1u << f.mbits) - 1u;
  if (std::isnan(v)) {
    if (!f.ieee_top) return (e_all << f.mbits) | m_all;              // 0x7F
    if (dtype == E5M2) return (e_all << f.mbits) | m_all;            // 0x7F
    return (e_all << f.mbits) | (1u << (f.mbits - 1));               // quiet NaN
  }
  const uint32_t sign = std::signbit(v) ? 1u : 0u;
  double a = std::fabs(v);
  const double amax = max_finite(dtype);
  uint32_t mag;  // magnitude bits
  auto bits_of_finite = [&](double x) -> uint32_t {
    // x is exactly representable, 0 <= x <= amax
    if (x == 0.0) return 0u;
    int ex;
    std::frexp(x, &ex);
    int e = ex - 1;                       // x in [2^e, 2^(e+1))
    const int emin = 1 - f.bias;          // smallest normal exponent
    if (e < emin) {
      double q = std::ldexp(1.0, emin - f.mbits);
      return static_cast<uint32_t>(x / q);  // exponent field 0
    }
    double q = std::ldexp(1.0, e - f.mbits);
    uint32_t sig = static_cast<uint32_t>(x / q);  // in [2^mbits, 2^(mbits+1))
    return (static_cast<uint32_t>(e - emin + 1) << f.mbits) | (sig - (1u << f.mbits));
  };
  if (std::isinf(a)) {
    mag = f.saturate ? bits_of_finite(amax) : (e_all << f.mbits);
  } else if (a == 0.0) {
    mag = 0u;
  } else {
    int ex;
    std::frexp(a, &ex);
    int e = ex - 1;
    const int emin = 1 - f.bias;
    if (e < emin) e = emin;               // subnormal range shares the quantum of the lowest binade
    const int qexp = e - f.mbits;         // quantum = 2^qexp
    double n = std::ldexp(a, -qexp);      // exact unless a is far below the quantum (then n < 1/2 anyway)
    double r = std::nearbyint(n);         // default rounding mode: to nearest, ties to even
    double rounded = std::ldexp(r, qexp);
    if (rounded > amax) {
      mag = f.saturate ? bits_of_finite(amax) : (e_all << f.mbits);
    } else {
      mag = bits_of_finite(rounded);
    }
  }
  return (sign << (total - 1)) | mag;
}

// largest power of two <= x, x finite and > 0 (Section 3.2: scales are rounded down)
double p2f(double x) {
  int ex;
  std::frexp(x, &ex);
  return std::ldexp(1.0, ex - 1);
}

bool usable_stat(double s) {
  // a statistic that is zero, non-finite or below the smallest normal fp32
  // cannot define a scale: leave the array as it is (reading: rescale by 1)
  return std::isfinite(s) && s >= std::ldexp(1.0, -126);
}

// static factor of a contraction over K independent unit-variance products:
// sqrt(K) rounded down to a power of two = 2^(floor(log2 K) div 2)
double kf(int64_t K) {
  if (K < 1) return 1.0;
  int l = 0;
  while ((int64_t(1) << (l + 1)) <= K) ++l;
  return std::ldexp(1.0, l / 2);
}

double statistic(const std::vector<double>& x, int stat) {
  const int64_t n = static_cast<int64_t>(x.size());
  if (stat == STAT_AMAX) {
    double m = 0.0;
    bool nan = false;
    for (int64_t i = 0; i < n; ++i) {
      if (std::isnan(x[i])) nan = true;
      else if (std::fabs(x[i]) > m) m = std::fabs(x[i]);
    }
    return nan ? std::numeric_limits<double>::quiet_NaN() : m;
  }
  if (stat == STAT_L2) {
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += x[i] * x[i];
    return n > 0 ? std::sqrt(s / static_cast<double>(n)) : 0.0;
  }
  return 0.0;
}

double gelu_gate(double x, int exact_erf) {
  // f(x) = x * g(x).  Both gates are written in the form that keeps relative accuracy where the
  // gate is tiny (x << 0): 0.5*(1+erf(x/sqrt2)) = 0.5*erfc(-x/sqrt2) (exact Gaussian CDF) and
  // 0.5*(1+tanh(u)) = 1/(1+exp(-2u)) (GPT-2's tanh form); the left-hand forms cancel to 0 there.
  if (exact_erf) return 0.5 * std::erfc(-x / std::sqrt(2.0));
  const double c = std::sqrt(2.0 / M_PI);
  const double u = c * (x + 0.044715 * x * x * x);
  return 1.0 / (1.0 + std::exp(-2.0 * u));
}

double gelu_gate_deriv(double x, int exact_erf) {
  if (exact_erf) return std::exp(-0.5 * x * x) / std::sqrt(2.0 * M_PI);
  const double c = std::sqrt(2.0 / M_PI);
  const double g = gelu_gate(x, 0);
  // d/dx sigma(2u) = 2*sigma*(1-sigma)*u'
  return 2.0 * g * (1.0 - g) * c * (1.0 + 3.0 * 0.044715 * x * x);
}

}  // namespace

extern "C" {

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

double orc_decode(uint32_t bits, int dtype) { return decode(bits, dtype); }
uint32_t orc_encode(double v, int dtype) { return encode(v, dtype); }
double orc_p2f(double x) { return p2f(x); }
double orc_kf(int64_t K) { return kf(K); }

void orc_decode_array(const void* bits, int dtype, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = decode(load_bits(bits, dtype, i), dtype);
}

void orc_encode_array(const double* v, int dtype, int64_t n, void* out) {
  for (int64_t i = 0; i < n; ++i) store_bits(out, dtype, i, encode(v[i], dtype));
}

// Statistic of the DATA component of an array (Section 3.3: the statistic is
// taken after get_data_and_scale, i.e. on data, not on value).
double orc_statistic(const void* x, int dtype, int64_t n, int stat) {
  std::vector<double> d(static_cast<size_t>(n));
  orc_decode_array(x, dtype, n, d.data());
  return statistic(d, stat);
}

// Scaled matmul (Section 3.2, the matmul rule of Algorithm 3 rebuilt from the
// prose: static rule from the operand scales and the contraction size under
// the independent unit-Gaussian assumption, scale rounded down to a power of 2).
//   Y_s = A_s * B_s * kf(K);  Y_d = (A_d . B_d) / kf(K)
// A is [M,K] (or stored [K,M] when transA), B is [K,N] (or stored [N,K] when
// transB); lda/ldb/ldy are row strides in elements of the STORED matrices.
// Optional outputs: acc (fp64 dot product divided by kf(K)) and sabs
// (sum_k |a*b| divided by kf(K)), both [M,N] dense; either may be NULL.
void orc_scaled_matmul(const void* A, int a_dtype, int64_t lda, int transA, float a_scale,
                       const void* B, int b_dtype, int64_t ldb, int transB, float b_scale,
                       int64_t M, int64_t N, int64_t K,
                       int y_dtype, void* Y, int64_t ldy, float* y_scale,
                       double* acc_out, double* sabs_out) {
  std::vector<double> Ad(static_cast<size_t>(M * K)), Bd(static_cast<size_t>(K * N));
  for (int64_t i = 0; i < M; ++i)
    for (int64_t k = 0; k < K; ++k)
      Ad[i * K + k] = decode(load_bits(A, a_dtype, transA ? k * lda + i : i * lda + k), a_dtype);
  for (int64_t k = 0; k < K; ++k)
    for (int64_t j = 0; j < N; ++j)
      Bd[k * N + j] = decode(load_bits(B, b_dtype, transB ? j * ldb + k : k * ldb + j), b_dtype);
  const double f = kf(K);
  if (y_scale) *y_scale = static_cast<float>(static_cast<double>(a_scale) * static_cast<double>(b_scale) * f);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    std::vector<double> acc(static_cast<size_t>(N), 0.0), sab(static_cast<size_t>(N), 0.0);
    for (int64_t k = 0; k < K; ++k) {
      const double a = Ad[i * K + k];
      const double* brow = &Bd[k * N];
      for (int64_t j = 0; j < N; ++j) {
        const double p = a * brow[j];
        acc[j] += p;
        sab[j] += std::fabs(p);
      }
    }
    for (int64_t j = 0; j < N; ++j) {
      const double yd = acc[j] / f;
      if (Y) store_bits(Y, y_dtype, i * ldy + j, encode(yd, y_dtype));
      if (acc_out) acc_out[i * N + j] = yd;
      if (sabs_out) sabs_out[i * N + j] = sab[j] / f;
    }
  }
}

// Scaled matmul with DELAYED rescaling (Section 3.3: the statistic and the rebalancing are
// decoupled, the statistic of an earlier step is kept in the state).  The output is written
// already rebalanced by r = p2f(stat_in) (r = 1 when stat_in cannot define a scale):
//   Y_d = encode((A_d . B_d) / kf(K) / r),  Y_s = A_s * B_s * kf(K) * r,
// and the statistic of THIS step's un-rebalanced data (A_d . B_d)/kf(K), taken before any
// rounding, is returned for the next step.
double orc_scaled_matmul_delayed(const void* A, int a_dtype, int64_t lda, int transA, float a_scale,
                                 const void* B, int b_dtype, int64_t ldb, int transB, float b_scale,
                                 int64_t M, int64_t N, int64_t K, double stat_in, int stat,
                                 int y_dtype, void* Y, int64_t ldy, float* y_scale) {
  std::vector<double> acc(static_cast<size_t>(M * N));
  float ys0 = 0.f;
  orc_scaled_matmul(A, a_dtype, lda, transA, a_scale, B, b_dtype, ldb, transB, b_scale, M, N, K, F32, nullptr, N, &ys0,
                    acc.data(), nullptr);
  const double r = usable_stat(stat_in) ? p2f(stat_in) : 1.0;
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) store_bits(Y, y_dtype, i * ldy + j, encode(acc[i * N + j] / r, y_dtype));
  if (y_scale) *y_scale = static_cast<float>(static_cast<double>(ys0) * r);
  return statistic(acc, stat);
}

// The same rule evaluated for a list of output positions only (full-size
// parity checks on sampled outputs).
void orc_scaled_matmul_samples(const void* A, int a_dtype, int64_t lda, int transA,
                               const void* B, int b_dtype, int64_t ldb, int transB,
                               int64_t K, int64_t n_samples, const int64_t* rows, const int64_t* cols,
                               double* acc_out, double* sabs_out) {
  const double f = kf(K);
#pragma omp parallel for schedule(static)
  for (int64_t s = 0; s < n_samples; ++s) {
    const int64_t i = rows[s], j = cols[s];
    double acc = 0.0, sab = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      const double a = decode(load_bits(A, a_dtype, transA ? k * lda + i : i * lda + k), a_dtype);
      const double b = decode(load_bits(B, b_dtype, transB ? j * ldb + k : k * ldb + j), b_dtype);
      acc += a * b;
      sab += std::fabs(a * b);
    }
    acc_out[s] = acc / f;
    if (sabs_out) sabs_out[s] = sab / f;
  }
}

// Dynamic rescale (Section 3.3, Algorithm 4 rebuilt from the prose):
// statistic of the data -> rounded down to a power of two r -> rebalance:
// data / r, scale * r.  stat_override >= 0 replaces the computed statistic
// (delayed rescaling: statistic gathered elsewhere).  Returns the statistic.
double orc_rescale(const void* x, int x_dtype, int64_t n, float x_scale, int stat, double stat_override,
                   int y_dtype, void* y, float* y_scale) {
  std::vector<double> d(static_cast<size_t>(n));
  orc_decode_array(x, x_dtype, n, d.data());
  double s = (stat_override >= 0.0) ? stat_override : statistic(d, stat);
  double r = usable_stat(s) ? p2f(s) : 1.0;
  for (int64_t i = 0; i < n; ++i) store_bits(y, y_dtype, i, encode(d[i] / r, y_dtype));
  if (y_scale) *y_scale = static_cast<float>(static_cast<double>(x_scale) * r);
  return s;
}

// set_scaling (Section 3.1): force the scale; data rescaled by old/new.  A
// requested scale that is not a power of two is rounded down first.
void orc_set_scaling(const void* x, int x_dtype, int64_t n, float x_scale, float new_scale,
                     int y_dtype, void* y, float* y_scale) {
  const double ns = p2f(static_cast<double>(new_scale));
  const double ratio = static_cast<double>(x_scale) / ns;
  for (int64_t i = 0; i < n; ++i)
    store_bits(y, y_dtype, i, encode(decode(load_bits(x, x_dtype, i), x_dtype) * ratio, y_dtype));
  if (y_scale) *y_scale = static_cast<float>(ns);
}

// Scaled add / sub (Section 3.2, the add rule of Algorithm 3 rebuilt from the
// prose: independent Gaussians => variances add):
//   Y_s = p2f(sqrt(A_s^2 + B_s^2));  Y_d = A_d*(A_s/Y_s) +- B_d*(B_s/Y_s)
// A is [M,N]; B is [M,N], or [N] broadcast over rows when b_row_broadcast.
void orc_scaled_add(const void* A, int a_dtype, float a_scale,
                    const void* B, int b_dtype, float b_scale, int b_row_broadcast, int subtract,
                    int64_t M, int64_t N, int y_dtype, void* Y, float* y_scale) {
  const double as = a_scale, bs = b_scale;
  const double ys = p2f(std::sqrt(as * as + bs * bs));
  const double fa = as / ys, fb = (subtract ? -bs : bs) / ys;
  for (int64_t i = 0; i < M; ++i)
    for (int64_t j = 0; j < N; ++j) {
      const double a = decode(load_bits(A, a_dtype, i * N + j), a_dtype);
      const double b = decode(load_bits(B, b_dtype, b_row_broadcast ? j : i * N + j), b_dtype);
      store_bits(Y, y_dtype, i * N + j, encode(a * fa + b * fb, y_dtype));
    }
  if (y_scale) *y_scale = static_cast<float>(ys);
}

// Scaled LayerNorm forward (Appendix C.2): normalise the DATA component,
// output scale 1, epsilon added to the standard deviation as printed
// (eps_inside_sqrt = 1 gives the textbook sqrt(var + eps)); then the affine
// part by the ordinary mul and add rules:
//   n = (x_d - mean)/(sigma + eps);  Y_s = p2f(sqrt(g_s^2 + b_s^2));
//   Y_d = n*gamma_d*(g_s/Y_s) + beta_d*(b_s/Y_s)
// gamma/beta may be NULL (then Y_d = n, Y_s = 1).  mean/rinv: [R] fp64 out.
void orc_layernorm_fwd(const void* X, int x_dtype, int64_t R, int64_t d,
                       const void* gamma, int g_dtype, float g_scale,
                       const void* beta, int b_dtype, float b_scale,
                       double eps, int eps_inside_sqrt,
                       int y_dtype, void* Y, float* y_scale, double* mean_out, double* rinv_out) {
  double ys = 1.0, fg = 1.0, fb = 0.0;
  if (gamma) {
    const double gs = g_scale, bs = beta ? static_cast<double>(b_scale) : 0.0;
    ys = p2f(std::sqrt(gs * gs + bs * bs));
    fg = gs / ys;
    fb = bs / ys;
  }
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < R; ++r) {
    std::vector<double> x(static_cast<size_t>(d));
    double mu = 0.0;
    for (int64_t j = 0; j < d; ++j) {
      x[j] = decode(load_bits(X, x_dtype, r * d + j), x_dtype);
      mu += x[j];
    }
    mu /= static_cast<double>(d);
    double var = 0.0;
    for (int64_t j = 0; j < d; ++j) var += (x[j] - mu) * (x[j] - mu);
    var /= static_cast<double>(d);
    const double rinv = eps_inside_sqrt ? 1.0 / std::sqrt(var + eps) : 1.0 / (std::sqrt(var) + eps);
    if (mean_out) mean_out[r] = mu;
    if (rinv_out) rinv_out[r] = rinv;
    for (int64_t j = 0; j < d; ++j) {
      double n = (x[j] - mu) * rinv;
      double y = n;
      if (gamma) {
        y = n * decode(load_bits(gamma, g_dtype, j), g_dtype) * fg;
        if (beta) y += decode(load_bits(beta, b_dtype, j), b_dtype) * fb;
      }
      store_bits(Y, y_dtype, r * d + j, encode(y, y_dtype));
    }
  }
  if (y_scale) *y_scale = static_cast<float>(ys);
}

// Scaled LayerNorm backward (Section 4, custom LayerNorm of Algorithm 5; the
// dynamic rescale of the input gradient is a separate orc_rescale call on dX).
//   ghat = G_d*gamma_d (scale G_s*gamma_s), n as in the forward,
//   eps outside the root:  dx = (ghat - mean(ghat))/(s+eps) - n*mean(ghat*n)/s   (second term 0 if s == 0)
//   eps inside the root:   dx = r*(ghat - mean(ghat) - n*mean(ghat*n)), r = 1/sqrt(var+eps)
//   dX_s = G_s*gamma_s / X_s  (chain rule through X = X_d*X_s)
//   dgamma_d = sum_rows(G_d*n)/kf(R), dbeta_d = sum_rows(G_d)/kf(R), both with scale G_s*kf(R)
// dx_f64 (optional, [R,d]) receives dx before encoding.
void orc_layernorm_bwd(const void* G, int gr_dtype, float gr_scale,
                       const void* X, int x_dtype, float x_scale,
                       const void* gamma, int g_dtype, float g_scale,
                       int64_t R, int64_t d, double eps, int eps_inside_sqrt,
                       int dx_dtype, void* dX, float* dx_scale,
                       int dg_dtype, void* dgamma, float* dgamma_scale,
                       void* dbeta, float* dbeta_scale, double* dx_f64) {
  std::vector<double> dg(static_cast<size_t>(d), 0.0), db(static_cast<size_t>(d), 0.0);
  std::vector<double> gam(static_cast<size_t>(d), 1.0);
  if (gamma) for (int64_t j = 0; j < d; ++j) gam[j] = decode(load_bits(gamma, g_dtype, j), g_dtype);
  for (int64_t r = 0; r < R; ++r) {
    std::vector<double> x(static_cast<size_t>(d)), g(static_cast<size_t>(d)), n(static_cast<size_t>(d));
    double mu = 0.0;
    for (int64_t j = 0; j < d; ++j) {
      x[j] = decode(load_bits(X, x_dtype, r * d + j), x_dtype);
      g[j] = decode(load_bits(G, gr_dtype, r * d + j), gr_dtype);
      mu += x[j];
    }
    mu /= static_cast<double>(d);
    double var = 0.0;
    for (int64_t j = 0; j < d; ++j) var += (x[j] - mu) * (x[j] - mu);
    var /= static_cast<double>(d);
    const double s = std::sqrt(var);
    const double rinv = eps_inside_sqrt ? 1.0 / std::sqrt(var + eps) : 1.0 / (s + eps);
    double m1 = 0.0, m2 = 0.0;
    for (int64_t j = 0; j < d; ++j) {
      n[j] = (x[j] - mu) * rinv;
      const double gh = g[j] * gam[j];
      m1 += gh;
      m2 += gh * n[j];
      dg[j] += g[j] * n[j];
      db[j] += g[j];
    }
    m1 /= static_cast<double>(d);
    m2 /= static_cast<double>(d);
    for (int64_t j = 0; j < d; ++j) {
      const double gh = g[j] * gam[j];
      double dx;
      if (eps_inside_sqrt) dx = rinv * (gh - m1 - n[j] * m2);
      else dx = (gh - m1) * rinv - (s > 0.0 ? n[j] * m2 / s : 0.0);
      if (dX) store_bits(dX, dx_dtype, r * d + j, encode(dx, dx_dtype));
      if (dx_f64) dx_f64[r * d + j] = dx;
    }
  }
  const double f = kf(R);
  const double gs = gamma ? static_cast<double>(g_scale) : 1.0;
  if (dx_scale) *dx_scale = static_cast<float>(p2f(static_cast<double>(gr_scale) * gs / static_cast<double>(x_scale)));
  for (int64_t j = 0; j < d; ++j) {
    if (dgamma) store_bits(dgamma, dg_dtype, j, encode(dg[j] / f, dg_dtype));
    if (dbeta) store_bits(dbeta, dg_dtype, j, encode(db[j] / f, dg_dtype));
  }
  if (dgamma_scale) *dgamma_scale = static_cast<float>(static_cast<double>(gr_scale) * f);
  if (dbeta_scale) *dbeta_scale = static_cast<float>(static_cast<double>(gr_scale) * f);
}

// Scaled GELU (Appendix C.1): f_scaled(X_d, X_s) = (X_d * g(X_d*X_s), X_s);
// backward dX_d = G_d * f'(X_d*X_s), dX_s = G_s.
void orc_gelu_fwd(const void* X, int x_dtype, float x_scale, int64_t n, int exact_erf,
                  int y_dtype, void* Y, float* y_scale) {
  for (int64_t i = 0; i < n; ++i) {
    const double xd = decode(load_bits(X, x_dtype, i), x_dtype);
    store_bits(Y, y_dtype, i, encode(xd * gelu_gate(xd * static_cast<double>(x_scale), exact_erf), y_dtype));
  }
  if (y_scale) *y_scale = x_scale;
}

void orc_gelu_bwd(const void* G, int g_dtype, float g_scale, const void* X, int x_dtype, float x_scale,
                  int64_t n, int exact_erf, int y_dtype, void* dX, float* dx_scale) {
  for (int64_t i = 0; i < n; ++i) {
    const double gd = decode(load_bits(G, g_dtype, i), g_dtype);
    const double x = decode(load_bits(X, x_dtype, i), x_dtype) * static_cast<double>(x_scale);
    const double fp = gelu_gate(x, exact_erf) + x * gelu_gate_deriv(x, exact_erf);
    store_bits(dX, y_dtype, i, encode(gd * fp, y_dtype));
  }
  if (dx_scale) *dx_scale = g_scale;
}

// ---- support operations of a GPT-style training step.  The paper gives no rule for attention,
// softmax or the loss (Section 3.2.1 only says custom rules are possible there); these are the
// readings this repository takes, stated in value space so that model invariance (Section 1) can
// be checked against a plain unscaled implementation.

// Embedding lookup: Y = wte[ids] + wpe[pos], pos = i mod seq_len, through the add rule.
void orc_embedding_fwd(const int64_t* ids, int64_t n, int64_t seq_len, int64_t d,
                       const void* wte, int wte_dtype, float wte_scale, const void* wpe, int wpe_dtype, float wpe_scale,
                       int y_dtype, void* Y, float* y_scale) {
  const double ts = wte_scale, ps = wpe ? static_cast<double>(wpe_scale) : 0.0;
  const double ys = p2f(std::sqrt(ts * ts + ps * ps));
  for (int64_t i = 0; i < n; ++i)
    for (int64_t j = 0; j < d; ++j) {
      double v = decode(load_bits(wte, wte_dtype, ids[i] * d + j), wte_dtype) * (ts / ys);
      if (wpe) v += decode(load_bits(wpe, wpe_dtype, (i % seq_len) * d + j), wpe_dtype) * (ps / ys);
      store_bits(Y, y_dtype, i * d + j, encode(v, y_dtype));
    }
  if (y_scale) *y_scale = static_cast<float>(ys);
}

// Embedding backward: dwte[v] = sum of the gradient rows whose token is v (scale unchanged: the
// number of addends per row is data dependent, so no static factor is applied and the sum is kept in
// a wide output format); dwpe[p] = sum over the n/seq_len sequences, a reduction of known size B,
// divided by kf(B) with scale dY_s*kf(B).
void orc_embedding_bwd(const int64_t* ids, int64_t n, int64_t seq_len, int64_t d, int64_t vocab,
                       const void* dY, int dy_dtype, float dy_scale, int out_dtype,
                       void* dwte, float* dwte_scale, void* dwpe, float* dwpe_scale) {
  std::vector<double> te(static_cast<size_t>(vocab * d), 0.0), pe(static_cast<size_t>(seq_len * d), 0.0);
  for (int64_t i = 0; i < n; ++i)
    for (int64_t j = 0; j < d; ++j) {
      const double g = decode(load_bits(dY, dy_dtype, i * d + j), dy_dtype);
      te[ids[i] * d + j] += g;
      pe[(i % seq_len) * d + j] += g;
    }
  const double f = kf(n / seq_len);
  for (int64_t k = 0; k < vocab * d; ++k) store_bits(dwte, out_dtype, k, encode(te[k], out_dtype));
  if (dwpe)
    for (int64_t k = 0; k < seq_len * d; ++k) store_bits(dwpe, out_dtype, k, encode(pe[k] / f, out_dtype));
  if (dwte_scale) *dwte_scale = dy_scale;
  if (dwpe_scale) *dwpe_scale = static_cast<float>(static_cast<double>(dy_scale) * f);
}

// Row softmax of the VALUES S_d*S_s with an optional causal mask (row i of each [Tq,Tk] matrix sees
// columns j <= i + Tk - Tq); the probabilities are bounded in [0,1] and carry scale 1, like the gate
// of an activation (Appendix C.1).  Masked positions are exactly 0.
void orc_softmax_fwd(const void* S, int s_dtype, float s_scale, int64_t batch, int64_t Tq, int64_t Tk, int causal,
                     int p_dtype, void* P, float* p_scale) {
  for (int64_t b = 0; b < batch; ++b)
    for (int64_t i = 0; i < Tq; ++i) {
      const int64_t lim = causal ? std::min<int64_t>(Tk, i + Tk - Tq + 1) : Tk;
      const int64_t off = (b * Tq + i) * Tk;
      double mx = -std::numeric_limits<double>::infinity();
      for (int64_t j = 0; j < lim; ++j)
        mx = std::max(mx, decode(load_bits(S, s_dtype, off + j), s_dtype) * static_cast<double>(s_scale));
      double sum = 0.0;
      for (int64_t j = 0; j < lim; ++j)
        sum += std::exp(decode(load_bits(S, s_dtype, off + j), s_dtype) * static_cast<double>(s_scale) - mx);
      for (int64_t j = 0; j < Tk; ++j) {
        double p = 0.0;
        if (j < lim) p = std::exp(decode(load_bits(S, s_dtype, off + j), s_dtype) * static_cast<double>(s_scale) - mx) / sum;
        store_bits(P, p_dtype, off + j, encode(p, p_dtype));
      }
    }
  if (p_scale) *p_scale = 1.0f;
}

// Softmax backward in value space: dS = P * (dP - sum_j dP_j P_j); the Jacobian is bounded by 1, so
// the gradient scale passes through unchanged (dS_s = dP_s * P_s), as for activations.
void orc_softmax_bwd(const void* dP, int dp_dtype, float dp_scale, const void* P, int p_dtype, float p_scale,
                     int64_t rows, int64_t Tk, int ds_dtype, void* dS, float* ds_scale) {
  for (int64_t r = 0; r < rows; ++r) {
    double dot = 0.0;
    for (int64_t j = 0; j < Tk; ++j)
      dot += decode(load_bits(dP, dp_dtype, r * Tk + j), dp_dtype) * decode(load_bits(P, p_dtype, r * Tk + j), p_dtype);
    for (int64_t j = 0; j < Tk; ++j) {
      const double p = decode(load_bits(P, p_dtype, r * Tk + j), p_dtype);
      const double g = decode(load_bits(dP, dp_dtype, r * Tk + j), dp_dtype);
      store_bits(dS, ds_dtype, r * Tk + j, encode(p * (g - dot), ds_dtype));
    }
  }
  if (ds_scale) *ds_scale = static_cast<float>(static_cast<double>(dp_scale) * static_cast<double>(p_scale));
}

// Mean cross-entropy of the VALUES z = logits_d*logits_s over n rows and the first n_classes columns
// (row stride ld >= n_classes; padding columns are ignored and receive zero gradient), through
// logsumexp (Appendix B).  Gradient w.r.t. the logits' values: (softmax(z) - onehot)/n, written as
// data softmax - onehot in [-1,1] with scale 1/n rounded down to a power of two times the remainder
// folded into the data.  Returns the loss.
double orc_cross_entropy(const void* logits, int l_dtype, float l_scale, int64_t n, int64_t n_classes, int64_t ld,
                         const int64_t* targets, int g_dtype, void* dlogits, float* g_scale) {
  const double inv_n = 1.0 / static_cast<double>(n);
  const double gs = p2f(inv_n);
  const double rem = inv_n / gs;  // in [1,2): kept in the data
  double loss = 0.0;
  for (int64_t i = 0; i < n; ++i) {
    double mx = -std::numeric_limits<double>::infinity();
    for (int64_t j = 0; j < n_classes; ++j)
      mx = std::max(mx, decode(load_bits(logits, l_dtype, i * ld + j), l_dtype) * static_cast<double>(l_scale));
    double sum = 0.0;
    for (int64_t j = 0; j < n_classes; ++j)
      sum += std::exp(decode(load_bits(logits, l_dtype, i * ld + j), l_dtype) * static_cast<double>(l_scale) - mx);
    const double zt = decode(load_bits(logits, l_dtype, i * ld + targets[i]), l_dtype) * static_cast<double>(l_scale);
    loss += (mx + std::log(sum)) - zt;
    if (dlogits)
      for (int64_t j = 0; j < ld; ++j) {
        double g = 0.0;
        if (j < n_classes) {
          g = std::exp(decode(load_bits(logits, l_dtype, i * ld + j), l_dtype) * static_cast<double>(l_scale) - mx) / sum;
          if (j == targets[i]) g -= 1.0;
        }
        store_bits(dlogits, g_dtype, i * ld + j, encode(g * rem, g_dtype));
      }
  }
  if (g_scale) *g_scale = static_cast<float>(gs);
  return loss * inv_n;
}

// Scaled Adam step.  The paper states only that the optimizer update is traced
// with the same static rules and that state is FP16 ScaledArray (Sections 1, 3
// and 4, Table 3 row 4).  Value-space mathematics: textbook Adam with bias
// correction and eps added to sqrt(v_hat).  Output scales: the static rules
// applied to that expression, a scalar constant c carrying scale p2f(|c|)
// (Section 3.4, mantissa/exponent split), mul -> product of scales, add ->
// p2f(sqrt(a^2+b^2)), div -> ratio, sqrt -> p2f(sqrt(s)):
//   m'_s = add(p2f(b1)*m_s, p2f(1-b1)*g_s)
//   v'_s = add(p2f(b2)*v_s, p2f(1-b2)*g_s^2)
//   u_s  = p2f(lr) * (m'_s / p2f(1-b1^t)) / add(p2f(sqrt(v'_s / p2f(1-b2^t))), p2f(eps))
//   w'_s = add(w_s, u_s)
// Data: each output is encoded once from the fp64 value divided by its scale.
// g: g_dtype; m, v: m_dtype (F16 or F32); w: w_dtype (F16 or F32).  In place.
void orc_adam_step(int64_t n, const void* g, int g_dtype, float g_scale,
                   void* m, void* v, int mv_dtype, float* m_scale, float* v_scale,
                   void* w, int w_dtype, float* w_scale,
                   float lr, float beta1, float beta2, float eps, int64_t step) {
  auto add_rule = [](double a, double b) { return p2f(std::sqrt(a * a + b * b)); };
  auto cscale = [](double c) { return c == 0.0 ? 1.0 : p2f(std::fabs(c)); };
  const double b1 = beta1, b2 = beta2, l = lr, e = eps;
  const double bc1 = 1.0 - std::pow(b1, static_cast<double>(step));
  const double bc2 = 1.0 - std::pow(b2, static_cast<double>(step));
  const double gs = g_scale, ms = *m_scale, vs = *v_scale, ws = *w_scale;
  const double one_m_b1 = 1.0 - b1, one_m_b2 = 1.0 - b2;
  const double ms2 = add_rule(cscale(b1) * ms, cscale(one_m_b1) * gs);
  const double vs2 = add_rule(cscale(b2) * vs, cscale(one_m_b2) * gs * gs);
  const double den_s = add_rule(p2f(std::sqrt(vs2 / cscale(bc2))), cscale(e));
  const double us = cscale(l) * (ms2 / cscale(bc1)) / den_s;
  const double ws2 = add_rule(ws, us);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const double gv = decode(load_bits(g, g_dtype, i), g_dtype) * gs;
    const double mv = decode(load_bits(m, mv_dtype, i), mv_dtype) * ms;
    const double vv = decode(load_bits(v, mv_dtype, i), mv_dtype) * vs;
    const double wv = decode(load_bits(w, w_dtype, i), w_dtype) * ws;
    const double m2 = b1 * mv + one_m_b1 * gv;
    const double v2 = b2 * vv + one_m_b2 * gv * gv;
    const double mhat = m2 / bc1;
    const double vhat = v2 / bc2;
    const double w2 = wv - l * mhat / (std::sqrt(vhat) + e);
    store_bits(m, mv_dtype, i, encode(m2 / ms2, mv_dtype));
    store_bits(v, mv_dtype, i, encode(v2 / vs2, mv_dtype));
    store_bits(w, w_dtype, i, encode(w2 / ws2, w_dtype));
  }
  *m_scale = static_cast<float>(ms2);
  *v_scale = static_cast<float>(vs2);
  *w_scale = static_cast<float>(ws2);
}

// ---------------------------------------------------------------------------------------------
// Block scales (Section 2: the scale component may be any array broadcastable to the data; the
// paper names E8M0 and the OCP micro-scaling formats as the standard it follows).
//
// Reading used here: a block-scaled ScaledArray is (data, E, scale) with
//   value[i,k] = data[i,k] * 2^(E[i, k/32] - 127) * scale,
// E an E8M0 code (0..254; 255 is NaN) shared by 32 consecutive elements of a row, i.e. along
// the contraction dimension (OCP MX).  The tensor-wide scale stays one fp32 power of two and is
// the only thing the static rules see; the block exponents belong to the data component.
// ---------------------------------------------------------------------------------------------

double orc_e8m0_decode(uint32_t code) {
  if (code >= 255u) return std::numeric_limits<double>::quiet_NaN();
  return std::ldexp(1.0, static_cast<int>(code) - 127);
}

// Largest power-of-two exponent of a normal number of the element format (OCP MX: "emax").
static int elem_emax(int dtype) { return dtype == 0 ? 8 : 15; }

// Quantise the data component of X [R,K] (K a multiple of 32) to FP8 elements with one E8M0
// exponent per 32 elements: per block, e = floor(log2(max|x|)) - emax(element format), clamped
// to the E8M0 range, data = encode(x / 2^e) (saturating, round to nearest even).  A block whose
// maximum is zero or not finite gets e = 0, like a dynamic rescale whose statistic cannot
// define a scale (Section 3.3).  This is the dynamic rescale with the AMAX statistic applied per
// block, the power of two rounded DOWN as everywhere else (Section 3.2).
void orc_mx_quantize(const void* X, int x_dtype, int64_t R, int64_t K, int elem_dtype, void* data_out,
                     uint8_t* e8m0_out) {
  const int64_t nb = K / 32;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < R; ++i) {
    for (int64_t b = 0; b < nb; ++b) {
      double v[32], amax = 0.0;
      bool finite = true;
      for (int t = 0; t < 32; ++t) {
        v[t] = decode(load_bits(X, x_dtype, i * K + b * 32 + t), x_dtype);
        if (!std::isfinite(v[t])) finite = false;
        amax = std::max(amax, std::fabs(v[t]));
      }
      int e = 0;
      if (finite && amax > 0.0) {
        int ex;
        std::frexp(amax, &ex);  // amax = f * 2^ex, f in [0.5, 1)  =>  floor(log2 amax) = ex - 1
        e = (ex - 1) - elem_emax(elem_dtype);
        e = std::max(-127, std::min(127, e));
      }
      e8m0_out[i * nb + b] = static_cast<uint8_t>(e + 127);
      for (int t = 0; t < 32; ++t)
        store_bits(data_out, elem_dtype, i * K + b * 32 + t, encode(std::ldexp(v[t], -e), elem_dtype));
    }
  }
}

// Block-scaled matmul with the static matmul rule on the tensor scales:
//   Y_s = A_s * B_s * kf(K),   Y_d = (sum_k a[i,k] * b[j,k]) / kf(K),
// a[i,k] = A_d[i,k] * 2^(Ea[i,k/32]-127), b[j,k] = B_d[j,k] * 2^(Eb[j,k/32]-127).
// A is [M,K], B is [N,K] (both with the contraction dimension innermost), Ea [M,K/32],
// Eb [N,K/32].  Optional acc / sabs outputs as in orc_scaled_matmul.
void orc_mx_matmul(const void* A, int a_dtype, const uint8_t* Ea, float a_scale,
                   const void* B, int b_dtype, const uint8_t* Eb, float b_scale,
                   int64_t M, int64_t N, int64_t K, int y_dtype, void* Y, int64_t ldy, float* y_scale,
                   double* acc_out, double* sabs_out) {
  const int64_t nb = K / 32;
  std::vector<double> Ad(static_cast<size_t>(M * K)), Bd(static_cast<size_t>(N * K));
  for (int64_t i = 0; i < M; ++i)
    for (int64_t k = 0; k < K; ++k)
      Ad[i * K + k] = decode(load_bits(A, a_dtype, i * K + k), a_dtype) * orc_e8m0_decode(Ea[i * nb + k / 32]);
  for (int64_t j = 0; j < N; ++j)
    for (int64_t k = 0; k < K; ++k)
      Bd[j * K + k] = decode(load_bits(B, b_dtype, j * K + k), b_dtype) * orc_e8m0_decode(Eb[j * nb + k / 32]);
  const double f = kf(K);
  if (y_scale) *y_scale = static_cast<float>(static_cast<double>(a_scale) * static_cast<double>(b_scale) * f);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < M; ++i) {
    for (int64_t j = 0; j < N; ++j) {
      double acc = 0.0, sab = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        const double p = Ad[i * K + k] * Bd[j * K + k];
        acc += p;
        sab += std::fabs(p);
      }
      const double yd = acc / f;
      if (Y) store_bits(Y, y_dtype, i * ldy + j, encode(yd, y_dtype));
      if (acc_out) acc_out[i * N + j] = yd;
      if (sabs_out) sabs_out[i * N + j] = sab / f;
    }
  }
}

}  // extern "C"
