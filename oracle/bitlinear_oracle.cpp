// CPU oracle for the BitLinear forward pass (BitNet, Sec. 2.1).
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, double-precision
// restatement of the paper's equations, taken one step at a time in the paper's order and
// notation.  It shares no code, header, table or constant with the CUDA library; only the
// tests, the smoke check and the CPU-baseline leg of the benchmark may call it.
//
// Conventions fixed where the paper is silent, and one departure from it as printed:
//   * rounding is round-half-to-even (nearbyint under FE_TONEAREST) applied to the double
//     product, then the clip: codes lie in [-(Q_b-1), Q_b-1], or [0, Q_b-1] in eta mode;
//   * Sign(0) = -1 (Eq. 2), evaluated on the double difference W_ij - alpha_g;
//   * groups split the contraction dimension K into G equal slices (Eq. 13-15);
//   * LN has no gain or bias and uses the population variance (Eq. 12);
//   * gamma == 0 gives all-zero codes (no division by zero);
//   * in the eta form (Eq. 6) gamma = max x^ - min x^, the range of the shifted values.  This departs
//     from Eq. 5 / 14 as printed, which define gamma = ||x||_inf once and redefine only eta for Eq. 6:
//     with that gamma the shifted values would not land in [0, Q_b], which Eq. 6 says they do.
//
// Pins (tests/test_oracle_pins.py): hand-computed worked examples under tests/golden/,
// closed forms for alpha/beta, the Sign tie, code bounds and saturation, the half-to-even
// ties, LN moments, brute force on tiny shapes, one-hot read-back of the bit order, a
// float64 library GEMM on the unpacked operands, group identities, and planted-mistake
// checks.  No function here is "parity unpinned".
//
// Build: g++ -O2 -fopenmp -shared -fPIC (see oracle/build.py).  OpenMP only splits
// independent output rows; there is no blocking, fusion or reordering.

#include <cfenv>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// Neumaier-compensated running sum of doubles.
struct CompSum {
  double s = 0.0, c = 0.0;
  void add(double v) {
    double t = s + v;
    if (std::fabs(s) >= std::fabs(v)) c += (s - t) + v; else c += (v - t) + s;
    s = t;
  }
  double value() const { return s + c; }
};

inline double round_half_even(double v) {
  // nearbyint honours the current rounding mode; the mode is set to nearest-even by callers.
  return std::nearbyint(v);
}

}  // namespace

extern "C" {

enum { ORACLE_ABSMAX = 0, ORACLE_ETA = 1 };
enum { ORACLE_PER_TENSOR = 0, ORACLE_PER_TOKEN = 1 };

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Eq. 1-3 and the group form Eq. 13; beta from Eq. 12.
//   W [N,K] row-major; group g owns columns [g*K/G, (g+1)*K/G) of every row.
//   alpha_in: NULL, or G values used in place of the computed mean.
//   bits  [N*K/8]: bit (k%8) of byte n*K/8 + k/8 is 1 when Sign(W[n,k]-alpha_g) = +1.
//   alpha,beta [G] doubles; rowsum [N*G] = sum over the group's columns of Sign(..).
int oracle_binarize(const float* W, int64_t N, int64_t K, int G, const double* alpha_in,
                    uint8_t* bits, double* alpha, double* beta, int32_t* rowsum) {
  if (!W || !bits || !alpha || !beta || N <= 0 || K <= 0 || G <= 0) return 1;
  if (K % (8 * (int64_t)G) != 0) return 2;
  const int64_t Kg = K / G;
  for (int g = 0; g < G; ++g) {
    CompSum s, a;
    for (int64_t n = 0; n < N; ++n)
      for (int64_t k = g * Kg; k < (g + 1) * Kg; ++k) {
        double w = (double)W[n * K + k];
        s.add(w);
        a.add(std::fabs(w));
      }
    double cnt = (double)N * (double)Kg;
    alpha[g] = alpha_in ? alpha_in[g] : s.value() / cnt;   // Eq. 3 / Eq. 13
    beta[g] = a.value() / cnt;                             // Eq. 12 / Eq. 13
  }
  std::memset(bits, 0, (size_t)(N * K / 8));
  for (int64_t n = 0; n < N; ++n)
    for (int g = 0; g < G; ++g) {
      int32_t rs = 0;
      for (int64_t k = g * Kg; k < (g + 1) * Kg; ++k) {
        double centred = (double)W[n * K + k] - alpha[g];
        int sign = (centred > 0.0) ? +1 : -1;              // Eq. 2: Sign(0) = -1
        if (sign > 0) bits[n * (K / 8) + k / 8] |= (uint8_t)(1u << (k % 8));
        rs += sign;
      }
      if (rowsum) rowsum[n * G + g] = rs;
    }
  return 0;
}

// LN (Eq. 12, per group Eq. 15) followed by Quant (Eq. 4-6, per group Eq. 14), b = 8.
//   x [M,K] row-major (values of the input dtype held exactly in float).
//   ln_eps < 0 skips the normalisation.
//   gran = PER_TOKEN: gamma/eta [M*G] (index m*G+g); PER_TENSOR: gamma/eta [G].
//   codes [M,K]; xhat (optional) [M,K] receives LN(x) in double.
int oracle_quant_act(const float* x, int64_t M, int64_t K, int G, int mode, int gran,
                     double ln_eps, int8_t* codes, double* gamma, double* eta, double* xhat_out) {
  if (!x || !codes || !gamma || M <= 0 || K <= 0 || G <= 0) return 1;
  if (K % (8 * (int64_t)G) != 0) return 2;
  if (mode == ORACLE_ETA && !eta) return 1;
  std::fesetround(FE_TONEAREST);
  const int64_t Kg = K / G;
  const double Qb = 128.0;  // Q_b = 2^(b-1), b = 8
  std::vector<double> xhat((size_t)(M * K));
  // Step 1: LN per token and group.
  for (int64_t m = 0; m < M; ++m)
    for (int g = 0; g < G; ++g) {
      const float* row = x + m * K + g * Kg;
      double* out = xhat.data() + m * K + g * Kg;
      if (ln_eps < 0) {
        for (int64_t k = 0; k < Kg; ++k) out[k] = (double)row[k];
        continue;
      }
      CompSum s;
      for (int64_t k = 0; k < Kg; ++k) s.add((double)row[k]);
      double mu = s.value() / (double)Kg;                  // E(x)
      CompSum v;
      for (int64_t k = 0; k < Kg; ++k) { double d = (double)row[k] - mu; v.add(d * d); }
      double var = v.value() / (double)Kg;                 // Var(x), population
      double denom = std::sqrt(var + ln_eps);
      for (int64_t k = 0; k < Kg; ++k) out[k] = ((double)row[k] - mu) / denom;
    }
  if (xhat_out) std::memcpy(xhat_out, xhat.data(), sizeof(double) * (size_t)(M * K));
  // Step 2: gamma (and eta) over the quantisation scope, then the codes.
  const int64_t scopes = (gran == ORACLE_PER_TOKEN) ? M : 1;
  for (int64_t sc = 0; sc < scopes; ++sc) {
    int64_t m0 = (gran == ORACLE_PER_TOKEN) ? sc : 0;
    int64_t m1 = (gran == ORACLE_PER_TOKEN) ? sc + 1 : M;
    for (int g = 0; g < G; ++g) {
      double mx = -std::numeric_limits<double>::infinity();
      double mn = std::numeric_limits<double>::infinity();
      double amax = 0.0;
      for (int64_t m = m0; m < m1; ++m)
        for (int64_t k = g * Kg; k < (g + 1) * Kg; ++k) {
          double v = xhat[m * K + k];
          if (v > mx) mx = v;
          if (v < mn) mn = v;
          if (std::fabs(v) > amax) amax = std::fabs(v);
        }
      double gam, et;
      if (mode == ORACLE_ABSMAX) { gam = amax; et = 0.0; }          // gamma = ||x||_inf
      else { et = mn; gam = mx - mn; }                              // eta = min x; range [0,Q_b]
      gamma[sc * G + g] = gam;
      if (eta) eta[sc * G + g] = et;
      double s = (gam > 0.0) ? Qb / gam : 0.0;
      for (int64_t m = m0; m < m1; ++m)
        for (int64_t k = g * Kg; k < (g + 1) * Kg; ++k) {
          double r = round_half_even((xhat[m * K + k] - et) * s);
          double lo = (mode == ORACLE_ABSMAX) ? -(Qb - 1.0) : 0.0;  // Clip with eps == 1 code
          double hi = Qb - 1.0;
          if (r < lo) r = lo;
          if (r > hi) r = hi;
          codes[m * K + k] = (int8_t)r;
        }
    }
  }
  return 0;
}

// Eq. 7 per group: acc[g,m,n] = sum_{k in group g} Wt[n,k] * code[m,k], exact integers.
int oracle_matmul(const int8_t* codes, const uint8_t* bits, int64_t M, int64_t N, int64_t K,
                  int G, int32_t* acc) {
  if (!codes || !bits || !acc || M <= 0 || N <= 0 || K <= 0 || G <= 0) return 1;
  if (K % (8 * (int64_t)G) != 0) return 2;
  const int64_t Kg = K / G;
  if (Kg > (int64_t)16000000) return 3;  // 127*Kg must stay below 2^31
  // W-tilde written out as +1/-1 (the plain definition), then the triple loop.
  std::vector<int8_t> Wt((size_t)(N * K));
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k)
      Wt[n * K + k] = ((bits[n * (K / 8) + k / 8] >> (k % 8)) & 1) ? (int8_t)1 : (int8_t)-1;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n)
      for (int g = 0; g < G; ++g) {
        int32_t a = 0;
        const int8_t* wr = Wt.data() + n * K + g * Kg;
        const int8_t* xr = codes + m * K + g * Kg;
        for (int64_t k = 0; k < Kg; ++k) a += (int32_t)wr[k] * (int32_t)xr[k];
        acc[((int64_t)g * M + m) * N + n] = a;
      }
  return 0;
}

// Same sum for selected outputs only: pairs (ms[i], ns[i]) -> acc[i*G + g].
int oracle_matmul_samples(const int8_t* codes, const uint8_t* bits, int64_t M, int64_t N,
                          int64_t K, int G, const int64_t* ms, const int64_t* ns,
                          int64_t count, int32_t* acc) {
  if (!codes || !bits || !acc || !ms || !ns) return 1;
  if (K % (8 * (int64_t)G) != 0) return 2;
  const int64_t Kg = K / G;
  for (int64_t i = 0; i < count; ++i) {
    int64_t m = ms[i], n = ns[i];
    if (m < 0 || m >= M || n < 0 || n >= N) return 4;
    for (int g = 0; g < G; ++g) {
      int64_t a = 0;
      for (int64_t k = g * Kg; k < (g + 1) * Kg; ++k) {
        int w = ((bits[n * (K / 8) + k / 8] >> (k % 8)) & 1) ? 1 : -1;
        a += (int64_t)w * (int64_t)codes[m * K + k];
      }
      acc[i * G + g] = (int32_t)a;
    }
  }
  return 0;
}

// Eq. 11: y[m,n] = sum_g acc[g,m,n] * beta_g * gamma_(m),g / Q_b, groups in ascending order.
// eta_correction != 0 adds eta_(m),g * beta_g * rowsum[n,g], which restores W~ x-hat for
// the shifted codes; 0 is the literal Eq. 11.
int oracle_dequant(const int32_t* acc, int64_t M, int64_t N, int G, int gran,
                   const double* beta, const double* gamma, const double* eta,
                   const int32_t* rowsum, int eta_correction, double* y) {
  if (!acc || !beta || !gamma || !y) return 1;
  if (eta_correction && (!eta || !rowsum)) return 1;
  const double Qb = 128.0;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double s = 0.0;
      for (int g = 0; g < G; ++g) {
        int64_t sc = (gran == ORACLE_PER_TOKEN) ? m * G + g : g;
        s += (double)acc[((int64_t)g * M + m) * N + n] * beta[g] * gamma[sc] / Qb;
        if (eta_correction) s += eta[sc] * beta[g] * (double)rowsum[n * G + g];
      }
      y[m * N + n] = s;
    }
  return 0;
}

// The whole layer, Eq. 11, as the four steps above in order.
int oracle_forward(const float* x, int64_t M, int64_t K, int64_t N, int G, int mode, int gran,
                   double ln_eps, int eta_correction, const uint8_t* bits, const double* beta,
                   const int32_t* rowsum, int8_t* codes_out, double* gamma_out, double* eta_out,
                   int32_t* acc_out, double* y) {
  if (!x || !bits || !beta || !y) return 1;
  const int64_t ns = (gran == ORACLE_PER_TOKEN) ? M * G : G;
  std::vector<int8_t> codes((size_t)(M * K));
  std::vector<double> gamma((size_t)ns), eta((size_t)ns, 0.0);
  int rc = oracle_quant_act(x, M, K, G, mode, gran, ln_eps, codes.data(), gamma.data(),
                            eta.data(), nullptr);
  if (rc) return rc;
  std::vector<int32_t> acc((size_t)((int64_t)G * M * N));
  rc = oracle_matmul(codes.data(), bits, M, N, K, G, acc.data());
  if (rc) return rc;
  rc = oracle_dequant(acc.data(), M, N, G, gran, beta, gamma.data(), eta.data(), rowsum,
                      eta_correction, y);
  if (rc) return rc;
  if (codes_out) std::memcpy(codes_out, codes.data(), codes.size());
  if (gamma_out) std::memcpy(gamma_out, gamma.data(), sizeof(double) * gamma.size());
  if (eta_out) std::memcpy(eta_out, eta.data(), sizeof(double) * eta.size());
  if (acc_out) std::memcpy(acc_out, acc.data(), sizeof(int32_t) * acc.size());
  return 0;
}


// Causal self-attention core of the decoder block (Sec. 2, Fig. 2b), written out from its
// definition in double precision: for query t of (batch b, head h)
//   o_t = sum_{s <= t} softmax_s(q_t . k_s / sqrt(d_h)) v_s .
// q, k, v: float [batch*seq, heads*dh] row-major (values of the 16-bit inputs held exactly).
// rows: `count` token indices (0 .. batch*seq-1) to evaluate, all heads each; out [count, heads*dh].
int oracle_attention_rows(const float* q, const float* k, const float* v, int64_t batch, int64_t seq,
                          int64_t heads, int64_t dh, const int64_t* rows, int64_t count, double* out) {
  if (!q || !k || !v || !rows || !out || batch <= 0 || seq <= 0 || heads <= 0 || dh <= 0) return 1;
  const int64_t ld = heads * dh;
  const double scale = 1.0 / std::sqrt((double)dh);
  for (int64_t i = 0; i < count; ++i)
    if (rows[i] < 0 || rows[i] >= batch * seq) return 4;
#pragma omp parallel for schedule(dynamic)
  for (int64_t job = 0; job < count * heads; ++job) {
    const int64_t i = job / heads, h = job % heads;
    const int64_t tok = rows[i], b = tok / seq, t = tok % seq;
    const float* qt = q + tok * ld + h * dh;
    std::vector<double> score((size_t)(t + 1));
    double mx = -std::numeric_limits<double>::infinity();
    for (int64_t s = 0; s <= t; ++s) {                       // causal: keys 0..t of the same sequence
      const float* ks = k + (b * seq + s) * ld + h * dh;
      double dot = 0.0;
      for (int64_t e = 0; e < dh; ++e) dot += (double)qt[e] * (double)ks[e];
      score[(size_t)s] = dot * scale;
      if (score[(size_t)s] > mx) mx = score[(size_t)s];
    }
    double denom = 0.0;
    for (int64_t s = 0; s <= t; ++s) { score[(size_t)s] = std::exp(score[(size_t)s] - mx); denom += score[(size_t)s]; }
    double* o = out + i * ld + h * dh;
    for (int64_t e = 0; e < dh; ++e) o[e] = 0.0;
    for (int64_t s = 0; s <= t; ++s) {
      const float* vs = v + (b * seq + s) * ld + h * dh;
      const double p = score[(size_t)s] / denom;
      for (int64_t e = 0; e < dh; ++e) o[e] += p * (double)vs[e];
    }
  }
  return 0;
}

}  // extern "C"
