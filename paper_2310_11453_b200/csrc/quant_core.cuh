// LN statistics and the quantisation map of one (token, group) segment, shared by the
// LN+quant kernels and the fused decode kernel.
//
// Precision plan.  The reference semantics are in double precision, and a code flips whenever
// fp32 rounding pushes x^.Q_b/gamma across a half-integer.  To keep such flips rare at HBM
// speed:
//   * sums are fp32 over 8 elements and fp64 from there on (one conversion per 8 elements), so
//     mean and rstd carry ~1e-9 relative error;
//   * extremes are taken on the raw inputs (x -> x^ is increasing), then mapped in fp64;
//   * each element costs one fp32 FMA, code = rne(x*A + B) with A = rstd.Q_b/gamma and
//     B = -(mean.rstd + eta).Q_b/gamma rounded once from fp64;
//   * only when x*A + B lands within a small window of a half-integer (a ~1e-4 fraction of
//     the elements) is that element redone in fp64, in the order the equations are written.
#pragma once

#include "common.cuh"

namespace bl {

struct SegMoments {      // Eq. 12 statistics of a segment
  double mean, rstd;
};

struct QuantMap {        // everything needed to turn a raw x into its code
  double mean, rstd, eta, scale;   // fp64 parameters (slow path)
  float A, B, tau;                 // fp32 fast path and its near-tie window
  int code_lo;                     // -127 (absmax) or 0 (eta mode)
};

template <int kThreads>
struct QuantRed {
  double d[kThreads / 32];
  float lo[kThreads / 32], hi[kThreads / 32];
  SegMoments mom;
  float xlo, xhi;
};

// Pass A: sum and raw extremes.  Pass B: sum of squared deviations from the fp32-rounded mean,
// corrected exactly for that rounding.  seg[] holds the raw segment as fp32 in shared memory.
// On return every thread has mom (mean, rstd) and the raw extremes xlo, xhi.
template <int kThreads>
__device__ __forceinline__ void segment_moments(const float* seg, int Kg, float ln_eps,
                                                QuantRed<kThreads>& red, SegMoments& mom,
                                                float& xlo, float& xhi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double s = 0.0;
  float mn = INFINITY, mx = -INFINITY;
  for (int k = threadIdx.x * 8; k < Kg; k += kThreads * 8) {
    const float4 a = *reinterpret_cast<const float4*>(seg + k);
    const float4 b = *reinterpret_cast<const float4*>(seg + k + 4);
    const float p = ((a.x + a.y) + (a.z + a.w)) + ((b.x + b.y) + (b.z + b.w));
    s += (double)p;
    mn = fminf(mn, fminf(fminf(fminf(a.x, a.y), fminf(a.z, a.w)), fminf(fminf(b.x, b.y), fminf(b.z, b.w))));
    mx = fmaxf(mx, fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w))));
  }
  s = warp_sum(s); mn = warp_min(mn); mx = warp_max(mx);
  __syncthreads();
  if (lane == 0) { red.d[warp] = s; red.lo[warp] = mn; red.hi[warp] = mx; }
  __syncthreads();
  double tot = 0.0;
  mn = red.lo[0]; mx = red.hi[0];
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    tot += red.d[w]; mn = fminf(mn, red.lo[w]); mx = fmaxf(mx, red.hi[w]);
  }
  xlo = mn; xhi = mx;
  if (ln_eps < 0.f) { mom.mean = 0.0; mom.rstd = 1.0; return; }   // LN skipped
  const double mean = tot / (double)Kg;
  const float mean_f = (float)mean;
  double q = 0.0;
  for (int k = threadIdx.x * 8; k < Kg; k += kThreads * 8) {
    const float4 a = *reinterpret_cast<const float4*>(seg + k);
    const float4 b = *reinterpret_cast<const float4*>(seg + k + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float p = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { const float d = v[i] - mean_f; p = fmaf(d, d, p); }
    q += (double)p;
  }
  q = warp_sum(q);
  __syncthreads();
  if (lane == 0) red.d[warp] = q;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) t += red.d[w];
    const double dm = mean - (double)mean_f;
    double var = t / (double)Kg - dm * dm;       // sum (x-mean)^2 = sum (x-mean_f)^2 - K dm^2
    if (var < 0.0) var = 0.0;
    const double denom = var + (double)ln_eps;
    red.mom.mean = mean;
    red.mom.rstd = denom > 0.0 ? 1.0 / sqrt(denom) : 0.0;
  }
  __syncthreads();
  mom = red.mom;
}

// gamma / eta of a scope from the extremes of x^ over it (Eq. 5, 6, 14).
__device__ __forceinline__ void scope_gamma_eta(int mode, double lo, double hi, double& gamma,
                                                double& eta) {
  if (mode == BL_ABSMAX) { gamma = fmax(fabs(lo), fabs(hi)); eta = 0.0; }
  else { eta = lo; gamma = hi - lo; }
}

// The affine fp32 map of a segment given its moments and the scope's gamma / eta;
// xabs bounds |x| over the segment (for the near-tie window).
__device__ __forceinline__ QuantMap make_quant_map(int mode, const SegMoments& mom, double gamma,
                                                   double eta, float xabs) {
  QuantMap m;
  m.mean = mom.mean; m.rstd = mom.rstd; m.eta = eta;
  m.scale = gamma > 0.0 ? (double)kQb / gamma : 0.0;
  const double A = mom.rstd * m.scale;
  const double B = -(mom.mean * mom.rstd + eta) * m.scale;
  m.A = (float)A; m.B = (float)B;
  m.tau = 4e-7f * (fabsf(m.A) * xabs + fabsf(m.B) + 1.0f);
  m.code_lo = (mode == BL_ABSMAX) ? -kCodeMax : 0;
  return m;
}

// Eq. 4 / 6 for one raw element: round-half-to-even, then clip.
__device__ __forceinline__ int quant_element(float x, const QuantMap& m) {
  const float v = fmaf(x, m.A, m.B);
  float r = rintf(v);
  if (fabsf(fabsf(v - r) - 0.5f) < m.tau) {       // too close to a tie for fp32: redo in fp64
    const double xh = ((double)x - m.mean) * m.rstd;
    r = (float)rint((xh - m.eta) * m.scale);
  }
  return max(m.code_lo, min(kCodeMax, (int)r));
}

__device__ __forceinline__ uint2 quant_pack8(const float (&v)[8], const QuantMap& m) {
  uint32_t w[2];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    uint32_t packed = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) packed |= (uint32_t)(quant_element(v[4 * j + i], m) & 0xFF) << (8 * i);
    w[j] = packed;
  }
  return make_uint2(w[0], w[1]);
}

// Order-preserving double <-> u64 encoding for atomic min/max across CTAs.
__device__ __forceinline__ unsigned long long enc_ordered64(double f) {
  unsigned long long b = (unsigned long long)__double_as_longlong(f);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double dec_ordered64(unsigned long long e) {
  unsigned long long b = (e >> 63) ? (e & 0x7FFFFFFFFFFFFFFFull) : ~e;
  return __longlong_as_double((long long)b);
}

}  // namespace bl
