// One (token, group) segment per warp: Eq. 12 statistics and Eq. 4-6 codes of a segment that a warp
// walks in chunks of 8 elements per lane (chunk c = lane + 32 i, i < ni).  Shared by the LN+quant
// kernels (segment staged in shared memory) and the batched decode kernel; `slot` is the 16-byte
// aligned start of the segment, in shared or global memory.
#pragma once

#include <type_traits>

#include "quant_core.cuh"

namespace bl {
namespace rows {

constexpr float kRoundMagic = 12582912.f;                     // 1.5 * 2^23: x + magic - magic = rne(x), |x| < 2^22

__device__ __forceinline__ double rcp_newton(double d) {      // d > 0
  if (!(d > 1e-30 && d < 1e30)) return 1.0 / d;
  double y = (double)__frcp_rn((float)d);
  y = y * (2.0 - d * y);
  return y * (2.0 - d * y);
}
__device__ __forceinline__ double rsqrt_newton(double d) {    // d >= 0
  if (!(d > 1e-30 && d < 1e30)) return d > 0.0 ? 1.0 / sqrt(d) : 0.0;
  double y = (double)rsqrtf((float)d);
  y = y * (1.5 - 0.5 * d * y * y);
  return y * (1.5 - 0.5 * d * y * y);
}

template <typename H2> __device__ __forceinline__ H2 as_h2(uint32_t w) { return *reinterpret_cast<H2*>(&w); }
template <typename H2> __device__ __forceinline__ uint32_t h2_bits(H2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// Chunk c of a staged segment (8 consecutive elements) as fp32.
template <typename T> struct Chunk;
template <> struct Chunk<float> {
  uint4 a, b;
  __device__ __forceinline__ void load(const uint4* slot, int c) { a = slot[2 * c]; b = slot[2 * c + 1]; }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    v[0] = __uint_as_float(a.x); v[1] = __uint_as_float(a.y); v[2] = __uint_as_float(a.z); v[3] = __uint_as_float(a.w);
    v[4] = __uint_as_float(b.x); v[5] = __uint_as_float(b.y); v[6] = __uint_as_float(b.z); v[7] = __uint_as_float(b.w);
  }
};
template <> struct Chunk<__half> {
  uint4 a;
  __device__ __forceinline__ void load(const uint4* slot, int c) { a = slot[c]; }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(as_h2<__half2>(w[j]));
      v[2 * j] = f.x; v[2 * j + 1] = f.y;
    }
  }
};
template <> struct Chunk<__nv_bfloat16> {
  uint4 a;
  __device__ __forceinline__ void load(const uint4* slot, int c) { a = slot[c]; }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[2 * j] = __uint_as_float(w[j] << 16);
      v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
    }
  }
};

struct RowStats { double mean, rstd; float xlo, xhi; };

// Eq. 12 statistics of the staged segment (ni chunks per lane): every lane returns the same values.
// One pass: deviations are taken from a pilot value c (the mean of the segment's first 8
// elements), which keeps sum (x - c) and sum (x - c)^2 small and well conditioned:
//   mean = c + sum (x - c) / K,   Var = sum (x - c)^2 / K - (mean - c)^2.
template <typename T>
__device__ __forceinline__ RowStats row_stats(const uint4* slot, int ni, int lane, float ln_eps, double inv_kg) {
  float pilot;
  {
    Chunk<T> ch; float v[8];
    ch.load(slot, 0); ch.unpack(v);                  // same address in every lane: a broadcast
    pilot = 0.125f * (((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7])));
    if (ln_eps < 0.f) pilot = 0.f;
  }
  float s = 0.f, q = 0.f, mn = INFINITY, mx = -INFINITY;
  uint32_t plo = slot[0].x, phi = plo;               // 16-bit inputs: running packed extremes
#pragma unroll 4
  for (int i = 0; i < ni; ++i) {
    Chunk<T> ch; float v[8], d[8];
    ch.load(slot, lane + 32 * i); ch.unpack(v);
#pragma unroll
    for (int j = 0; j < 8; ++j) d[j] = v[j] - pilot;
    s += ((d[0] + d[1]) + (d[2] + d[3])) + ((d[4] + d[5]) + (d[6] + d[7]));
    float p0 = d[0] * d[0], p1 = d[1] * d[1];
#pragma unroll
    for (int j = 2; j < 8; j += 2) { p0 = fmaf(d[j], d[j], p0); p1 = fmaf(d[j + 1], d[j + 1], p1); }
    q += p0 + p1;
    if constexpr (sizeof(T) == 4) {
#pragma unroll
      for (int j = 0; j < 8; ++j) { mn = fminf(mn, v[j]); mx = fmaxf(mx, v[j]); }
    } else {
      using H2 = typename std::conditional<std::is_same<T, __half>::value, __half2, __nv_bfloat162>::type;
      const uint32_t w[4] = {ch.a.x, ch.a.y, ch.a.z, ch.a.w};
      const H2 a = __hmin2(__hmin2(as_h2<H2>(w[0]), as_h2<H2>(w[1])), __hmin2(as_h2<H2>(w[2]), as_h2<H2>(w[3])));
      const H2 b = __hmax2(__hmax2(as_h2<H2>(w[0]), as_h2<H2>(w[1])), __hmax2(as_h2<H2>(w[2]), as_h2<H2>(w[3])));
      plo = h2_bits(__hmin2(a, as_h2<H2>(plo))); phi = h2_bits(__hmax2(b, as_h2<H2>(phi)));
    }
  }
  if constexpr (std::is_same<T, __half>::value) {
    const float2 fa = __half22float2(as_h2<__half2>(plo)), fb = __half22float2(as_h2<__half2>(phi));
    mn = fminf(fa.x, fa.y); mx = fmaxf(fb.x, fb.y);
  } else if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    const float2 fa = __bfloat1622float2(as_h2<__nv_bfloat162>(plo)), fb = __bfloat1622float2(as_h2<__nv_bfloat162>(phi));
    mn = fminf(fa.x, fa.y); mx = fmaxf(fb.x, fb.y);
  }
  const double S = warp_sum((double)s), Q = warp_sum((double)q);
  RowStats st;
  st.xlo = warp_min(mn); st.xhi = warp_max(mx);
  if (ln_eps < 0.f) { st.mean = 0.0; st.rstd = 1.0; return st; }
  const double dm = S * inv_kg;                      // mean - pilot
  st.mean = (double)pilot + dm;
  double var = Q * inv_kg - dm * dm;
  if (var < 0.0) var = 0.0;
  st.rstd = rsqrt_newton(var + (double)ln_eps);
  return st;
}

struct RowMap {            // Quant of Eq. 4-6 as one fp32 FMA, plus what the exact redo needs
  double mean, rstd, eta, scale;
  float A, B, tau;
  int code_lo;
  bool clip;               // some element of the segment may reach a clip bound (uniform over the segment)
};
__device__ __forceinline__ RowMap row_map(int mode, double mean, double rstd, double gamma, double eta, float xlo,
                                          float xhi) {
  RowMap m;
  m.mean = mean; m.rstd = rstd; m.eta = eta;
  m.scale = gamma > 0.0 ? (double)kQb * rcp_newton(gamma) : 0.0;
  m.A = (float)(rstd * m.scale);
  m.B = (float)(-(mean * rstd + eta) * m.scale);
  m.tau = 4e-7f * (fabsf(m.A) * fmaxf(fabsf(xlo), fabsf(xhi)) + fabsf(m.B) + 1.0f);
  m.code_lo = (mode == BL_ABSMAX) ? -kCodeMax : 0;
  // A >= 0, so x*A + B over the segment spans [xlo*A + B, xhi*A + B]: a quarter inside the
  // bounds, rounding cannot leave them and the clip of Eq. 4 / 6 is the identity.
  m.clip = !(fmaf(xlo, m.A, m.B) > (float)m.code_lo - 0.25f && fmaf(xhi, m.A, m.B) < (float)kCodeMax + 0.25f);
  return m;
}
// The rare chunk with an element too close to a rounding tie for fp32: the equations in fp64,
// in their order, four elements per call.
__device__ __forceinline__ uint32_t row_code_exact(float x, double mean, double rstd, double eta, double scale,
                                                   int code_lo) {
  const double xh = ((double)x - mean) * rstd;
  return (uint32_t)(max(code_lo, min(kCodeMax, (int)rint((xh - eta) * scale))) & 0xFF);
}
static __device__ __noinline__ uint32_t row_codes4_exact(float v0, float v1, float v2, float v3, double mean, double rstd,
                                                  double eta, double scale, int code_lo) {
  return row_code_exact(v0, mean, rstd, eta, scale, code_lo) | row_code_exact(v1, mean, rstd, eta, scale, code_lo) << 8 |
         row_code_exact(v2, mean, rstd, eta, scale, code_lo) << 16 |
         row_code_exact(v3, mean, rstd, eta, scale, code_lo) << 24;
}
template <bool kClip>
__device__ __forceinline__ uint2 row_codes8(const float (&v)[8], const RowMap& m) {
  // Adding the magic constant leaves rne(f) as a two's-complement byte in the low bits of the
  // sum.  With kClip, f is clipped in fp32 first (the bounds are integers, so clip and rne
  // commute).  dist collects max |f - rne(f)| to spot elements within tau of a rounding tie
  // (and, with kClip, elements the clip moved: both go to the exact redo).
  uint32_t t[8];
  float dist = 0.f;
  const float lo = (float)m.code_lo, hi = (float)kCodeMax;
#pragma unroll
  for (int j = 0; j < 8; j += 2) {
    const float f0 = fmaf(v[j], m.A, m.B), f1 = fmaf(v[j + 1], m.A, m.B);
    const float t0 = (kClip ? fminf(fmaxf(f0, lo), hi) : f0) + kRoundMagic;
    const float t1 = (kClip ? fminf(fmaxf(f1, lo), hi) : f1) + kRoundMagic;
    dist = fmaxf(fmaxf(dist, fabsf(f0 - (t0 - kRoundMagic))), fabsf(f1 - (t1 - kRoundMagic)));
    t[j] = __float_as_uint(t0); t[j + 1] = __float_as_uint(t1);
  }
  uint2 out;
  out.x = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
  out.y = __byte_perm(__byte_perm(t[4], t[5], 0x0040), __byte_perm(t[6], t[7], 0x0040), 0x5410);
  if (dist > 0.5f - m.tau) {                                 // rare
    out.x = row_codes4_exact(v[0], v[1], v[2], v[3], m.mean, m.rstd, m.eta, m.scale, m.code_lo);
    out.y = row_codes4_exact(v[4], v[5], v[6], v[7], m.mean, m.rstd, m.eta, m.scale, m.code_lo);
  }
  return out;
}

template <typename T, bool kClip>
__device__ __forceinline__ void row_store_codes_impl(const uint4* slot, int ni, int lane, const RowMap& map,
                                                     int8_t* __restrict__ dst) {
#pragma unroll 2
  for (int i = 0; i < ni; ++i) {
    const int c = lane + 32 * i;
    Chunk<T> ch; float v[8];
    ch.load(slot, c); ch.unpack(v);
    const uint2 cd = row_codes8<kClip>(v, map);
    // (streamed out past L1: nothing on this SM reads the codes again; 1 % on the bench shape)
    asm volatile("st.global.L1::no_allocate.v2.b32 [%0], {%1, %2};" ::"l"(dst + (size_t)c * 8), "r"(cd.x), "r"(cd.y) : "memory");
  }
}
template <typename T>
__device__ __forceinline__ void row_store_codes(const uint4* slot, int ni, int lane, const RowMap& map,
                                                int8_t* __restrict__ dst) {
  if (map.clip) row_store_codes_impl<T, true>(slot, ni, lane, map, dst);
  else row_store_codes_impl<T, false>(slot, ni, lane, map, dst);
}

}  // namespace rows
}  // namespace bl
