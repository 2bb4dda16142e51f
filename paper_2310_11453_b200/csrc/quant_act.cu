// Steps 1-2 of BitLinear: LN per token and group (Eq. 12, 15) fused with the 8-bit activation
// quantisation (Eq. 4-6, 14).  HBM-bound: x is read once (per token) or twice (per tensor) with
// 128-bit loads; the normalised row is never written to HBM.
//
// Two implementations.  Segments of up to 4096 16-bit (2048 fp32) features take the fast path in
// the second half of this file: one warp per segment, the segment in registers.  Longer segments
// take one CTA per (token m, group g) segment, staged in shared memory as fp32:
//   moments  sum, raw min/max, then sum of squared deviations      (quant_core.cuh)
//   codes    one FMA + round per element, 8 codes per 8-byte store
// Per-tensor scope splits in two kernels: the first leaves each segment's moments in the
// workspace and folds the extremes of x^ into a global atomic min/max on an order-preserving
// encoding (order-independent, hence deterministic); the second re-reads x and writes codes.
#include <mutex>
#include <type_traits>

#include "quant_core.cuh"

namespace bl {

namespace {

constexpr int kQuantThreads = 256;

struct SegRecord {                 // per-segment record kept between the two per-tensor kernels
  double mean, rstd;
  float xabs, pad;
};

struct TensorScope {               // workspace header for the per-tensor path
  unsigned long long enc_min[BL_MAX_GROUPS];
  unsigned long long enc_max[BL_MAX_GROUPS];
};

template <typename T>
__device__ __forceinline__ void stage_segment(const T* __restrict__ src, int Kg, float* seg) {
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    float v[8];
    Elem<T>::load8(src + k, v);
    *reinterpret_cast<float4*>(seg + k) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(seg + k + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
quant_per_token(const T* __restrict__ x, int64_t K, int G, int mode, float ln_eps,
                int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  extern __shared__ __align__(16) float seg[];
  __shared__ QuantRed<kQuantThreads> red;
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t base = m * K + (int64_t)g * Kg;
  stage_segment<T>(x + base, Kg, seg);
  SegMoments mom; float xlo, xhi;
  segment_moments<kQuantThreads>(seg, Kg, ln_eps, red, mom, xlo, xhi);
  const double lo = ((double)xlo - mom.mean) * mom.rstd, hi = ((double)xhi - mom.mean) * mom.rstd;
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const QuantMap map = make_quant_map(mode, mom, gam, et, fmaxf(fabsf(xlo), fabsf(xhi)));
  if (threadIdx.x == 0) {
    gamma[m * G + g] = (float)gam;
    if (eta) eta[m * G + g] = (float)et;
  }
  int8_t* dst = x_q + base;
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    const float4 a = *reinterpret_cast<const float4*>(seg + k);
    const float4 b = *reinterpret_cast<const float4*>(seg + k + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    *reinterpret_cast<uint2*>(dst + k) = quant_pack8(v, map);
  }
}

__global__ void init_scope(TensorScope* sc) {
  const int g = threadIdx.x;
  if (g < BL_MAX_GROUPS) { sc->enc_min[g] = ~0ull; sc->enc_max[g] = 0ull; }
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
tensor_stats(const T* __restrict__ x, int64_t K, int G, float ln_eps, TensorScope* sc,
             SegRecord* __restrict__ recs) {
  extern __shared__ __align__(16) float seg[];
  __shared__ QuantRed<kQuantThreads> red;
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  stage_segment<T>(x + m * K + (int64_t)g * Kg, Kg, seg);
  SegMoments mom; float xlo, xhi;
  segment_moments<kQuantThreads>(seg, Kg, ln_eps, red, mom, xlo, xhi);
  if (threadIdx.x == 0) {
    recs[blockIdx.x] = SegRecord{mom.mean, mom.rstd, fmaxf(fabsf(xlo), fabsf(xhi)), 0.f};
    atomicMin(&sc->enc_min[g], enc_ordered64(((double)xlo - mom.mean) * mom.rstd));
    atomicMax(&sc->enc_max[g], enc_ordered64(((double)xhi - mom.mean) * mom.rstd));
  }
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
tensor_codes(const T* __restrict__ x, int64_t K, int G, int mode, const TensorScope* __restrict__ sc,
             const SegRecord* __restrict__ recs, int8_t* __restrict__ x_q,
             float* __restrict__ gamma, float* __restrict__ eta) {
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t base = m * K + (int64_t)g * Kg;
  const SegRecord rec = recs[blockIdx.x];
  const double lo = dec_ordered64(sc->enc_min[g]), hi = dec_ordered64(sc->enc_max[g]);
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const QuantMap map = make_quant_map(mode, SegMoments{rec.mean, rec.rstd}, gam, et, rec.xabs);
  if (m == 0 && threadIdx.x == 0) {
    gamma[g] = (float)gam;
    if (eta) eta[g] = (float)et;
  }
  const T* src = x + base;
  int8_t* dst = x_q + base;
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    float v[8];
    Elem<T>::load8(src + k, v);
    *reinterpret_cast<uint2*>(dst + k) = quant_pack8(v, map);
  }
}


// ================================================================================================
// Fast path: one warp per (token, group) segment, the whole segment held in registers.
//
// Used when a segment fits 16 x 16 bytes per lane (K_g <= 4096 for 16-bit inputs, <= 2048 for
// fp32), which covers every shape of the paper's model table.  A warp issues all loads of its
// segment at once (up to 8 KB in flight per warp, 16 warps per SM), then takes the two LN passes
// and the quantisation out of registers with warp shuffles only: no shared memory, no block
// barrier.  Sums are fp32 inside a lane and fp64 across lanes; the second pass sums squared
// deviations from the fp32-rounded mean and corrects for that rounding exactly.  Reciprocals and
// the inverse square root are hardware seeds refined by Newton steps in fp64 (below one ulp of
// fp64 after two steps), which keeps fp64 division and square-root routines out of the kernels.
constexpr int kRowWarps = 8;
constexpr int kRowRegs = 16;                                  // uint4 per lane
constexpr float kRoundMagic = 12582912.f;                     // 1.5 * 2^23: x + magic - magic = rne(x), |x| < 2^22

template <typename T> struct RowTraits {                      // chunk = 8 consecutive elements
  static constexpr int kVecPerChunk = sizeof(T) == 4 ? 2 : 1;
  static constexpr int kChunks = kRowRegs / kVecPerChunk;     // chunks per lane
  static constexpr int kMaxKg = kChunks * 32 * 8;
};

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

template <typename T>
__device__ __forceinline__ void row_load(const T* __restrict__ src, int nchunks, int lane, uint4 (&raw)[kRowRegs]) {
  constexpr int V = RowTraits<T>::kVecPerChunk;
#pragma unroll
  for (int i = 0; i < RowTraits<T>::kChunks; ++i) {
    const int c = lane + 32 * i;
#pragma unroll
    for (int j = 0; j < V; ++j) {
      raw[i * V + j] = make_uint4(0u, 0u, 0u, 0u);
      if (c < nchunks) raw[i * V + j] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)c * 8) + j);
    }
  }
}

template <typename T> __device__ __forceinline__ void row_unpack(const uint4 (&raw)[kRowRegs], int i, float (&v)[8]);
template <> __device__ __forceinline__ void row_unpack<float>(const uint4 (&raw)[kRowRegs], int i, float (&v)[8]) {
  const uint4 a = raw[2 * i], b = raw[2 * i + 1];
  v[0] = __uint_as_float(a.x); v[1] = __uint_as_float(a.y); v[2] = __uint_as_float(a.z); v[3] = __uint_as_float(a.w);
  v[4] = __uint_as_float(b.x); v[5] = __uint_as_float(b.y); v[6] = __uint_as_float(b.z); v[7] = __uint_as_float(b.w);
}
template <> __device__ __forceinline__ void row_unpack<__half>(const uint4 (&raw)[kRowRegs], int i, float (&v)[8]) {
  const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
    v[2 * j] = f.x; v[2 * j + 1] = f.y;
  }
}
template <> __device__ __forceinline__ void row_unpack<__nv_bfloat16>(const uint4 (&raw)[kRowRegs], int i, float (&v)[8]) {
  const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    v[2 * j] = __uint_as_float(w[j] << 16);
    v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
  }
}

struct RowStats { double mean, rstd; float xlo, xhi; };

template <typename H2> __device__ __forceinline__ H2 as_h2(uint32_t w) { return *reinterpret_cast<H2*>(&w); }
template <typename H2> __device__ __forceinline__ uint32_t h2_bits(H2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// Eq. 12 statistics of the segment held in raw[]: every lane returns the same values.
// One pass: deviations are taken from a pilot value c (the mean of the segment's first 8
// elements), which keeps sum (x - c) and sum (x - c)^2 small and well conditioned:
//   mean = c + sum (x - c) / K,   Var = sum (x - c)^2 / K - (mean - c)^2.
template <typename T>
__device__ __forceinline__ RowStats row_stats(const uint4 (&raw)[kRowRegs], int nchunks, int lane, float ln_eps,
                                              double inv_kg) {
  float pilot = 0.f;
  {
    float v[8];
    row_unpack<T>(raw, 0, v);                        // lane 0 holds chunk 0
    pilot = 0.125f * (((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7])));
    pilot = __shfl_sync(0xFFFFFFFFu, pilot, 0);
    if (ln_eps < 0.f) pilot = 0.f;
  }
  float s = 0.f, q = 0.f, mn = INFINITY, mx = -INFINITY;
  uint32_t plo = 0, phi = 0;
  bool have16 = false;
#pragma unroll
  for (int i = 0; i < RowTraits<T>::kChunks; ++i) {
    if (lane + 32 * i < nchunks) {
      float v[8];
      row_unpack<T>(raw, i, v);
      float d[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) d[j] = v[j] - pilot;
      s += ((d[0] + d[1]) + (d[2] + d[3])) + ((d[4] + d[5]) + (d[6] + d[7]));
      float p = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) p = fmaf(d[j], d[j], p);
      q += p;
      if constexpr (sizeof(T) == 4) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { mn = fminf(mn, v[j]); mx = fmaxf(mx, v[j]); }
      } else {
        using H2 = typename std::conditional<std::is_same<T, __half>::value, __half2, __nv_bfloat162>::type;
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
        H2 a = __hmin2(__hmin2(as_h2<H2>(w[0]), as_h2<H2>(w[1])), __hmin2(as_h2<H2>(w[2]), as_h2<H2>(w[3])));
        H2 b = __hmax2(__hmax2(as_h2<H2>(w[0]), as_h2<H2>(w[1])), __hmax2(as_h2<H2>(w[2]), as_h2<H2>(w[3])));
        if (have16) { a = __hmin2(a, as_h2<H2>(plo)); b = __hmax2(b, as_h2<H2>(phi)); }
        plo = h2_bits(a); phi = h2_bits(b); have16 = true;
      }
    }
  }
  if constexpr (sizeof(T) != 4) {
    if (have16) {
      using H2 = typename std::conditional<std::is_same<T, __half>::value, __half2, __nv_bfloat162>::type;
      const H2 a = as_h2<H2>(plo), b = as_h2<H2>(phi);
      if constexpr (std::is_same<T, __half>::value) {
        const float2 fa = __half22float2(a), fb = __half22float2(b);
        mn = fminf(fa.x, fa.y); mx = fmaxf(fb.x, fb.y);
      } else {
        const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
        mn = fminf(fa.x, fa.y); mx = fmaxf(fb.x, fb.y);
      }
    }
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
};
__device__ __forceinline__ RowMap row_map(int mode, double mean, double rstd, double gamma, double eta, float xabs) {
  RowMap m;
  m.mean = mean; m.rstd = rstd; m.eta = eta;
  m.scale = gamma > 0.0 ? (double)kQb * rcp_newton(gamma) : 0.0;
  m.A = (float)(rstd * m.scale);
  m.B = (float)(-(mean * rstd + eta) * m.scale);
  m.tau = 4e-7f * (fabsf(m.A) * xabs + fabsf(m.B) + 1.0f);
  m.code_lo = (mode == BL_ABSMAX) ? -kCodeMax : 0;
  return m;
}
// The rare element too close to a rounding tie for fp32: the equations in fp64, in their order.
__device__ __noinline__ int row_code_exact(float x, double mean, double rstd, double eta, double scale) {
  const double xh = ((double)x - mean) * rstd;
  return (int)rint((xh - eta) * scale);
}
__device__ __forceinline__ uint2 row_codes8(const float (&v)[8], const RowMap& m) {
  // f is clipped in fp32 (the clip bounds are integers, so clip and rne commute); adding the
  // magic constant leaves rne(f) as a two's-complement byte in the low bits of the sum.
  uint32_t t[8];
  bool near_tie = false;
  const float lo = (float)m.code_lo, hi = (float)kCodeMax, edge = 0.5f - m.tau;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float f = fmaf(v[j], m.A, m.B);
    const float tj = fminf(fmaxf(f, lo), hi) + kRoundMagic;
    near_tie |= fabsf(f - (tj - kRoundMagic)) > edge;         // inside the clip range: within tau of a tie
    t[j] = __float_as_uint(tj);
  }
  uint2 out;
  out.x = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
  out.y = __byte_perm(__byte_perm(t[4], t[5], 0x0040), __byte_perm(t[6], t[7], 0x0040), 0x5410);
  if (near_tie) {                                            // rare: redo the 8 codes exactly
    uint32_t w[2] = {0u, 0u};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int c = max(m.code_lo, min(kCodeMax, row_code_exact(v[j], m.mean, m.rstd, m.eta, m.scale)));
      w[j >> 2] |= (uint32_t)(c & 0xFF) << (8 * (j & 3));
    }
    out = make_uint2(w[0], w[1]);
  }
  return out;
}

template <typename T>
__device__ __forceinline__ void row_store_codes(const uint4 (&raw)[kRowRegs], int nchunks, int lane, const RowMap& map,
                                                int8_t* __restrict__ dst) {
#pragma unroll
  for (int i = 0; i < RowTraits<T>::kChunks; ++i) {
    const int c = lane + 32 * i;
    if (c < nchunks) {
      float v[8];
      row_unpack<T>(raw, i, v);
      *reinterpret_cast<uint2*>(dst + (size_t)c * 8) = row_codes8(v, map);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 2)
rows_per_token(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, int mode, float ln_eps,
               double inv_kg, int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  const int lane = threadIdx.x & 31;
  const int64_t seg = (int64_t)blockIdx.x * kRowWarps + (threadIdx.x >> 5);
  if (seg >= segments) return;                                   // whole warp
  const int64_t base = (seg / G) * K + (seg % G) * (int64_t)Kg;
  const int nchunks = Kg / 8;
  uint4 raw[kRowRegs];
  row_load<T>(x + base, nchunks, lane, raw);
  const RowStats st = row_stats<T>(raw, nchunks, lane, ln_eps, inv_kg);
  const double lo = ((double)st.xlo - st.mean) * st.rstd, hi = ((double)st.xhi - st.mean) * st.rstd;
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const RowMap map = row_map(mode, st.mean, st.rstd, gam, et, fmaxf(fabsf(st.xlo), fabsf(st.xhi)));
  if (lane == 0) {
    gamma[seg] = (float)gam;
    if (eta) eta[seg] = (float)et;
  }
  row_store_codes<T>(raw, nchunks, lane, map, x_q + base);
}

template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 3)
rows_tensor_stats(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, float ln_eps, double inv_kg,
                  TensorScope* sc, SegRecord* __restrict__ recs) {
  const int lane = threadIdx.x & 31;
  const int64_t seg = (int64_t)blockIdx.x * kRowWarps + (threadIdx.x >> 5);
  if (seg >= segments) return;
  const int g = (int)(seg % G);
  const int64_t base = (seg / G) * K + g * (int64_t)Kg;
  const int nchunks = Kg / 8;
  uint4 raw[kRowRegs];
  row_load<T>(x + base, nchunks, lane, raw);
  const RowStats st = row_stats<T>(raw, nchunks, lane, ln_eps, inv_kg);
  if (lane == 0) {
    recs[seg] = SegRecord{st.mean, st.rstd, fmaxf(fabsf(st.xlo), fabsf(st.xhi)), 0.f};
    atomicMin(&sc->enc_min[g], enc_ordered64(((double)st.xlo - st.mean) * st.rstd));
    atomicMax(&sc->enc_max[g], enc_ordered64(((double)st.xhi - st.mean) * st.rstd));
  }
}

template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 2)
rows_tensor_codes(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, int mode,
                  const TensorScope* __restrict__ sc, const SegRecord* __restrict__ recs,
                  int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  const int lane = threadIdx.x & 31;
  const int64_t seg = (int64_t)blockIdx.x * kRowWarps + (threadIdx.x >> 5);
  if (seg >= segments) return;
  const int g = (int)(seg % G);
  const int64_t base = (seg / G) * K + g * (int64_t)Kg;
  const int nchunks = Kg / 8;
  uint4 raw[kRowRegs];
  row_load<T>(x + base, nchunks, lane, raw);                      // in flight during the scalar work below
  const SegRecord rec = recs[seg];
  const double lo = dec_ordered64(sc->enc_min[g]), hi = dec_ordered64(sc->enc_max[g]);
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const RowMap map = row_map(mode, rec.mean, rec.rstd, gam, et, rec.xabs);
  if (seg < G && lane == 0) {                                      // token 0 reports the scope's gamma / eta
    gamma[g] = (float)gam;
    if (eta) eta[g] = (float)et;
  }
  row_store_codes<T>(raw, nchunks, lane, map, x_q + base);
}

template <typename T>
cudaError_t run(const QuantArgs& a, cudaStream_t s) {
  const T* x = reinterpret_cast<const T*>(a.x);
  const int64_t Kg = a.K / a.G;
  const size_t smem = (size_t)Kg * sizeof(float);
  const unsigned grid = (unsigned)(a.M * a.G);
  cudaError_t e;
  if (Kg <= RowTraits<T>::kMaxKg) {                              // a segment fits a warp's registers
    const int64_t segments = a.M * a.G;
    const unsigned rgrid = (unsigned)((segments + kRowWarps - 1) / kRowWarps);
    const double inv_kg = 1.0 / (double)Kg;
    if (a.gran == BL_PER_TOKEN) {
      rows_per_token<T><<<rgrid, kRowWarps * 32, 0, s>>>(x, segments, a.K, a.G, (int)Kg, (int)a.mode, a.ln_eps,
                                                         inv_kg, a.x_q, a.gamma, a.eta);
      return cudaGetLastError();
    }
    TensorScope* sc = reinterpret_cast<TensorScope*>(a.ws);
    SegRecord* recs = reinterpret_cast<SegRecord*>(reinterpret_cast<char*>(a.ws) + sizeof(TensorScope));
    init_scope<<<1, BL_MAX_GROUPS, 0, s>>>(sc);
    rows_tensor_stats<T><<<rgrid, kRowWarps * 32, 0, s>>>(x, segments, a.K, a.G, (int)Kg, a.ln_eps, inv_kg, sc, recs);
    rows_tensor_codes<T><<<rgrid, kRowWarps * 32, 0, s>>>(x, segments, a.K, a.G, (int)Kg, (int)a.mode, sc, recs,
                                                          a.x_q, a.gamma, a.eta);
    return cudaGetLastError();
  }
  if (a.gran == BL_PER_TOKEN) {
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(quant_per_token<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    quant_per_token<T><<<grid, kQuantThreads, smem, s>>>(x, a.K, a.G, (int)a.mode, a.ln_eps, a.x_q,
                                                        a.gamma, a.eta);
    return cudaGetLastError();
  }
  TensorScope* sc = reinterpret_cast<TensorScope*>(a.ws);
  SegRecord* recs = reinterpret_cast<SegRecord*>(reinterpret_cast<char*>(a.ws) + sizeof(TensorScope));
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(tensor_stats<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  init_scope<<<1, BL_MAX_GROUPS, 0, s>>>(sc);
  tensor_stats<T><<<grid, kQuantThreads, smem, s>>>(x, a.K, a.G, a.ln_eps, sc, recs);
  tensor_codes<T><<<grid, kQuantThreads, 0, s>>>(x, a.K, a.G, (int)a.mode, sc, recs, a.x_q, a.gamma, a.eta);
  return cudaGetLastError();
}

}  // namespace

size_t quant_ws_bytes(int64_t M, int G) {
  return sizeof(TensorScope) + (size_t)M * (size_t)G * sizeof(SegRecord);
}

// ---- built-in scratch of bitlinear_quant_act_noalloc -------------------------------------------
// Room for the per-tensor statistics of up to BL_NOALLOC_MAX_SEGMENTS (token, group) segments.
// The array lives in the library image: every GPU that loads the library holds these bytes until
// the process exits.  Host code must not hand the symbol itself to a kernel (on the host the name
// is only a stand-in); it asks the runtime for the device address once per device.
constexpr size_t kNoAllocBytes = sizeof(TensorScope) + (size_t)BL_NOALLOC_MAX_SEGMENTS * sizeof(SegRecord);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Device address of the built-in scratch on the current device (cached per device ordinal).
static cudaError_t noalloc_scratch_address(void** out) {
  constexpr int kMaxDevices = 64;
  static void* cached[kMaxDevices] = {};
  static std::mutex guard;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(guard);
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    cached[dev] = p;
  }
  *out = cached[dev];
  return cudaSuccess;
}

cudaError_t launch_quant_act(const QuantArgs& a, cudaStream_t s) {
  switch (a.xt) {
    case BL_F32: return run<float>(a, s);
    case BL_F16: return run<__half>(a, s);
    case BL_BF16: return run<__nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl

extern "C" bl_status bitlinear_quant_act_noalloc(const void* x, bl_dtype xt, int64_t M, int64_t K, int G, int b,
                                                 bl_quant_mode mode, bl_gran gran, float ln_eps, int8_t* x_q,
                                                 float* gamma, float* eta, void* stream) {
  // Refuse what the built-in scratch cannot hold before anything else is looked at.
  if (M > 0 && G > 0 && gran == BL_PER_TENSOR && M * (int64_t)G > (int64_t)BL_NOALLOC_MAX_SEGMENTS)
    return BL_ERR_TOO_LARGE;
  void* scratch = nullptr;
  if (bl::noalloc_scratch_address(&scratch) != cudaSuccess) return BL_ERR_CUDA;
  // Same validation and the same kernels as bitlinear_quant_act, with the scratch passed as its
  // workspace.  tensor_stats rewrites every record it later reads and init_scope resets the
  // running extremes, so nothing of an earlier call survives into this one.
  return bitlinear_quant_act(x, xt, M, K, G, b, mode, gran, ln_eps, x_q, gamma, eta, scratch,
                             bl::kNoAllocBytes, stream);
}

