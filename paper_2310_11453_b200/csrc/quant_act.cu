// Steps 1-2 of BitLinear: LN per token and group (Eq. 12, 15) fused with the 8-bit activation
// quantisation (Eq. 4-6, 14).  HBM-bound: x is read once (per token) or twice (per tensor) with
// 128-bit loads; the normalised row is never written to HBM.
//
// One CTA per (token m, group g) segment of K_g features, staged in shared memory as fp32:
//   moments  sum, raw min/max, then sum of squared deviations      (quant_core.cuh)
//   codes    one FMA + round per element, 8 codes per 8-byte store
// Per-tensor scope splits in two kernels: the first leaves each segment's moments in the
// workspace and folds the extremes of x^ into a global atomic min/max on an order-preserving
// encoding (order-independent, hence deterministic); the second re-reads x and writes codes.
#include <mutex>

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

template <typename T>
cudaError_t run(const QuantArgs& a, cudaStream_t s) {
  const T* x = reinterpret_cast<const T*>(a.x);
  const int64_t Kg = a.K / a.G;
  const size_t smem = (size_t)Kg * sizeof(float);
  const unsigned grid = (unsigned)(a.M * a.G);
  cudaError_t e;
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

