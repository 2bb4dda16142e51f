// Batch-1 decode: LN + Quant of the single token (Eq. 12, 4-6) and the 1-bit x 8-bit product
// with its rescale (Eq. 7, 11) in one kernel.  Bound by streaming the packed weights
// (N*K/8 bytes) once from HBM; everything else is a few KB.
//
// Every CTA first normalises and quantises x itself (K values, L2-resident) - cheaper than a
// separate launch and a round trip through HBM.  Then each warp owns a 4096-weight slice of
// K: its lane keeps the 128 codes of "its" chunk in registers, so per row a lane issues one
// 16-byte weight load and 32 dp4a on {0,1}-expanded bits:
//     sum_k W~[n,k] x~[k] = 2 * sum_{bit=1} x~[k] - sum_k x~[k].
// DECODE layout: row-major like CANONICAL, but inside every 32-weight word weight q sits at bit
// q/4 + 8*(q%4), so (word >> j) & 0x01010101 is the 0/1 byte mask of weights 4j..4j+3.
#include "quant_core.cuh"

namespace bl {

namespace {

constexpr int kGemvThreads = 512;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kRowsPerIter = 4;          // rows in flight per warp (independent 16-byte loads)
constexpr int kSlice = 4096;             // weights per warp slice = 32 lanes x 128

struct GemvShared {
  QuantRed<kGemvThreads> red;
  float gamma[BL_MAX_GROUPS];
  float eta[BL_MAX_GROUPS];
  float partial[kGemvWarps][kRowsPerIter];
};

template <typename TX, typename TY>
__global__ void __launch_bounds__(kGemvThreads)
gemv_decode_kernel(GemvArgs a, int rows_per_cta) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ GemvShared sh;
  float* xf = reinterpret_cast<float*>(smem_raw);                      // [K] raw, then x^
  int8_t* codes = reinterpret_cast<int8_t*>(smem_raw + a.K * sizeof(float));  // [K]
  const int K = (int)a.K, G = a.G, Kg = K / G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const TX* x = reinterpret_cast<const TX*>(a.x);

  // ---- steps 1-2 on the token: LN per group, gamma/eta, codes --------------------------------
  for (int k = threadIdx.x * 8; k < K; k += kGemvThreads * 8) {
    float v[8];
    Elem<TX>::load8(x + k, v);
    *reinterpret_cast<float4*>(xf + k) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(xf + k + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  __syncthreads();
  for (int g = 0; g < G; ++g) {
    const float* seg = xf + g * Kg;
    SegMoments mom; float xlo, xhi;
    segment_moments<kGemvThreads>(seg, Kg, a.ln_eps, sh.red, mom, xlo, xhi);
    const double lo = ((double)xlo - mom.mean) * mom.rstd, hi = ((double)xhi - mom.mean) * mom.rstd;
    double gam, et;
    scope_gamma_eta((int)a.mode, lo, hi, gam, et);
    const QuantMap map = make_quant_map((int)a.mode, mom, gam, et, fmaxf(fabsf(xlo), fabsf(xhi)));
    if (threadIdx.x == 0) { sh.gamma[g] = (float)gam; sh.eta[g] = (float)et; }
    for (int k = threadIdx.x * 8; k < Kg; k += kGemvThreads * 8) {
      const float4 p = *reinterpret_cast<const float4*>(seg + k);
      const float4 q = *reinterpret_cast<const float4*>(seg + k + 4);
      const float v[8] = {p.x, p.y, p.z, p.w, q.x, q.y, q.z, q.w};
      *reinterpret_cast<uint2*>(codes + g * Kg + k) = quant_pack8(v, map);
    }
  }
  __syncthreads();

  // ---- this lane's 128 codes and their sum ---------------------------------------------------
  const int nslices = (K + kSlice - 1) / kSlice;       // warps that share one row
  const int slice = warp % nslices, rowslot = warp / nslices;
  const int rowslots = kGemvWarps / nslices;           // rows handled side by side
  const int chunk = slice * 32 + lane;                 // 128-weight chunk of this lane
  const bool active = chunk * 128 < K && rowslot < rowslots;
  uint32_t xr[32];
  int csum = 0;
  float lane_scale = 0.f;
  if (active) {
    const uint4* src = reinterpret_cast<const uint4*>(codes + chunk * 128);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint4 v = src[i];
      xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) csum = __dp4a((int)xr[i], 0x01010101, csum);
    const int g = (chunk * 128) / Kg;
    lane_scale = a.beta[g] * sh.gamma[g] * kInvQb;
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) xr[i] = 0;
  }

  // ---- stream the rows of this CTA ------------------------------------------------------------
  const int64_t row_begin = (int64_t)blockIdx.x * rows_per_cta;
  const int64_t row_end = min((int64_t)a.N, row_begin + rows_per_cta);
  const int64_t Kb = a.K / 8;
  TY* y = reinterpret_cast<TY*>(a.y);
  const int rows_per_iter = rowslots * kRowsPerIter;
  for (int64_t base = row_begin; base < row_end; base += rows_per_iter) {
    uint4 bits[kRowsPerIter];
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) {
      const int64_t n = base + rowslot * kRowsPerIter + r;
      bits[r] = make_uint4(0u, 0u, 0u, 0u);
      if (active && n < row_end)
        bits[r] = __ldcs(reinterpret_cast<const uint4*>(a.W_packed + n * Kb + (int64_t)chunk * 16));
    }
#pragma unroll
    for (int r = 0; r < kRowsPerIter; ++r) {
      const uint32_t w[4] = {bits[r].x, bits[r].y, bits[r].z, bits[r].w};
      int accb = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int j = 0; j < 8; ++j)
          accb = __dp4a((int)((w[q] >> j) & 0x01010101u), (int)xr[q * 8 + j], accb);
      const int acc = 2 * accb - csum;                 // Eq. 7 over this lane's chunk
      float part;
      if (G == 1) part = (float)warp_sum(active ? acc : 0) * lane_scale;
      else part = warp_sum(active ? (float)acc * lane_scale : 0.f);
      if (lane == 0) sh.partial[warp][r] = part;
    }
    __syncthreads();
    // fold the K slices of each row and write y (one thread per row of this iteration)
    if (threadIdx.x < rows_per_iter) {
      const int rs = threadIdx.x / kRowsPerIter, r = threadIdx.x % kRowsPerIter;
      const int64_t n = base + rs * kRowsPerIter + r;
      if (n < row_end) {
        float v = 0.f;
        for (int s = 0; s < nslices; ++s) v += sh.partial[rs * nslices + s][r];
        if (a.eta_correction) {
          for (int g = 0; g < G; ++g) v += sh.eta[g] * a.beta[g] * (float)a.rowsum[n * G + g];
        }
        y[n] = out_cast<TY>(v);
      }
    }
    __syncthreads();
  }
}

template <typename TX, typename TY>
cudaError_t run2(const GemvArgs& a, cudaStream_t s) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = (size_t)a.K * (sizeof(float) + 1);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(gemv_decode_kernel<TX, TY>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int nslices = (int)((a.K + kSlice - 1) / kSlice);
  const int unit = (kGemvWarps / nslices) * kRowsPerIter;
  int64_t rows_per_cta = (a.N + sms - 1) / sms;
  rows_per_cta = (rows_per_cta + unit - 1) / unit * unit;
  const unsigned grid = (unsigned)((a.N + rows_per_cta - 1) / rows_per_cta);
  gemv_decode_kernel<TX, TY><<<grid, kGemvThreads, smem, s>>>(a, (int)rows_per_cta);
  return cudaGetLastError();
}

template <typename TX>
cudaError_t run1(const GemvArgs& a, cudaStream_t s) {
  switch (a.yt) {
    case BL_F32: return run2<TX, float>(a, s);
    case BL_F16: return run2<TX, __half>(a, s);
    case BL_BF16: return run2<TX, __nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_gemv_decode(const GemvArgs& a, cudaStream_t s) {
  switch (a.xt) {
    case BL_F32: return run1<float>(a, s);
    case BL_F16: return run1<__half>(a, s);
    case BL_BF16: return run1<__nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl
