// Step 4 of BitLinear on CUDA cores: acc = W~ x~ (Eq. 7) with dp4a, for the CANONICAL bit
// layout and any shape.  This is the shape-general path (small or ragged problems) and the
// second, independent GPU implementation the tensor-core kernel is diffed against at full
// size; it is not the fast path.  64x64 output tile per CTA, 64 weights per K step; the
// packed bits are expanded to +-1 bytes in shared memory.  Optionally fuses the Eq. 11 rescale.
#include "common.cuh"

namespace bl {

namespace {

constexpr int kTile = 64;        // outputs per CTA along m and n
constexpr int kStepK = 64;       // weights per K step (16 dp4a words)
constexpr int kWords = kStepK / 4;

// 4 sign bits (LSB first) -> 4 bytes, +1 = 0x01, -1 = 0xFF.
__device__ __forceinline__ uint32_t expand4(uint32_t nib) {
  const uint32_t t = (nib * 0x00204081u) & 0x01010101u;
  return 0xFFFFFFFFu ^ (t * 0xFEu);
}

template <bool kDequant, typename TY>
__global__ void __launch_bounds__(256)
gemm_simple_kernel(GemmArgs a) {
  __shared__ uint32_t xs[kTile][kWords + 1];
  __shared__ uint32_t wsm[kTile][kWords + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * kTile, n0 = (int64_t)blockIdx.x * kTile;
  const int64_t Kg = a.K / a.G, Kb = a.K / 8;
  int acc[4][4];
  float fsum[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0; fsum[i][j] = 0.f; }

  for (int g = 0; g < a.G; ++g) {
    const int64_t kend = (int64_t)(g + 1) * Kg;
    for (int64_t k0 = (int64_t)g * Kg; k0 < kend; k0 += kStepK) {
      // codes: 64 rows x 8 chunks of 8 bytes
      for (int idx = threadIdx.x; idx < kTile * 8; idx += 256) {
        const int r = idx >> 3, c = idx & 7;
        const int64_t m = m0 + r, k = k0 + c * 8;
        uint2 v = make_uint2(0u, 0u);
        if (m < a.M && k < kend) v = __ldg(reinterpret_cast<const uint2*>(a.x_q + m * a.K + k));
        xs[r][2 * c] = v.x; xs[r][2 * c + 1] = v.y;
      }
      // weights: 64 rows x 8 packed bytes -> 16 words of +-1
      for (int idx = threadIdx.x; idx < kTile * 8; idx += 256) {
        const int r = idx >> 3, c = idx & 7;
        const int64_t n = n0 + r, k = k0 + c * 8;
        uint32_t byte = 0;
        if (n < a.N && k < kend) byte = __ldg(a.W_packed + n * Kb + (k >> 3));
        wsm[r][2 * c] = expand4(byte & 15u); wsm[r][2 * c + 1] = expand4(byte >> 4);
      }
      __syncthreads();
#pragma unroll
      for (int kw = 0; kw < kWords; ++kw) {
        int xa[4], wb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) xa[i] = (int)xs[ty * 4 + i][kw];
#pragma unroll
        for (int j = 0; j < 4; ++j) wb[j] = (int)wsm[tx * 4 + j][kw];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(xa[i], wb[j], acc[i][j]);
      }
      __syncthreads();
    }
    // fold this group
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t m = m0 + ty * 4 + i;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int64_t n = n0 + tx * 4 + j;
        if (m < a.M && n < a.N) {
          if (kDequant) {
            const int64_t sc = (a.gran == BL_PER_TOKEN) ? m * a.G + g : g;
            const bool corr = a.eta_correction != 0;
            const int64_t bb = a.beta_rows > 0 ? n / a.beta_rows : 0;
            fsum[i][j] += dequant_term(acc[i][j], a.beta[bb * a.G + g], a.gamma[sc], corr ? a.eta[sc] : 0.f,
                                       corr ? a.rowsum[n * a.G + g] : 0, corr);
          } else {
            a.acc[((int64_t)g * a.M + m) * a.N + n] = acc[i][j];
          }
        }
        acc[i][j] = 0;
      }
    }
  }
  if (kDequant) {
    TY* y = reinterpret_cast<TY*>(a.y);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t m = m0 + ty * 4 + i;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int64_t n = n0 + tx * 4 + j;
        if (m < a.M && n < a.N) {
          float v = fsum[i][j];
          if (a.relu) v = fmaxf(v, 0.f);
          if (a.residual) v += in_cast(reinterpret_cast<const TY*>(a.residual)[m * a.ld_res + n]);
          y[m * (a.ld_y > 0 ? a.ld_y : a.N) + n] = out_cast<TY>(v);
        }
      }
    }
  }
}

}  // namespace

cudaError_t launch_gemm_simple(const GemmArgs& a, cudaStream_t s) {
  dim3 grid((unsigned)((a.N + kTile - 1) / kTile), (unsigned)((a.M + kTile - 1) / kTile));
  if (a.y == nullptr) {
    gemm_simple_kernel<false, float><<<grid, 256, 0, s>>>(a);
  } else {
    switch (a.yt) {
      case BL_F32: gemm_simple_kernel<true, float><<<grid, 256, 0, s>>>(a); break;
      case BL_F16: gemm_simple_kernel<true, __half><<<grid, 256, 0, s>>>(a); break;
      case BL_BF16: gemm_simple_kernel<true, __nv_bfloat16><<<grid, 256, 0, s>>>(a); break;
    }
  }
  return cudaGetLastError();
}

}  // namespace bl
