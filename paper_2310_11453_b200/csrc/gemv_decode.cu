// Batch-1 decode: LN + Quant of the single token (Eq. 12, 4-6) and the 1-bit x 8-bit product
// with its rescale (Eq. 7, 11) in one kernel.  Bound by streaming the packed weights
// (N*K/8 bytes) once from HBM; everything else is a few KB.
//
// Shape of one call.  The grid splits the N rows evenly over the SMs.  A CTA
//   1. asks the L2 to fetch its slice of the packed weights (prefetch.global.L2), tells the
//      runtime that the next kernel on the stream may start (programmatic dependent launch),
//      and only then waits for everything earlier on the stream (griddepcontrol.wait).  The
//      prefetch has no architectural effect, so stream order is kept for all data, while the
//      weights of the next calls already travel from HBM to L2 during this call;
//   2. loads x, issues the 16-byte loads of its first rows, then normalises and quantises x
//      itself (K values, one pass: sums of x and x^2, raw extremes; cheaper than a separate
//      launch and a round trip through HBM).  The codes do not depend on the variance:
//      rne((x^ - eta) Q_b / gamma) = rne((x - c) A) with c = mean, A = Q_b / max|x - mean| for
//      absmax and c = min x, A = Q_b / (max x - min x) for the eta form, so the chain from x to
//      the codes is one block reduction, one reciprocal and one FMA per element; gamma and
//      eta (which do need 1/sqrt(Var + eps)) are only used by the final rescale;
//   3. per row, each lane multiplies its 128-weight chunk with the 128 codes it keeps in
//      registers: sum_k W~[n,k] x~[k] = 2 * sum_{bit=1} x~[k] - sum_k x~[k].  Rows come in
//      batches of up to 7 per warp; a row's register is reloaded with the next batch's row as
//      soon as the row has been used.
//
// DECODE layout: row-major like CANONICAL, but inside every 32-weight word weight q sits at bit
// q/4 + 8*(q%4).  Then word & (0x01010101 << j) holds weights 4j..4j+3 as bytes that are 0 or
// 2^j, and one dp4a against the matching four codes adds 2^j * (their masked sum): two
// instructions per four weights (a logic op and a dot product, on different pipes).  The
// eight partial sums of a chunk are folded as sum_j acc_j * 2^(7-j) = 128 * (masked sum).
#include "quant_core.cuh"

namespace bl {

namespace {

#ifndef BL_GEMV_THREADS
#define BL_GEMV_THREADS 256
#endif
constexpr int kGemvThreads = BL_GEMV_THREADS;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kBatchRows = 7;            // rows per warp and batch (two batches live in registers)
constexpr int kSlice = 4096;             // weights per warp slice = 32 lanes x 128
constexpr float kRoundMagic = 12582912.f;   // 1.5 * 2^23: x + magic - magic is rne(x) for |x| < 2^22

struct GemvShared {
  float s1[kGemvWarps], s2[kGemvWarps];
  float lo[kGemvWarps], hi[kGemvWarps];
  float gamma[BL_MAX_GROUPS];
  float eta[BL_MAX_GROUPS];
  float partial[2][kGemvWarps][8];
};

// Where the code of feature k sits in shared memory: inside each 4096-feature slice the 16-byte
// pieces are stored piece-major ([piece 0..7][chunk 0..31]), so that the 32 lanes of a warp,
// which own consecutive 128-feature chunks, read piece i of their chunks from consecutive
// 16-byte slots (no bank conflicts).
__device__ __forceinline__ int code_slot(int k) {
  return (k & ~(kSlice - 1)) | ((((k >> 4) & 7) * 32 + ((k >> 7) & 31)) << 4) | (k & 15);
}

// 1/sqrt(v) to fp32 accuracy (it only scales the output); exact routine outside the fp32 range.
__device__ __forceinline__ float rsqrt_scale(double v) {
  if (!(v > 1e-30 && v < 1e30)) return v > 0.0 ? (float)(1.0 / sqrt(v)) : 0.f;
  const float f = (float)v;
  float y = rsqrtf(f);
  return y * (1.5f - 0.5f * f * y * y);
}
// The rare element whose fp32 image is too close to a rounding tie: redone in fp64.  Kept out of
// line so that the common path carries no fp64 instructions.
__device__ __noinline__ int code_slow_path(float x, double c, double span) {
  return (int)rint(((double)x - c) * ((double)kQb / span));
}

// 128 * sum over this lane's chunk of bit * code, for one row.
__device__ __forceinline__ int chunk_dot128(const uint4& bits, const uint32_t (&xr)[32]) {
  const uint32_t w[4] = {bits.x, bits.y, bits.z, bits.w};
  int acc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) acc[j] = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q)
#pragma unroll
    for (int j = 0; j < 8; ++j)
      acc[j] = __dp4a((int)(w[q] & (0x01010101u << j)), (int)xr[q * 8 + j], acc[j]);
  // acc[j] = 2^j * S_j for j < 7 and -128 * S_7 (the byte 0x80 is -128 as a signed operand)
  int t = -acc[7];
#pragma unroll
  for (int j = 0; j < 7; ++j) t += acc[j] * (1 << (7 - j));
  return t;
}

// Sums each of 8 per-lane values over the 32 lanes with 9 shuffles: after the call, lane l
// holds in v[0] the warp total of value number (l >> 2) & 7 (every lane of a quad the same).
template <typename T>
__device__ __forceinline__ void warp_sum8(T (&v)[8], int lane) {
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const T send = b4 ? v[i] : v[i + 4], keep = b4 ? v[i + 4] : v[i];
    v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 16);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const T send = b3 ? v[i] : v[i + 2], keep = b3 ? v[i + 2] : v[i];
    v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 8);
  }
  {
    const T send = b2 ? v[0] : v[1], keep = b2 ? v[1] : v[0];
    v[0] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, 4);
  }
  v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 2);
  v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], 1);
}

// Moments of 8 raw values.  Inside a warp the sums are fp32 (at most K/8 values per lane); the
// eight warp totals are then combined in fp64.  The mean moves a code by about 1e-7 of a step
// at worst this way, and the sum of squares only feeds the output scale.
__device__ __forceinline__ void accumulate8(const float (&v)[8], float& s1, float& s2, float& mn, float& mx) {
  s1 += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
  float p2 = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) { p2 = fmaf(v[i], v[i], p2); mn = fminf(mn, v[i]); mx = fmaxf(mx, v[i]); }
  s2 += p2;
}

struct GemvGeom {            // decided on the host
  int rows_per_cta, rpw, nbatches, nslices, rowslots;
  uint32_t inv_nslices, inv_group_chunks;   // ceil(2^16 / d): (v * inv) >> 16 == v / d for v < 256
  double inv_kg;
};

template <typename TX, typename TY>
__global__ void __launch_bounds__(kGemvThreads, kGemvThreads <= 256 ? 2 : 1)
gemv_decode_kernel(GemvArgs a, GemvGeom geo) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ GemvShared sh;
  float* xf = reinterpret_cast<float*>(smem_raw);                              // [K] raw x
  int8_t* codes = reinterpret_cast<int8_t*>(smem_raw + a.K * sizeof(float));   // [nslices * 4096]
  const int K = (int)a.K, G = a.G, Kg = K / G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t Kb = a.K / 8;
  const int rpw = geo.rpw, nbatches = geo.nbatches, nslices = geo.nslices, rowslots = geo.rowslots;
  const int64_t row_begin = (int64_t)blockIdx.x * geo.rows_per_cta;
  const int64_t row_end = min((int64_t)a.N, row_begin + geo.rows_per_cta);

  // ---- ahead of stream order: pull this CTA's weights towards L2 ---------------------------------
  {
    const char* base = reinterpret_cast<const char*>(a.W_packed) + row_begin * Kb;
    const int64_t bytes = (row_end - row_begin) * Kb;
    for (int64_t off = (int64_t)threadIdx.x * 128; off < bytes; off += (int64_t)kGemvThreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
  }
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- x first (the chain to the codes hangs on it), staged as fp32 ------------------------------
  const TX* x = reinterpret_cast<const TX*>(a.x);
  float s1 = 0.f, s2 = 0.f;
  float mn = INFINITY, mx = -INFINITY;
  for (int k = threadIdx.x * 8; k < K; k += kGemvThreads * 8) {
    float v[8];
    Elem<TX>::load8(x + k, v);
    *reinterpret_cast<float4*>(xf + k) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(xf + k + 4) = make_float4(v[4], v[5], v[6], v[7]);
    if (G == 1) accumulate8(v, s1, s2, mn, mx);
  }

  // ---- work split inside the CTA; first batch of rows: loads in flight during the prologue --------
  const int rowslot = (int)(((uint32_t)warp * geo.inv_nslices) >> 16);   // rows side by side
  const int slice = warp - rowslot * nslices;                            // warps that share a row
  const int chunk = slice * 32 + lane;                                   // 128-weight chunk of this lane
  const bool active = chunk * 128 < K && rowslot < rowslots;
  const int my_group = active ? (int)(((uint32_t)chunk * geo.inv_group_chunks) >> 16) : 0;
  const float beta_mine = __ldg(a.beta + my_group);
  const uint8_t* wlane = a.W_packed + (int64_t)chunk * 16;
  // Row r of batch b for this warp slot; rows past the end read as all-zero bits.
  auto load_row = [&](int b, int r) -> uint4 {
    const int64_t n = row_begin + ((int64_t)b * rowslots + rowslot) * rpw + r;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (active && r < rpw && b < nbatches && n < row_end)
      v = __ldcs(reinterpret_cast<const uint4*>(wlane + n * Kb));
    return v;
  };
  uint4 cur[kBatchRows];
#pragma unroll
  for (int r = 0; r < kBatchRows; ++r) cur[r] = load_row(0, r);

  // ---- steps 1-2 on the token: LN per group, gamma/eta, codes ------------------------------------
  __syncthreads();
  for (int g = 0; g < G; ++g) {
    const float* seg = xf + g * Kg;
    if (G > 1) {
      s1 = 0.f; s2 = 0.f; mn = INFINITY; mx = -INFINITY;
      for (int k = threadIdx.x * 8; k < Kg; k += kGemvThreads * 8) {
        const float4 p = *reinterpret_cast<const float4*>(seg + k);
        const float4 q = *reinterpret_cast<const float4*>(seg + k + 4);
        const float v[8] = {p.x, p.y, p.z, p.w, q.x, q.y, q.z, q.w};
        accumulate8(v, s1, s2, mn, mx);
      }
    }
    s1 = warp_sum(s1); s2 = warp_sum(s2); mn = warp_min(mn); mx = warp_max(mx);
    if (lane == 0) { sh.s1[warp] = s1; sh.s2[warp] = s2; sh.lo[warp] = mn; sh.hi[warp] = mx; }
    __syncthreads();
    double t1 = 0.0;
#pragma unroll
    for (int w = 0; w < kGemvWarps; w += 4)
      t1 += ((double)sh.s1[w] + (double)sh.s1[w + 1]) + ((double)sh.s1[w + 2] + (double)sh.s1[w + 3]);
    float xlo = sh.lo[0], xhi = sh.hi[0];
#pragma unroll
    for (int w = 1; w < kGemvWarps; ++w) { xlo = fminf(xlo, sh.lo[w]); xhi = fmaxf(xhi, sh.hi[w]); }
    // location c and slope A of the code map (see the header).  The fast path only needs fp32
    // images of A and B = -c A (its error is covered by the tie window tau); the exact fp64
    // values are rebuilt inside the slow path.
    const bool ln = a.ln_eps >= 0.f;
    const double mean = ln ? t1 * geo.inv_kg : 0.0;
    const float mean_f = (float)mean;
    const float cf = (a.mode == BL_ABSMAX) ? mean_f : xlo;
    const float span_f = (a.mode == BL_ABSMAX) ? fmaxf(fabsf(xlo - mean_f), fabsf(xhi - mean_f)) : xhi - xlo;
    // a constant segment has gamma = 0 whatever eps is: all codes are 0
    float Af = 0.f;
    if (span_f > 0.f) {
      const float y = __frcp_rn(span_f);
      Af = (float)kQb * (y * (2.f - span_f * y));
    }
    const float Bf = -cf * Af;
    const float tau = 1e-6f * (fabsf(Af) * fmaxf(fabsf(xlo), fabsf(xhi)) + fabsf(Bf) + 1.0f);
    const int code_lo = (a.mode == BL_ABSMAX) ? -kCodeMax : 0;
    for (int k = threadIdx.x * 8; k < Kg; k += kGemvThreads * 8) {
      const float4 p = *reinterpret_cast<const float4*>(seg + k);
      const float4 q = *reinterpret_cast<const float4*>(seg + k + 4);
      const float v[8] = {p.x, p.y, p.z, p.w, q.x, q.y, q.z, q.w};
      int code[8];
      bool near_tie = false;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float f = fmaf(v[i], Af, Bf);
        const float t = f + kRoundMagic;                               // rne(f) in the low mantissa bits
        const float r = t - kRoundMagic;
        code[i] = __float_as_int(t) - __float_as_int(kRoundMagic);
        near_tie |= fabsf(fabsf(f - r) - 0.5f) < tau;
      }
      if (near_tie && span_f > 0.f) {                                  // rare: redo the 8 codes exactly
        const double c = (a.mode == BL_ABSMAX) ? mean : (double)xlo;
        const double span = (a.mode == BL_ABSMAX) ? fmax(fabs((double)xlo - mean), fabs((double)xhi - mean))
                                                  : (double)xhi - (double)xlo;
#pragma unroll
        for (int i = 0; i < 8; ++i) code[i] = code_slow_path(v[i], c, span);
      }
      uint32_t wq[2] = {0u, 0u};
#pragma unroll
      for (int i = 0; i < 8; ++i)
        wq[i >> 2] |= (uint32_t)(max(code_lo, min(kCodeMax, code[i])) & 0xFF) << (8 * (i & 3));
      *reinterpret_cast<uint2*>(codes + code_slot(g * Kg + k)) = make_uint2(wq[0], wq[1]);
    }
    if (threadIdx.x == 0) {
      // gamma and eta of Eq. 5 / 6 on x^ = (x - mean) rstd; only the final rescale reads them,
      // so fp32 is enough unless the mean dwarfs the spread (then the variance is formed in fp64)
      float t2 = 0.f;
#pragma unroll
      for (int w = 0; w < kGemvWarps; w += 4) t2 += (sh.s2[w] + sh.s2[w + 1]) + (sh.s2[w + 2] + sh.s2[w + 3]);
      float rstd = 1.f;
      if (ln) {
        const float inv_f = (float)geo.inv_kg;
        float var_f = fmaf(-mean_f, mean_f, t2 * inv_f);
        double var = (double)var_f;
        if (!(mean_f * mean_f <= 16.f * var_f)) var = (double)t2 * geo.inv_kg - mean * mean;
        if (var < 0.0) var = 0.0;
        rstd = rsqrt_scale(var + (double)a.ln_eps);
      }
      sh.gamma[g] = span_f * rstd;
      sh.eta[g] = (a.mode == BL_ABSMAX) ? 0.f : (xlo - mean_f) * rstd;
    }
    __syncthreads();                                   // codes and gamma of g visible; sh.s1.. reusable
  }

  // ---- this lane's 128 codes and their sum ---------------------------------------------------------
  uint32_t xr[32];
  int csum = 0;
  if (active) {
    const uint4* src = reinterpret_cast<const uint4*>(codes + slice * kSlice) + lane;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint4 v = src[i * 32];
      xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
    }
    int cs[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < 32; ++i) cs[i & 3] = __dp4a((int)xr[i], 0x01010101, cs[i & 3]);
    csum = (cs[0] + cs[1]) + (cs[2] + cs[3]);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) xr[i] = 0;
  }
  const float lane_scale = beta_mine * sh.gamma[my_group] * kInvQb;   // inactive lanes: group 0, sums 0

  // ---- stream the rows of this CTA, one batch of rpw rows per warp at a time -------------------------
  TY* y = reinterpret_cast<TY*>(a.y);
  for (int b = 0; b < nbatches; ++b) {
    // each row's register is refilled with the same row of the next batch as soon as it is used
    float (&part)[kGemvWarps][8] = sh.partial[b & 1];
    if (G == 1) {
      int v[8];
#pragma unroll
      for (int r = 0; r < kBatchRows; ++r) {
        v[r] = active ? (chunk_dot128(cur[r], xr) >> 6) - csum : 0;   // Eq. 7: 2 S - sum x~
        cur[r] = load_row(b + 1, r);
      }
      v[7] = 0;
      warp_sum8(v, lane);
      if ((lane & 3) == 0) part[warp][lane >> 2] = (float)v[0] * lane_scale;   // one group: the scale is uniform
    } else {
      float v[8];
#pragma unroll
      for (int r = 0; r < kBatchRows; ++r) {
        v[r] = active ? (float)((chunk_dot128(cur[r], xr) >> 6) - csum) * lane_scale : 0.f;
        cur[r] = load_row(b + 1, r);
      }
      v[7] = 0.f;
      warp_sum8(v, lane);
      if ((lane & 3) == 0) part[warp][lane >> 2] = v[0];
    }
    __syncthreads();
    // fold the K slices of each row and write y (one thread per row of this batch)
    if (threadIdx.x < rowslots * 8) {
      const int rs = threadIdx.x >> 3, r = threadIdx.x & 7;
      const int64_t n = row_begin + ((int64_t)b * rowslots + rs) * rpw + r;
      if (r < rpw && n < row_end) {
        float v = 0.f;
        for (int s = 0; s < nslices; ++s) v += part[rs * nslices + s][r];
        if (a.eta_correction) {
          for (int g = 0; g < G; ++g) v += sh.eta[g] * a.beta[g] * (float)a.rowsum[n * G + g];
        }
        y[n] = out_cast<TY>(v);
      }
    }
  }
}

template <typename TX, typename TY>
cudaError_t run2(const GemvArgs& a, cudaStream_t s) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // One CTA per SM when there are enough rows; every warp slot takes its rows in batches of at
  // most kBatchRows.
  GemvGeom geo;
  geo.nslices = (int)((a.K + kSlice - 1) / kSlice);
  geo.rowslots = kGemvWarps / geo.nslices;
  const int64_t rows_per_cta = (a.N + sms - 1) / sms;
  const int64_t per_slot = (rows_per_cta + geo.rowslots - 1) / geo.rowslots;
  const int64_t nbatches = (per_slot + kBatchRows - 1) / kBatchRows;
  geo.rows_per_cta = (int)rows_per_cta;
  geo.nbatches = (int)nbatches;
  geo.rpw = (int)((per_slot + nbatches - 1) / nbatches);
  geo.inv_kg = 1.0 / (double)(a.K / a.G);
  geo.inv_nslices = (65536u + geo.nslices - 1) / geo.nslices;
  const uint32_t group_chunks = a.G > 1 ? (uint32_t)(a.K / a.G / 128) : 256u;   // G > 1 needs K_g % 128 == 0
  geo.inv_group_chunks = (65536u + group_chunks - 1) / group_chunks;
  const unsigned grid = (unsigned)((a.N + rows_per_cta - 1) / rows_per_cta);
  const size_t smem = (size_t)a.K * sizeof(float) + (size_t)geo.nslices * kSlice;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(gemv_decode_kernel<TX, TY>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kGemvThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemv_decode_kernel<TX, TY>, a, geo);
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
