// Causal self-attention core of the decoder block (Sec. 2, Fig. 2b): per batch and head,
//   O = softmax(Q K^T / sqrt(d_h) + causal mask) V,
// in fp16 with fp32 softmax statistics and accumulators.  The paper keeps this part in "high
// precision"; it is not the path being optimised, so the kernel is a flash-style loop on the
// legacy tensor-core MMA (mma.sync m16n8k16):
//   one CTA per (128 queries, head, batch), 8 warps of 16 query rows each; key/value tiles of 64
//   rows, row-major in shared memory, double-buffered with cp.async (the next tile is in flight
//   while this one is multiplied); B operands by ldmatrix (transposed for V); online softmax
//   (running row maximum and sum, accumulators rescaled when the maximum moves); the probability
//   fragment of the first MMA is reused as the A operand of the second.  CTAs with the most keys
//   are scheduled first.
// Layout: q, k, v, o are [batch * seq, heads * 128] row-major with a common row stride `ld`
// (elements), so the three inputs may also be column blocks of one fused buffer.
#include "common.cuh"

namespace bl {

namespace {

constexpr int kDh = 128;            // head dimension
constexpr int kBq = 128;            // queries per CTA
constexpr int kBk = 64;             // keys per tile
constexpr int kAttnWarps = kBq / 16;
constexpr int kPitch = kDh + 8;     // row pitch of the K and V tiles (halves): 272 bytes, conflict-free ldmatrix
constexpr int kTileHalves = kBk * kPitch;
constexpr int kAttnSmem = 2 * 2 * kTileHalves * (int)sizeof(__half);   // two stages of (K, V)

__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const __half* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const __half* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(gsrc) : "memory");
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__global__ void __launch_bounds__(kAttnWarps * 32)
attention_causal_kernel(const __half* __restrict__ q, const __half* __restrict__ k, const __half* __restrict__ v,
                        __half* __restrict__ o, int S, int64_t ld, int64_t ld_o, float scale_log2) {
  extern __shared__ __align__(16) unsigned char attn_smem[];
  __half* tiles = reinterpret_cast<__half*>(attn_smem);           // [stage][K | V][64][kPitch]
  const int qb = (int)gridDim.x - 1 - (int)blockIdx.x, head = blockIdx.y, batch = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, qd = lane & 3;
  const int64_t tok0 = (int64_t)batch * S;
  const __half* qh = q + tok0 * ld + (int64_t)head * kDh;
  const __half* kh = k + tok0 * ld + (int64_t)head * kDh;
  const __half* vh = v + tok0 * ld + (int64_t)head * kDh;
  const int wrow = qb * kBq + warp * 16;                          // first query row of this warp
  const int r0 = wrow + g, r1 = r0 + 8;                           // the two query rows of this thread
  const int r0c = min(r0, S - 1), r1c = min(r1, S - 1);           // S may end inside the last block
  const int last_key = min(qb * kBq + kBq, S) - 1;
  const int n_tiles = last_key / kBk + 1;

  auto stage_tile = [&](int kb, int stage) {
    __half* Ks = tiles + (size_t)stage * 2 * kTileHalves;
    __half* Vs = Ks + kTileHalves;
    for (int idx = threadIdx.x; idx < kBk * (kDh / 8); idx += kAttnWarps * 32) {
      const int key = idx / (kDh / 8), c = idx % (kDh / 8);
      const int64_t row = (int64_t)(kb * kBk + key) * ld + c * 8;
      cp_async16(Ks + key * kPitch + c * 8, kh + row);
      cp_async16(Vs + key * kPitch + c * 8, vh + row);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  stage_tile(0, 0);

  // Q fragments of this warp's 16 rows, all 8 k-steps over d
  uint32_t aq[8][4];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const int d = ks * 16 + 2 * qd;
    aq[ks][0] = *reinterpret_cast<const uint32_t*>(qh + (int64_t)r0c * ld + d);
    aq[ks][1] = *reinterpret_cast<const uint32_t*>(qh + (int64_t)r1c * ld + d);
    aq[ks][2] = *reinterpret_cast<const uint32_t*>(qh + (int64_t)r0c * ld + d + 8);
    aq[ks][3] = *reinterpret_cast<const uint32_t*>(qh + (int64_t)r1c * ld + d + 8);
  }
  float acc[16][4];
#pragma unroll
  for (int dt = 0; dt < 16; ++dt) { acc[dt][0] = acc[dt][1] = acc[dt][2] = acc[dt][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  for (int kb = 0; kb < n_tiles; ++kb) {
    const int stage = kb & 1;
    __syncthreads();                                             // every warp is done with the other stage
    if (kb + 1 < n_tiles) {
      stage_tile(kb + 1, stage ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                             // tile kb is complete for everyone
    if (kb * kBk > wrow + 15) continue;                          // all keys of the tile lie after this warp's rows
    const __half* Ks = tiles + (size_t)stage * 2 * kTileHalves;
    const __half* Vs = Ks + kTileHalves;

    // S = Q K^T for this warp's 16 rows x 64 keys
    float s[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
    // k-steps outside, key blocks inside: consecutive MMAs write different accumulators
#pragma unroll
    for (int kp = 0; kp < 4; ++kp) {                              // two k-steps of 16 per ldmatrix
#pragma unroll
      for (int nt = 0; nt < 8; nt += 2) {
        uint32_t b[4], c[4];
        ldmatrix_x4(b, Ks + (nt * 8 + (lane & 7)) * kPitch + kp * 32 + (lane >> 3) * 8);
        ldmatrix_x4(c, Ks + ((nt + 1) * 8 + (lane & 7)) * kPitch + kp * 32 + (lane >> 3) * 8);
        mma_f16(s[nt], aq[2 * kp], b[0], b[1]);
        mma_f16(s[nt + 1], aq[2 * kp], c[0], c[1]);
        mma_f16(s[nt], aq[2 * kp + 1], b[2], b[3]);
        mma_f16(s[nt + 1], aq[2 * kp + 1], c[2], c[3]);
      }
    }
    if (kb * kBk + kBk - 1 > wrow) {                             // the tile reaches past a row: mask later keys
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int key = kb * kBk + nt * 8 + 2 * qd;
        if (key > r0) s[nt][0] = -INFINITY;
        if (key + 1 > r0) s[nt][1] = -INFINITY;
        if (key > r1) s[nt][2] = -INFINITY;
        if (key + 1 > r1) s[nt][3] = -INFINITY;
      }
    }
    // online softmax: new row maxima (over the 4 lanes that share a row), rescale, exponentials
    float mx0 = m0, mx1 = m1;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 1)); mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 1)); mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, 2));
    const float c0 = exp2f((m0 - mx0) * scale_log2), c1 = exp2f((m1 - mx1) * scale_log2);
    m0 = mx0; m1 = mx1;
    l0 *= c0; l1 *= c1;
#pragma unroll
    for (int dt = 0; dt < 16; ++dt) { acc[dt][0] *= c0; acc[dt][1] *= c0; acc[dt][2] *= c1; acc[dt][3] *= c1; }
    uint32_t ap[4][4];                                           // P as A fragments: 4 k-steps of 16 keys
    const float ms0 = m0 * scale_log2, ms1 = m1 * scale_log2;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = exp2f(fmaf(s[nt][0], scale_log2, -ms0)), p1 = exp2f(fmaf(s[nt][1], scale_log2, -ms0));
      const float p2 = exp2f(fmaf(s[nt][2], scale_log2, -ms1)), p3 = exp2f(fmaf(s[nt][3], scale_log2, -ms1));
      l0 += p0 + p1; l1 += p2 + p3;
      ap[nt >> 1][(nt & 1) * 2 + 0] = pack_half2(p0, p1);
      ap[nt >> 1][(nt & 1) * 2 + 1] = pack_half2(p2, p3);
    }
    // O += P V
#pragma unroll
    for (int kp = 0; kp < 2; ++kp) {                              // two key steps of 16 per ldmatrix
#pragma unroll
      for (int dt = 0; dt < 16; dt += 2) {
        uint32_t b[4], c[4];
        ldmatrix_x4_trans(b, Vs + (kp * 32 + (lane >> 3) * 8 + (lane & 7)) * kPitch + dt * 8);
        ldmatrix_x4_trans(c, Vs + (kp * 32 + (lane >> 3) * 8 + (lane & 7)) * kPitch + (dt + 1) * 8);
        mma_f16(acc[dt], ap[2 * kp], b[0], b[1]);
        mma_f16(acc[dt + 1], ap[2 * kp], c[0], c[1]);
        mma_f16(acc[dt], ap[2 * kp + 1], b[2], b[3]);
        mma_f16(acc[dt + 1], ap[2 * kp + 1], c[2], c[3]);
      }
    }
  }
  // normalise and store
  l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 1); l0 += __shfl_xor_sync(0xFFFFFFFFu, l0, 2);
  l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 1); l1 += __shfl_xor_sync(0xFFFFFFFFu, l1, 2);
  const float i0 = 1.f / l0, i1 = 1.f / l1;
  __half* oh = o + tok0 * ld_o + (int64_t)head * kDh;
#pragma unroll
  for (int dt = 0; dt < 16; ++dt) {
    const int d = dt * 8 + 2 * qd;
    if (r0 < S) *reinterpret_cast<uint32_t*>(oh + (int64_t)r0 * ld_o + d) = pack_half2(acc[dt][0] * i0, acc[dt][1] * i0);
    if (r1 < S) *reinterpret_cast<uint32_t*>(oh + (int64_t)r1 * ld_o + d) = pack_half2(acc[dt][2] * i1, acc[dt][3] * i1);
  }
}

}  // namespace

cudaError_t launch_attention_causal(const void* q, const void* k, const void* v, void* o, int batch, int S,
                                    int heads, int64_t ld, int64_t ld_o, cudaStream_t s) {
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)kDh);
  dim3 grid((unsigned)((S + kBq - 1) / kBq), (unsigned)heads, (unsigned)batch);
  cudaError_t e = cudaFuncSetAttribute(attention_causal_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmem);
  if (e != cudaSuccess) return e;
  attention_causal_kernel<<<grid, kAttnWarps * 32, kAttnSmem, s>>>(
      reinterpret_cast<const __half*>(q), reinterpret_cast<const __half*>(k), reinterpret_cast<const __half*>(v),
      reinterpret_cast<__half*>(o), S, ld, ld_o, scale_log2);
  return cudaGetLastError();
}

}  // namespace bl
