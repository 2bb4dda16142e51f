// Step 3 of BitLinear: alpha_g = mean W^(g), beta_g = mean |W^(g)| (Eq. 3, 12, 13), then
// W~ = Sign(W - alpha_g) with Sign(0) = -1 (Eq. 1-2), packed to one bit per weight.
//
// Two launches on the caller's stream, both HBM-bound (W is read twice: the means must be known
// before any sign can be taken):
//   1. reduce_partials  every block accumulates sum W (every addition in fp64: alpha decides bits)
//                       and sum |W| (fp32 inside a chunk of 8 weights, fp64 above) of its rows;
//                       one (group, block) partial each - fixed order, no atomics, so results
//                       are run-to-run identical;
//   2. sign_pack        every CTA first folds the partials in the same fixed order (a few KB from
//                       L2; this replaces a separate finalize launch), keeps per group the largest
//                       float <= alpha_g (a float w exceeds the fp64 mean exactly when it exceeds
//                       that float, so the sign test needs no fp64 compare), then walks its rows,
//                       one warp per row: 8 weights per lane -> one byte, placed directly at its
//                       position in the requested storage order, plus the per-row sign sums.
//                       CTA 0 also writes alpha and beta.
#include "common.cuh"

namespace bl {

namespace {

constexpr int kPackThreads = 256;
constexpr int kPackWarps = kPackThreads / 32;
constexpr int kReduceBlocks = 148 * 4;

struct PackWs {                 // layout of the caller's workspace
  double partial[BL_MAX_GROUPS][kReduceBlocks][2];
};

template <typename T>
__global__ void __launch_bounds__(kPackThreads)
reduce_partials(const T* __restrict__ W, int64_t N, int64_t K, int G, PackWs* ws) {
  const int64_t Kg = K / G;
  __shared__ double red[2][kPackWarps];
  for (int g = 0; g < G; ++g) {
    double s = 0.0, a = 0.0;
    for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
      const T* row = W + n * K + (int64_t)g * Kg;
      for (int64_t k = (int64_t)threadIdx.x * 8; k < Kg; k += (int64_t)kPackThreads * 8) {
        float v[8];
        Elem<T>::load8(row + k, v);
        // sum W decides bits (an element within the error of alpha of it would flip), so every
        // addition is fp64; sum |W| only scales the output: fp32 inside the chunk is enough
        const double ps = (((double)v[0] + (double)v[1]) + ((double)v[2] + (double)v[3])) +
                          (((double)v[4] + (double)v[5]) + ((double)v[6] + (double)v[7]));
        const float pa = ((fabsf(v[0]) + fabsf(v[1])) + (fabsf(v[2]) + fabsf(v[3]))) +
                         ((fabsf(v[4]) + fabsf(v[5])) + (fabsf(v[6]) + fabsf(v[7])));
        s += ps;
        a += (double)pa;
      }
    }
    s = warp_sum(s);
    a = warp_sum(a);
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s; red[1][threadIdx.x >> 5] = a; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double ts = 0.0, ta = 0.0;
      for (int w = 0; w < kPackWarps; ++w) { ts += red[0][w]; ta += red[1][w]; }
      ws->partial[g][blockIdx.x][0] = ts;
      ws->partial[g][blockIdx.x][1] = ta;
    }
    __syncthreads();
  }
}

// Where weight i (0..7) of the byte owned by lane j = lane & 3 goes inside the 32-weight word.
// CANONICAL: bit 8 j + i.  PREFILL / DECODE: weight q = 8 j + i sits at bit q/4 + 8 (q%4)
// = 2 j + (i/4 + 8 (i%4)).  Both are "a constant per i, shifted by a multiple of j".
__device__ __forceinline__ uint32_t sign_word(const float (&v)[8], float t, int j, bool canonical) {
  uint32_t canon = 0, perm = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (v[i] > t) {                                   // Eq. 2, Sign(0) = -1
      canon |= 1u << i;
      perm |= 1u << ((i >> 2) + 8 * (i & 3));
    }
  }
  return canonical ? canon << (8 * j) : perm << (2 * j);
}

template <typename T>
__global__ void __launch_bounds__(kPackThreads)
sign_pack(const T* __restrict__ W, int64_t N, int64_t K, int G, int layout, int nblocks,
          const float* __restrict__ alpha_in, const PackWs* __restrict__ ws, uint8_t* __restrict__ out,
          float* __restrict__ alpha, float* __restrict__ beta, int32_t* __restrict__ rowsum) {
  __shared__ int cnt[kPackWarps][BL_MAX_GROUPS];
  __shared__ float thr_s[BL_MAX_GROUPS];
  __shared__ double red[2][kPackWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t Kg = K / G;
  // ---- fold the partial sums (identical arithmetic in every CTA) ---------------------------------
  for (int g = 0; g < G; ++g) {
    double s = 0.0, a = 0.0;
    for (int b = threadIdx.x; b < nblocks; b += kPackThreads) {
      s += ws->partial[g][b][0];
      a += ws->partial[g][b][1];
    }
    s = warp_sum(s);
    a = warp_sum(a);
    if (lane == 0) { red[0][warp] = s; red[1][warp] = a; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double ts = 0.0, ta = 0.0;
      for (int w = 0; w < kPackWarps; ++w) { ts += red[0][w]; ta += red[1][w]; }
      const double cnt_g = (double)N * (double)Kg;
      const double al = alpha_in ? (double)alpha_in[g] : ts / cnt_g;   // Eq. 3 / 13
      const double be = ta / cnt_g;                                    // Eq. 12 / 13
      thr_s[g] = __double2float_rd(al);
      if (blockIdx.x == 0) { alpha[g] = (float)al; beta[g] = (float)be; }
    }
    __syncthreads();
  }
  // ---- sign and pack: one warp per row -------------------------------------------------------------
  const int64_t Kp = (K + 127) / 128 * 128;  // PREFILL pads K to 128
  const bool canonical = layout == BL_LAYOUT_CANONICAL;
  const bool word_store = !canonical || (K % 32 == 0);
  for (int64_t n = (int64_t)blockIdx.x * kPackWarps + warp; n < N; n += (int64_t)gridDim.x * kPackWarps) {
    for (int g = lane; g < G; g += 32) cnt[warp][g] = 0;
    __syncwarp();
    const T* row = W + n * K;
    int cur_g = -1, local = 0;
    for (int64_t k0 = 0; k0 < K; k0 += 256) {
      const int64_t k = k0 + (int64_t)lane * 8;
      uint32_t word = 0;
      if (k < K) {
        float v[8];
        Elem<T>::load8(row + k, v);
        const int g = (int)(k / Kg);
        word = sign_word(v, thr_s[g], lane & 3, canonical);
        if (g != cur_g) {
          if (cur_g >= 0) atomicAdd(&cnt[warp][cur_g], local);
          cur_g = g; local = 0;
        }
        local += __popc(word);
      }
      if (word_store) {
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        if ((lane & 3) == 0 && k < K) {
          int64_t off;
          if (layout == BL_LAYOUT_PREFILL) {
            off = ((n >> 7) * (Kp >> 7) + (k >> 7)) * 2048 + (n & 127) * 16 + ((k & 127) >> 5) * 4;
          } else {
            off = n * (K / 8) + (k >> 5) * 4;
          }
          *reinterpret_cast<uint32_t*>(out + off) = word;
        }
      } else if (k < K) {
        out[n * (K / 8) + (k >> 3)] = (uint8_t)(word >> (8 * (lane & 3)));
      }
    }
    if (cur_g >= 0) atomicAdd(&cnt[warp][cur_g], local);
    __syncwarp();
    if (rowsum) {
      for (int g = lane; g < G; g += 32) rowsum[n * G + g] = 2 * cnt[warp][g] - (int)Kg;
    }
    __syncwarp();
  }
}

template <typename T>
cudaError_t run(const PackArgs& a, cudaStream_t s) {
  PackWs* ws = reinterpret_cast<PackWs*>(a.ws);
  const T* W = reinterpret_cast<const T*>(a.W);
  const int nblocks = (int)((a.N < kReduceBlocks) ? a.N : kReduceBlocks);
  reduce_partials<T><<<nblocks, kPackThreads, 0, s>>>(W, a.N, a.K, a.G, ws);
  if (a.layout == BL_LAYOUT_PREFILL && (a.N % 128 != 0 || a.K % 128 != 0)) {
    cudaError_t e = cudaMemsetAsync(a.W_packed, 0, (size_t)prefill_bytes(a.N, a.K), s);
    if (e != cudaSuccess) return e;
  }
  const int64_t want = (a.N + kPackWarps - 1) / kPackWarps;
  const unsigned grid = (unsigned)(want < kReduceBlocks ? want : kReduceBlocks);
  sign_pack<T><<<grid, kPackThreads, 0, s>>>(W, a.N, a.K, a.G, (int)a.layout, nblocks, a.alpha_in, ws,
                                            a.W_packed, a.alpha, a.beta, a.rowsum);
  return cudaGetLastError();
}

}  // namespace

size_t pack_ws_bytes(int G) { (void)G; return sizeof(PackWs); }

cudaError_t launch_binarize_pack(const PackArgs& a, cudaStream_t s) {
  switch (a.wt) {
    case BL_F32: return run<float>(a, s);
    case BL_F16: return run<__half>(a, s);
    case BL_BF16: return run<__nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

int64_t prefill_bytes(int64_t N, int64_t K) {
  const int64_t Np = (N + 127) / 128 * 128, Kp = (K + 127) / 128 * 128;
  return Np * Kp / 8;
}

void prefill_index(int64_t K, int64_t n, int64_t k, int64_t* byte_off, int* bit) {
  const int64_t Kp = (K + 127) / 128 * 128;
  const int64_t block = (n >> 7) * (Kp >> 7) + (k >> 7);
  const int q = (int)(k & 31);
  const int p = (q >> 2) + 8 * (q & 3);
  *byte_off = block * 2048 + (n & 127) * 16 + ((k & 127) >> 5) * 4 + (p >> 3);
  *bit = p & 7;
}

void decode_index(int64_t K, int64_t n, int64_t k, int64_t* byte_off, int* bit) {
  const int q = (int)(k & 31);
  const int p = (q >> 2) + 8 * (q & 3);
  *byte_off = n * (K / 8) + (k >> 5) * 4 + (p >> 3);
  *bit = p & 7;
}

}  // namespace bl
