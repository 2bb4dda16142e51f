// Step 3 of BitLinear: alpha_g = mean W^(g), beta_g = mean |W^(g)| (Eq. 3, 12, 13), then
// W~ = Sign(W - alpha_g) with Sign(0) = -1 (Eq. 1-2), packed to one bit per weight.
//
// Three launches on the caller's stream, all HBM-bound:
//   1. reduce_partials  every block accumulates sum W and sum |W| of its rows in fp64,
//                       one (group, block) partial each - fixed order, no atomics;
//   2. finalize         one block per group folds the partials, writes alpha/beta and the
//                       largest float <= alpha_g (a float w exceeds the fp64 mean exactly when
//                       it exceeds that float, so the sign test needs no fp64 compare);
//   3. sign_pack        one warp per row: 8 weights per lane -> one byte, regrouped into the
//                       requested storage order, plus the per-row sign sums.
#include "common.cuh"

namespace bl {

namespace {

constexpr int kPackThreads = 256;
constexpr int kReduceBlocks = 148 * 4;

struct PackWs {                 // layout of the caller's workspace
  double partial[BL_MAX_GROUPS][kReduceBlocks][2];
  double final_mean[BL_MAX_GROUPS][2];
  float thr[BL_MAX_GROUPS];     // largest float <= alpha_g
};

template <typename T>
__global__ void __launch_bounds__(kPackThreads)
reduce_partials(const T* __restrict__ W, int64_t N, int64_t K, int G, PackWs* ws) {
  const int64_t Kg = K / G;
  __shared__ double red[2][kPackThreads / 32];
  for (int g = 0; g < G; ++g) {
    double s = 0.0, a = 0.0;
    for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
      const T* row = W + n * K + (int64_t)g * Kg;
      for (int64_t k = (int64_t)threadIdx.x * 8; k < Kg; k += (int64_t)kPackThreads * 8) {
        float v[8];
        Elem<T>::load8(row + k, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) { s += (double)v[i]; a += fabs((double)v[i]); }
      }
    }
    s = warp_sum(s);
    a = warp_sum(a);
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s; red[1][threadIdx.x >> 5] = a; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double ts = 0.0, ta = 0.0;
      for (int w = 0; w < kPackThreads / 32; ++w) { ts += red[0][w]; ta += red[1][w]; }
      ws->partial[g][blockIdx.x][0] = ts;
      ws->partial[g][blockIdx.x][1] = ta;
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kPackThreads)
finalize_means(int64_t N, int64_t K, int G, int nblocks, const float* __restrict__ alpha_in,
               PackWs* ws, float* __restrict__ alpha, float* __restrict__ beta) {
  const int g = blockIdx.x;
  __shared__ double red[2][kPackThreads / 32];
  double s = 0.0, a = 0.0;
  for (int b = threadIdx.x; b < nblocks; b += kPackThreads) {
    s += ws->partial[g][b][0];
    a += ws->partial[g][b][1];
  }
  s = warp_sum(s);
  a = warp_sum(a);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s; red[1][threadIdx.x >> 5] = a; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ts = 0.0, ta = 0.0;
    for (int w = 0; w < kPackThreads / 32; ++w) { ts += red[0][w]; ta += red[1][w]; }
    const double cnt = (double)N * (double)(K / G);
    const double al = alpha_in ? (double)alpha_in[g] : ts / cnt;   // Eq. 3 / 13
    const double be = ta / cnt;                                    // Eq. 12 / 13
    ws->final_mean[g][0] = al;
    ws->final_mean[g][1] = be;
    ws->thr[g] = __double2float_rd(al);
    alpha[g] = (float)al;
    beta[g] = (float)be;
  }
}

// Bit scatter of one canonical byte (weights 8j..8j+7 of a 32-weight word, j = lane & 3)
// into the u32 that stores those 32 weights in each layout.
__device__ __forceinline__ uint32_t place_bits(uint32_t byte, int j, int layout) {
  if (layout == BL_LAYOUT_CANONICAL) return byte << (8 * j);
  uint32_t out = 0;
  // PREFILL and DECODE: weight q of the 32-weight word sits at bit q/4 + 8*(q%4).
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int q = 8 * j + i;
    out |= ((byte >> i) & 1u) << ((q >> 2) + 8 * (q & 3));
  }
  return out;
}

template <typename T>
__global__ void __launch_bounds__(kPackThreads)
sign_pack(const T* __restrict__ W, int64_t N, int64_t K, int G, int layout,
          const PackWs* __restrict__ ws, uint8_t* __restrict__ out, int32_t* __restrict__ rowsum) {
  __shared__ int cnt[kPackThreads / 32][BL_MAX_GROUPS];
  __shared__ float thr_s[BL_MAX_GROUPS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int g = threadIdx.x; g < G; g += kPackThreads) thr_s[g] = ws->thr[g];
  for (int g = lane; g < G; g += 32) cnt[warp][g] = 0;
  __syncthreads();
  const int64_t n = (int64_t)blockIdx.x * (kPackThreads / 32) + warp;
  if (n >= N) return;                        // whole warp leaves together
  const int64_t Kg = K / G;
  const int64_t Kp = (K + 127) / 128 * 128;  // PREFILL pads K to 128
  const bool word_store = (layout != BL_LAYOUT_CANONICAL) || (K % 32 == 0);
  const T* row = W + n * K;
  int cur_g = -1, local = 0;
  for (int64_t k0 = 0; k0 < K; k0 += 256) {
    const int64_t k = k0 + (int64_t)lane * 8;
    uint32_t byte = 0;
    if (k < K) {
      float v[8];
      Elem<T>::load8(row + k, v);
      const int g = (int)(k / Kg);
      const float t = thr_s[g];
#pragma unroll
      for (int i = 0; i < 8; ++i) byte |= (v[i] > t ? 1u : 0u) << i;   // Eq. 2, Sign(0) = -1
      if (g != cur_g) {
        if (cur_g >= 0) atomicAdd(&cnt[warp][cur_g], local);
        cur_g = g; local = 0;
      }
      local += __popc(byte);
    }
    if (word_store) {
      uint32_t word = place_bits(byte, lane & 3, layout);
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
      out[n * (K / 8) + (k >> 3)] = (uint8_t)byte;
    }
  }
  if (cur_g >= 0) atomicAdd(&cnt[warp][cur_g], local);
  __syncwarp();
  if (rowsum) {
    for (int g = lane; g < G; g += 32) rowsum[n * G + g] = 2 * cnt[warp][g] - (int)Kg;
  }
}

template <typename T>
cudaError_t run(const PackArgs& a, cudaStream_t s) {
  PackWs* ws = reinterpret_cast<PackWs*>(a.ws);
  const T* W = reinterpret_cast<const T*>(a.W);
  const int nblocks = (int)((a.N < kReduceBlocks) ? a.N : kReduceBlocks);
  reduce_partials<T><<<nblocks, kPackThreads, 0, s>>>(W, a.N, a.K, a.G, ws);
  finalize_means<<<a.G, kPackThreads, 0, s>>>(a.N, a.K, a.G, nblocks, a.alpha_in, ws, a.alpha, a.beta);
  if (a.layout == BL_LAYOUT_PREFILL && (a.N % 128 != 0 || a.K % 128 != 0)) {
    cudaError_t e = cudaMemsetAsync(a.W_packed, 0, (size_t)prefill_bytes(a.N, a.K), s);
    if (e != cudaSuccess) return e;
  }
  const int rows_per_block = kPackThreads / 32;
  const int64_t grid = (a.N + rows_per_block - 1) / rows_per_block;
  sign_pack<T><<<(unsigned)grid, kPackThreads, 0, s>>>(W, a.N, a.K, a.G, (int)a.layout, ws,
                                                      a.W_packed, a.rowsum);
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
