// Step 3 of BitLinear: alpha_g = mean W^(g), beta_g = mean |W^(g)| (Eq. 3, 12, 13), then
// W~ = Sign(W - alpha_g) with Sign(0) = -1 (Eq. 1-2), packed to one bit per weight.
//
// Two launches on the caller's stream, both HBM-bound (W is read twice: the means must be known
// before any sign can be taken).  The second read is served from L2 as far as L2 reaches: the first
// pass walks the rows forwards and asks L2 to keep the last kL2KeepBytes of the matrix it reads
// (evict-last), the second pass walks the rows backwards, starting with those, and marks what it
// reads evict-first.  Both passes keep four 32-byte (16-bit types: 16-byte) loads per thread in
// flight before the first is used.
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

constexpr int64_t kL2KeepBytes = 88ll << 20;   // what the first pass asks L2 to hold for the second
constexpr int kInFlight = 4;                   // chunks of 8 weights a thread loads before it uses the first

__device__ __forceinline__ uint64_t l2_policy(bool keep) {
  uint64_t p;
  if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint4 ldg128_hint(const void* p, uint64_t policy) {
  uint4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
  return v;
}
// Eight consecutive weights as raw 16-byte words, and their conversion to float.
template <typename T> struct Raw8 { uint4 a; };
template <> struct Raw8<float> { uint4 a, b; };
template <typename T>
__device__ __forceinline__ Raw8<T> load_raw8(const T* p, uint64_t policy) {
  Raw8<T> r;
  r.a = ldg128_hint(p, policy);
  if constexpr (sizeof(T) == 4) r.b = ldg128_hint(reinterpret_cast<const char*>(p) + 16, policy);
  return r;
}
__device__ __forceinline__ void to_float8(const Raw8<float>& r, float (&v)[8]) {
  v[0] = __uint_as_float(r.a.x); v[1] = __uint_as_float(r.a.y); v[2] = __uint_as_float(r.a.z); v[3] = __uint_as_float(r.a.w);
  v[4] = __uint_as_float(r.b.x); v[5] = __uint_as_float(r.b.y); v[6] = __uint_as_float(r.b.z); v[7] = __uint_as_float(r.b.w);
}
__device__ __forceinline__ void to_float8(const Raw8<__half>& r, float (&v)[8]) {
  const __half2* h = reinterpret_cast<const __half2*>(&r.a);
#pragma unroll
  for (int i = 0; i < 4; ++i) { const float2 f = __half22float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
}
__device__ __forceinline__ void to_float8(const Raw8<__nv_bfloat16>& r, float (&v)[8]) {
  const uint32_t* w = reinterpret_cast<const uint32_t*>(&r.a);
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}

struct PackWs {                 // layout of the caller's workspace
  double partial[BL_MAX_GROUPS][kReduceBlocks][2];
};

template <typename T>
__global__ void __launch_bounds__(kPackThreads)
reduce_partials(const T* __restrict__ W, int64_t N, int64_t K, int G, int64_t keep_from_row, PackWs* ws) {
  const int64_t Kg = K / G;
  __shared__ double red[2][kPackWarps];
  const uint64_t keep = l2_policy(true), stream = l2_policy(false);
  const int64_t cpr = (Kg + (int64_t)kPackThreads * 8 - 1) / ((int64_t)kPackThreads * 8);   // chunks of a thread per row and group
  const int64_t rows_b = N > blockIdx.x ? (N - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;  // rows of this block
  for (int g = 0; g < G; ++g) {
    double s = 0.0, a = 0.0;
    // the thread's chunks (row-major over the block's rows), kInFlight at a time
    int64_t r = 0, j = 0;                               // row of the block and chunk in it that comes next
    while (r < rows_b) {
      Raw8<T> raw[kInFlight];
      bool ok[kInFlight];
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        ok[i] = false;
        if (r < rows_b) {
          const int64_t n = blockIdx.x + r * (int64_t)gridDim.x;
          const int64_t k = ((int64_t)threadIdx.x + j * kPackThreads) * 8;
          ok[i] = k < Kg;
          if (ok[i]) raw[i] = load_raw8(W + n * K + (int64_t)g * Kg + k, n >= keep_from_row ? keep : stream);
          if (++j == cpr) { j = 0; ++r; }
        }
      }
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        if (!ok[i]) continue;
        float v[8];
        to_float8(raw[i], v);
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
__global__ void __launch_bounds__(kPackThreads, 4)
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
  const uint64_t stream = l2_policy(false);
  // rows from the last one backwards: the first pass read those last
  for (int64_t m = (int64_t)blockIdx.x * kPackWarps + warp; m < N; m += (int64_t)gridDim.x * kPackWarps) {
    const int64_t n = N - 1 - m;
    for (int g = lane; g < G; g += 32) cnt[warp][g] = 0;
    __syncwarp();
    const T* row = W + n * K;
    int cur_g = -1, local = 0;
    for (int64_t kb = 0; kb < K; kb += 256 * kInFlight) {
      Raw8<T> raw[kInFlight];
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        const int64_t k = kb + i * 256 + (int64_t)lane * 8;
        if (k < K) raw[i] = load_raw8(row + k, stream);
      }
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        const int64_t k0 = kb + i * 256;
        if (k0 >= K) break;                               // warp-uniform
        const int64_t k = k0 + (int64_t)lane * 8;
        uint32_t word = 0;
        if (k < K) {
          float v[8];
          to_float8(raw[i], v);
          const int g = G == 1 ? 0 : (int)(k / Kg);     // (a 64-bit division: only with groups)
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
    }
    if (cur_g >= 0) atomicAdd(&cnt[warp][cur_g], local);
    __syncwarp();
    if (rowsum) {
      for (int g = lane; g < G; g += 32) rowsum[n * G + g] = 2 * cnt[warp][g] - (int)Kg;
    }
    __syncwarp();
  }
}

// sign_pack for the common shape: one group, K a multiple of 256 (every lane of a warp has a chunk
// in every step, whole 32-weight words per quad).  Same results as sign_pack with about half the
// instructions per weight: the layout is a template parameter, output offsets advance by constants,
// the per-row count is one warp reduction, and the first loads of a warp's row are in flight while
// the CTA folds the partial sums.
template <typename T, int kLayout>
__global__ void __launch_bounds__(kPackThreads, 4)
sign_pack_rows(const T* __restrict__ W, int64_t N, int64_t K, int nblocks, const float* __restrict__ alpha_in,
               const PackWs* __restrict__ ws, uint8_t* __restrict__ out, float* __restrict__ alpha,
               float* __restrict__ beta, int32_t* __restrict__ rowsum) {
  __shared__ float thr_s;
  __shared__ double red[2][kPackWarps];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint64_t stream = l2_policy(false);
  constexpr bool kCanonical = kLayout == BL_LAYOUT_CANONICAL;
  const int64_t steps = K / (256 * kInFlight);           // whole batches; the rest (K % 1024) in a tail batch
  const int tail = (int)((K - steps * 256 * kInFlight) / 256);
  const int64_t m0 = (int64_t)blockIdx.x * kPackWarps + warp;
  // rows from the last one backwards: the first pass read those last
  auto row_of = [&](int64_t m) { return W + (N - 1 - m) * K + lane * 8; };
  Raw8<T> raw[kInFlight];
  auto issue = [&](const T* p, int count) {
#pragma unroll
    for (int i = 0; i < kInFlight; ++i)
      if (i < count) raw[i] = load_raw8(p + i * 256, stream);
  };
  if (m0 < N) issue(row_of(m0), steps > 0 ? kInFlight : tail);
  // ---- fold the partial sums (identical arithmetic in every CTA) ---------------------------------
  {
    double s = 0.0, a = 0.0;
    for (int b = threadIdx.x; b < nblocks; b += kPackThreads) {
      s += ws->partial[0][b][0];
      a += ws->partial[0][b][1];
    }
    s = warp_sum(s);
    a = warp_sum(a);
    if (lane == 0) { red[0][warp] = s; red[1][warp] = a; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double ts = 0.0, ta = 0.0;
      for (int w = 0; w < kPackWarps; ++w) { ts += red[0][w]; ta += red[1][w]; }
      const double cnt_g = (double)N * (double)K;
      const double al = alpha_in ? (double)alpha_in[0] : ts / cnt_g;   // Eq. 3
      const double be = ta / cnt_g;                                    // Eq. 12
      thr_s = __double2float_rd(al);
      if (blockIdx.x == 0) { alpha[0] = (float)al; beta[0] = (float)be; }
    }
    __syncthreads();
  }
  const float t = thr_s;
  const int64_t Kp = (K + 127) / 128 * 128;
  // byte offset of this lane's quad word inside a 256-weight step, and what a step adds
  const int64_t lane_off = kLayout == BL_LAYOUT_PREFILL ? (int64_t)(lane >> 4) * 2048 + ((lane & 15) >> 2) * 4 : (lane >> 2) * 4;
  constexpr int64_t kStepOff = kLayout == BL_LAYOUT_PREFILL ? 2 * 2048 : 32;
  for (int64_t m = m0; m < N; m += (int64_t)gridDim.x * kPackWarps) {
    const int64_t n = N - 1 - m;
    const T* row = row_of(m);
    uint8_t* o = out + lane_off +
                 (kLayout == BL_LAYOUT_PREFILL ? (n >> 7) * (Kp >> 7) * 2048 + (n & 127) * 16 : n * (K / 8));
    int ones = 0;
    auto consume = [&](int count) {
#pragma unroll
      for (int i = 0; i < kInFlight; ++i) {
        if (i >= count) break;                            // warp-uniform
        float v[8];
        to_float8(raw[i], v);
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j)                       // Eq. 2, Sign(0) = -1
          if (v[j] > t) word |= 1u << (kCanonical ? j : (j >> 2) + 8 * (j & 3));
        ones += __popc(word);
        word = kCanonical ? word << (8 * (lane & 3)) : word << (2 * (lane & 3));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        if ((lane & 3) == 0) *reinterpret_cast<uint32_t*>(o + i * kStepOff) = word;
      }
    };
    for (int64_t st = 0; st < steps; ++st) {
      if (m != m0 || st > 0) issue(row + st * (256 * kInFlight), kInFlight);
      consume(kInFlight);
      o += kInFlight * kStepOff;
    }
    if (tail) {
      if (m != m0 || steps > 0) issue(row + steps * (256 * kInFlight), tail);
      consume(tail);
    }
    ones = __reduce_add_sync(0xFFFFFFFFu, ones);
    if (rowsum && lane == 0) rowsum[n] = 2 * ones - (int)K;
  }
}

template <typename T>
cudaError_t run(const PackArgs& a, cudaStream_t s) {
  PackWs* ws = reinterpret_cast<PackWs*>(a.ws);
  const T* W = reinterpret_cast<const T*>(a.W);
  const int nblocks = (int)((a.N < kReduceBlocks) ? a.N : kReduceBlocks);
  // rows from keep_from on make up the last kL2KeepBytes of the matrix
  const int64_t row_bytes = a.K * (int64_t)sizeof(T);
  const int64_t keep_rows = kL2KeepBytes / row_bytes;
  const int64_t keep_from = a.N > keep_rows ? a.N - keep_rows : 0;
  reduce_partials<T><<<nblocks, kPackThreads, 0, s>>>(W, a.N, a.K, a.G, keep_from, ws);
  if (a.layout == BL_LAYOUT_PREFILL && (a.N % 128 != 0 || a.K % 128 != 0)) {
    cudaError_t e = cudaMemsetAsync(a.W_packed, 0, (size_t)prefill_bytes(a.N, a.K), s);
    if (e != cudaSuccess) return e;
  }
  const int64_t want = (a.N + kPackWarps - 1) / kPackWarps;
  const unsigned grid = (unsigned)(want < kReduceBlocks ? want : kReduceBlocks);
  if (a.G == 1 && a.K % 256 == 0) {
    switch (a.layout) {
      case BL_LAYOUT_CANONICAL:
        sign_pack_rows<T, BL_LAYOUT_CANONICAL><<<grid, kPackThreads, 0, s>>>(W, a.N, a.K, nblocks, a.alpha_in, ws, a.W_packed,
                                                                           a.alpha, a.beta, a.rowsum);
        break;
      case BL_LAYOUT_PREFILL:
        sign_pack_rows<T, BL_LAYOUT_PREFILL><<<grid, kPackThreads, 0, s>>>(W, a.N, a.K, nblocks, a.alpha_in, ws, a.W_packed,
                                                                         a.alpha, a.beta, a.rowsum);
        break;
      case BL_LAYOUT_DECODE:
        sign_pack_rows<T, BL_LAYOUT_DECODE><<<grid, kPackThreads, 0, s>>>(W, a.N, a.K, nblocks, a.alpha_in, ws, a.W_packed,
                                                                        a.alpha, a.beta, a.rowsum);
        break;
    }
    return cudaGetLastError();
  }
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
