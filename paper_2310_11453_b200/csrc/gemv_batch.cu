// Small-batch decode: up to 8 tokens share one pass over the packed weights (Eq. 7, 11 with
// per-token gamma), LN + Quant of the tokens (Eq. 12, 4-6) fused in front.  Bound by streaming the
// packed weights (N*K/8 bytes) once; the tokens and outputs are a few hundred KB.
//
// Shape of one call.  One CTA of 16 warps per SM.
//   1. Every warp loads its first two batches of packed-weight blocks into registers (they do not
//      depend on x), lets the next kernel on the stream be scheduled and waits for everything
//      earlier on the stream (programmatic dependent launch).
//   2. The tokens are copied to shared memory (all asynchronous copies in flight at once) and
//      quantised there, 16 / M' warps per token (M' = M rounded up to a power of two): each warp
//      takes every P-th row of 256 elements of a group segment, the warps of a token meet at a
//      named barrier to add up their partial sums, and each writes the codes of its rows to the
//      token's padded row of int8 codes in shared memory.  Every CTA does all tokens (8 x K values
//      out of L2: cheaper than a separate launch).
//   3. Two warps share a tile of 16 output rows, each taking half of the K blocks of every group.
//      The 1-bit x 8-bit product runs on the tensor cores without ever expanding the weights to
//      bytes.  DECODE layout puts weight q of a 32-weight word at bit q/4 + 8*(q%4), so
//      word & (0x01010101 << j) is four bytes that are 0 or 2^j, the weights 4j..4j+3 of the word.
//      Eight such words of a row (256 weights) are one 16 x 32 byte A operand per bit plane j (one
//      logic instruction per register), the tokens' matching codes the 32 x 8 B operand, and
//      mma.sync m16n8k32 (s8 x s8 -> s32) accumulates 2^j * sum_{bit = 1} x~ for 16 rows x 8 tokens
//      (-2^7 for plane 7, whose byte 0x80 reads as -128).  Planes keep separate accumulators (eight
//      independent chains); sum_j |acc_j| >> j is exact.  At the end of a group the second warp of
//      the pair hands its sums over through shared memory and the first one finishes:
//      sum_k W~ x~ = 2 * (sum over set bits) - sum_k x~, then the rescale of Eq. 11.
#include "quant_rows.cuh"

namespace bl {

namespace {

using namespace rows;

constexpr int kBatchTokens = 8;          // tokens per launch = columns of the MMA
constexpr int kBatchWarps = 16;
constexpr int kPairs = kBatchWarps / 2;  // two warps per 16-row tile
constexpr int kTileRows = 16;            // output rows per tile = rows of the MMA
constexpr int kBlockK = 256;             // weights per row and MMA step: 8 words of 32
constexpr int kPreload = 4;              // K blocks per batch; two batches are held in registers (2 x 4 x 4 words)
constexpr int kRowPad = 16;              // bytes between token rows beyond K (bank spread of the B loads)
constexpr int kZeroBytes = 64;           // zero area read by the lanes of absent tokens
constexpr size_t kSmemBudget = 210 * 1024;

struct BatchShared {
  int csum[kBatchTokens][BL_MAX_GROUPS];
  float gamma[kBatchTokens][BL_MAX_GROUPS];
  float eta[kBatchTokens][BL_MAX_GROUPS];
  double part_s[kBatchWarps][32], part_q[kBatchWarps][32];   // per-warp, per-lane partial sums of one group segment
  float part_lo[kBatchWarps], part_hi[kBatchWarps];
  int part_c[kBatchWarps];
  int handover[kPairs][32][4];                       // second warp of a pair -> first, per group
};

// Named barrier `id` (1..15) for `threads` threads (a multiple of 32): a hardware barrier, no polling.
__device__ __forceinline__ void bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(gsrc) : "memory");
}
__device__ __forceinline__ void mma_s8s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct BatchArgs {
  const void* x; int M; int64_t K, N; int G; int mode; float ln_eps; int eta_correction;
  const uint8_t* W_packed; const float* beta; const int32_t* rowsum; void* y;
  int stage_tokens;                      // the raw tokens fit in shared memory beside the codes
  double inv_kg;                         // 1 / K_g (a double-precision division per thread otherwise)
  uint32_t* clear_status;                // when set: a status word this launch clears, in stream order
  const int8_t* pre_codes;               // when set (one group): the tokens' codes [M][K], their gamma [M] and code
  const float* pre_gamma;                // sums [M], the work of a kernel earlier on the stream; the tokens are
  const int* pre_csum;                   // then not quantised here
};

// The four A words of K block b for this lane: rows g and g + 8, words qd and 4 + qd of the block.
__device__ __forceinline__ void load_block(const uint32_t* __restrict__ row_lo, const uint32_t* __restrict__ row_hi,
                                           int b, int qd, uint32_t (&w)[4]) {
  w[0] = __ldg(row_lo + 8 * b + qd);
  w[1] = __ldg(row_hi + 8 * b + qd);
  w[2] = __ldg(row_lo + 8 * b + 4 + qd);
  w[3] = __ldg(row_hi + 8 * b + 4 + qd);
}

template <typename TX, typename TY>
__global__ void __launch_bounds__(kBatchWarps * 32, 1)
gemv_batch_kernel(BatchArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ BatchShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g8 = lane >> 2, qd = lane & 3;                   // MMA fragment coordinates
  const int Kg = (int)(a.K / a.G);
  const int bpg = Kg / kBlockK;                              // K blocks per group
  const int64_t stride = a.K + kRowPad;                      // bytes between token rows of codes
  int8_t* codes = reinterpret_cast<int8_t*>(smem + kZeroBytes);
  unsigned char* raw = smem + kZeroBytes + (size_t)a.M * stride;   // staged tokens, [M][K] of TX
  const int64_t words_per_row = a.K / 32;
  const uint32_t* W32 = reinterpret_cast<const uint32_t*>(a.W_packed);
  const int64_t tiles = a.N / kTileRows;

  // ---- 1. work of this warp in the rows phase: half h of every group's blocks of the pair's tiles
  const int pair = warp >> 1, h = warp & 1;
  const int half0 = (bpg + 1) / 2;
  const int my_blocks = h == 0 ? half0 : bpg - half0;        // per group (may be 0 for h = 1)
  const int my_first = h == 0 ? 0 : half0;
  const int nbg = (my_blocks + kPreload - 1) / kPreload;     // my batches per group
  const int64_t tile_step = (int64_t)gridDim.x * kPairs;
  const int64_t tile0 = (int64_t)blockIdx.x + (int64_t)gridDim.x * pair;
  struct Item { int64_t tile; int g, b; };
  auto valid = [&](const Item& it) { return nbg > 0 && it.tile < tiles; };
  auto next = [&](const Item& it) {
    Item n = it;
    if (++n.b >= nbg) { n.b = 0; if (++n.g == a.G) { n.g = 0; n.tile += tile_step; } }
    return n;
  };
  auto load_item = [&](const Item& it, uint32_t (&w)[kPreload][4]) {
    const uint32_t* lo = W32 + (it.tile * kTileRows + g8) * words_per_row;
    const uint32_t* hi = lo + 8 * words_per_row;
    const int b0 = it.g * bpg + my_first + it.b * kPreload;
    const int left = my_blocks - it.b * kPreload;
    const int nb = left < kPreload ? left : kPreload;
#pragma unroll
    for (int i = 0; i < kPreload; ++i)
      if (i < nb) load_block(lo, hi, b0 + i, qd, w[i]);
  };
  Item it1{tile0, 0, 0};
  Item it2 = next(it1);
  uint32_t wa[kPreload][4], wb[kPreload][4];
  if (valid(it1)) load_item(it1, wa);
  if (valid(it2)) load_item(it2, wb);
  if (threadIdx.x < kZeroBytes / 4) reinterpret_cast<uint32_t*>(smem)[threadIdx.x] = 0u;
  pdl_launch_dependents();
  pdl_wait();
  if (a.clear_status != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *a.clear_status = 0u;

  // ---- 2. LN + Quant of the tokens (or their codes as another kernel left them)
  if (a.pre_codes != nullptr) {
    const int pieces_per_row = (int)(a.K / 16);
    for (int i = threadIdx.x; i < a.M * pieces_per_row; i += kBatchWarps * 32) {
      const int tok = i / pieces_per_row, p = i - tok * pieces_per_row;
      cp_async16(codes + (int64_t)tok * stride + (int64_t)p * 16, a.pre_codes + (int64_t)tok * a.K + (int64_t)p * 16);
    }
    if (threadIdx.x < a.M) {
      sh.gamma[threadIdx.x][0] = a.pre_gamma[threadIdx.x];
      sh.eta[threadIdx.x][0] = 0.f;
      sh.csum[threadIdx.x][0] = a.pre_csum[threadIdx.x];
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
  if (a.stage_tokens) {
    const uint4* src = reinterpret_cast<const uint4*>(a.x);
    uint4* dst = reinterpret_cast<uint4*>(raw);
    const int pieces = (int)((size_t)a.M * a.K * sizeof(TX) / 16);
    for (int i = threadIdx.x; i < pieces; i += kBatchWarps * 32) cp_async16(dst + i, src + i);
    asm volatile("cp.async.wait_all;" ::: "memory");
  }
  __syncthreads();
  {
    int mp = 1;
    while (mp < a.M) mp <<= 1;
    const int P = kBatchWarps / mp;                           // warps per token
    const int tok = warp / P, j = warp % P, w0 = tok * P;
    if (tok < a.M) {
      const TX* xt = a.stage_tokens ? reinterpret_cast<const TX*>(raw) + (int64_t)tok * a.K
                                    : reinterpret_cast<const TX*>(a.x) + (int64_t)tok * a.K;
      const int rows_per_group = Kg / 256;                    // 32-chunk rows of a group segment
      const double inv_kg = a.inv_kg;
      for (int g = 0; g < a.G; ++g) {
        const uint4* seg = reinterpret_cast<const uint4*>(xt + (int64_t)g * Kg);
        float pilot;
        {
          Chunk<TX> ch; float v[8];
          ch.load(seg, 0); ch.unpack(v);                      // same address in every thread: a broadcast
          pilot = 0.125f * (((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7])));
          if (a.ln_eps < 0.f) pilot = 0.f;
        }
        // The sums must not depend on how many warps share the token (a token's result is the same
        // whatever else is in the batch), so their order of additions is fixed: chunk row rr belongs
        // to strip rr % 16; a strip's sum is taken in fp32 per lane, rows ascending; the 16 strips
        // are then added per lane in fp64 by halving (strip v with v + 8, then + 4, + 2, + 1), the
        // first levels inside the warp that owns the strips, the rest across the token's warps;
        // the lanes are added last.
        float mn = INFINITY, mx = -INFINITY;
        // this warp's strips: j, j + P, ... (at most 8); strip i >= 4 meets strip i - 4 as soon as it is done
        double ls[kBatchWarps / 4], lq[kBatchWarps / 4];
#pragma unroll
        for (int i = 0; i < kBatchWarps / 2; ++i) {
          float sum = 0.f, sq = 0.f;
          if (i * P < kBatchWarps) {
            for (int rr = j + i * P; rr < rows_per_group; rr += kBatchWarps) {
              Chunk<TX> ch; float v[8], d[8];
              ch.load(seg, rr * 32 + lane); ch.unpack(v);
#pragma unroll
              for (int e = 0; e < 8; ++e) { d[e] = v[e] - pilot; mn = fminf(mn, v[e]); mx = fmaxf(mx, v[e]); }
              sum += ((d[0] + d[1]) + (d[2] + d[3])) + ((d[4] + d[5]) + (d[6] + d[7]));
              float p0 = d[0] * d[0], p1 = d[1] * d[1];
#pragma unroll
              for (int e = 2; e < 8; e += 2) { p0 = fmaf(d[e], d[e], p0); p1 = fmaf(d[e + 1], d[e + 1], p1); }
              sq += p0 + p1;
            }
          }
          if (i < kBatchWarps / 4) { ls[i] = (double)sum; lq[i] = (double)sq; }   // strips it does not own: +0.0, exact
          else if (i * P < kBatchWarps) { ls[i - kBatchWarps / 4] += (double)sum; lq[i - kBatchWarps / 4] += (double)sq; }
        }
        {
          // strips j + i P and j + (i + h) P differ by h P = 8, 4, 2 (only while h P < 16)
          const int n = kBatchWarps / P;                         // strips of this warp: 1, 2, 4 or 8
#pragma unroll
          for (int h = kBatchWarps / 8; h >= 1; h >>= 1)
            if (h < n) {
#pragma unroll
              for (int i = 0; i < kBatchWarps / 8; ++i)
                if (i < h) { ls[i] += ls[i + h]; lq[i] += lq[i + h]; }
            }
        }
        mn = warp_min(mn); mx = warp_max(mx);
        sh.part_s[warp][lane] = ls[0]; sh.part_q[warp][lane] = lq[0];
        if (lane == 0) { sh.part_lo[warp] = mn; sh.part_hi[warp] = mx; }
        bar_sync(1 + tok, P * 32);
        // across the token's warps, one quantity at a time (the kernel is at its register limit)
        auto fold = [&](const double (*part)[32]) -> double {
          double t[kBatchWarps / 2];
#pragma unroll
          for (int w = 0; w < kBatchWarps / 2; ++w) {
            t[w] = w < P ? part[w0 + w][lane] : 0.0;
            if (P > kBatchWarps / 2) t[w] += part[w0 + w + kBatchWarps / 2][lane];
          }
#pragma unroll
          for (int h = kBatchWarps / 4; h >= 1; h >>= 1)
            if (h < P) {
#pragma unroll
              for (int w = 0; w < kBatchWarps / 4; ++w)
                if (w < h) t[w] += t[w + h];
            }
          return warp_sum(t[0]);
        };
        const double St = fold(sh.part_s), Qt = fold(sh.part_q);
        float xlo = INFINITY, xhi = -INFINITY;
        for (int w = w0; w < w0 + P; ++w) { xlo = fminf(xlo, sh.part_lo[w]); xhi = fmaxf(xhi, sh.part_hi[w]); }
        double mean = 0.0, rstd = 1.0;
        if (!(a.ln_eps < 0.f)) {
          const double dm = St * inv_kg;                      // mean - pilot
          mean = (double)pilot + dm;
          double var = Qt * inv_kg - dm * dm;
          if (var < 0.0) var = 0.0;
          rstd = rsqrt_newton(var + (double)a.ln_eps);
        }
        double gam, et;
        scope_gamma_eta(a.mode, ((double)xlo - mean) * rstd, ((double)xhi - mean) * rstd, gam, et);
        const RowMap map = row_map(a.mode, mean, rstd, gam, et, xlo, xhi);
        int8_t* row = codes + (int64_t)tok * stride + (int64_t)g * Kg;
        int cs = 0;
        for (int rr = j; rr < rows_per_group; rr += P) {
          const int c = rr * 32 + lane;
          Chunk<TX> ch; float v[8];
          ch.load(seg, c); ch.unpack(v);
          const uint2 cd = map.clip ? row_codes8<true>(v, map) : row_codes8<false>(v, map);
          cs = __dp4a((int)cd.x, 0x01010101, cs);
          cs = __dp4a((int)cd.y, 0x01010101, cs);
          *reinterpret_cast<uint2*>(row + (size_t)c * 8) = cd;
        }
        cs = warp_sum(cs);
        if (lane == 0) sh.part_c[warp] = cs;
        bar_sync(1 + tok, P * 32);
        if (j == 0 && lane == 0) {
          int tot = 0;
          for (int w = w0; w < w0 + P; ++w) tot += sh.part_c[w];
          sh.csum[tok][g] = tot; sh.gamma[tok][g] = (float)gam; sh.eta[tok][g] = (float)et;
        }
        bar_sync(1 + tok, P * 32);                            // the partial sums may be overwritten
      }
    }
  }
  }
  __syncthreads();

  // ---- 3. rows.  Lanes of absent tokens read zeros.
  const bool tok_ok = g8 < a.M;
  const unsigned char* brow = tok_ok ? reinterpret_cast<const unsigned char*>(codes) + g8 * stride : smem;
  const uint32_t bmask = tok_ok ? 0xFFFFFFFFu : (uint32_t)(kZeroBytes - 1);
  const bool correct = a.eta_correction != 0;
  TY* y = reinterpret_cast<TY*>(a.y);
  Item it3 = next(it2);
  for (int64_t tile = tile0; tile < tiles; tile += tile_step) {
    const int64_t r0 = tile * kTileRows;
    float out[4] = {0.f, 0.f, 0.f, 0.f};
    for (int g = 0; g < a.G; ++g) {
      int acc[8][4];
#pragma unroll
      for (int jj = 0; jj < 8; ++jj)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[jj][c] = 0;
      for (int b = 0; b < nbg; ++b) {
        const int b0 = g * bpg + my_first + b * kPreload;
        const int left = my_blocks - b * kPreload;
        const int nb = left < kPreload ? left : kPreload;
#pragma unroll
        for (int i = 0; i < kPreload; ++i) {
          if (i < nb) {
            // B operand: the 8 planes' words for word qd (x0, x1) and word 4 + qd (x2, x3) of block b0 + i
            const uint32_t off0 = (uint32_t)(32 * (8 * (b0 + i) + qd)) & bmask;
            const uint32_t off1 = (uint32_t)(32 * (8 * (b0 + i) + 4 + qd)) & bmask;
            const uint4 x0 = *reinterpret_cast<const uint4*>(brow + off0);
            const uint4 x1 = *reinterpret_cast<const uint4*>(brow + off0 + 16);
            const uint4 x2 = *reinterpret_cast<const uint4*>(brow + off1);
            const uint4 x3 = *reinterpret_cast<const uint4*>(brow + off1 + 16);
            const uint32_t bl[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
            const uint32_t bh[8] = {x2.x, x2.y, x2.z, x2.w, x3.x, x3.y, x3.z, x3.w};
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              const uint32_t m = 0x01010101u << jj;
              const uint32_t af[4] = {wa[i][0] & m, wa[i][1] & m, wa[i][2] & m, wa[i][3] & m};
              mma_s8s8(acc[jj], af, bl[jj], bh[jj]);
            }
          }
        }
        // the next batch's weights move up; the one after it starts loading
#pragma unroll
        for (int i = 0; i < kPreload; ++i)
#pragma unroll
          for (int c = 0; c < 4; ++c) wa[i][c] = wb[i][c];
        if (valid(it3)) load_item(it3, wb);
        it3 = next(it3);
      }
      // the group is complete in this warp's half: sums over the set bits, per (row, token) of the fragment
      int s[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int t = 0;
#pragma unroll
        for (int jj = 0; jj < 7; ++jj) t += acc[jj][c] >> jj;
        s[c] = t - (acc[7][c] >> 7);                             // plane 7's bytes are 0x80 = -128 as s8
      }
      if (h == 1) *reinterpret_cast<int4*>(sh.handover[pair][lane]) = make_int4(s[0], s[1], s[2], s[3]);
      bar_sync(1 + pair, 64);
      if (h == 0) {
        const int4 o = *reinterpret_cast<const int4*>(sh.handover[pair][lane]);
        const int so[4] = {o.x, o.y, o.z, o.w};
        const float beta_g = a.beta[g];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int tok = 2 * qd + (c & 1);
          if (tok < a.M) {
            const int dot = 2 * (s[c] + so[c]) - sh.csum[tok][g];
            const int64_t n = r0 + g8 + 8 * (c >> 1);
            out[c] += dequant_term(dot, beta_g, sh.gamma[tok][g], correct ? sh.eta[tok][g] : 0.f,
                                   correct ? a.rowsum[n * a.G + g] : 0, correct);
          }
        }
      }
      bar_sync(1 + pair, 64);                                    // the hand-over slot may be rewritten
    }
    if (h == 0) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int tok = 2 * qd + (c & 1);
        if (tok < a.M) y[(int64_t)tok * a.N + r0 + g8 + 8 * (c >> 1)] = out_cast<TY>(out[c]);
      }
    }
  }
}

inline size_t batch_smem(int64_t M, int64_t K, size_t xsz, bool stage) {
  return kZeroBytes + (size_t)M * (size_t)(K + kRowPad) + (stage ? (size_t)M * (size_t)K * xsz : 0);
}

template <typename TX, typename TY>
cudaError_t run2(BatchArgs a, cudaStream_t s) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int64_t tiles = a.N / kTileRows;
  // With the tokens quantised by a kernel of one CTA per token just ahead of this one, leave that kernel its
  // SMs: a CTA here takes every register of an SM, so one that had to share would only start when the
  // other kernel's CTA has gone, without the head start on its weights.
  const int64_t usable = a.pre_codes != nullptr && sms > 2 * a.M ? sms - a.M : sms;
  const unsigned grid = (unsigned)(tiles < usable ? tiles : usable);
  a.stage_tokens = (a.pre_codes == nullptr && batch_smem(a.M, a.K, sizeof(TX), true) <= kSmemBudget) ? 1 : 0;
  const size_t smem = batch_smem(a.M, a.K, sizeof(TX), a.stage_tokens != 0);
  if ((e = cudaFuncSetAttribute(gemv_batch_kernel<TX, TY>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
      cudaSuccess)
    return e;
  return launch_pdl(gemv_batch_kernel<TX, TY>, grid, kBatchWarps * 32, smem, s, a);
}

template <typename TX>
cudaError_t run1(const BatchArgs& a, bl_dtype yt, cudaStream_t s) {
  switch (yt) {
    case BL_F32: return run2<TX, float>(a, s);
    case BL_F16: return run2<TX, __half>(a, s);
    case BL_BF16: return run2<TX, __nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

bool gemv_batch_supported(int64_t M, int64_t K, int64_t N, int G) {
  return M >= 1 && G >= 1 && K % kBlockK == 0 && (K / G) % kBlockK == 0 && N % kTileRows == 0 &&
         batch_smem(M < kBatchTokens ? M : kBatchTokens, K, 0, false) <= kSmemBudget;
}

// M tokens in launches of up to 8; later launches find the weights in L2.  A single token goes to the
// single-token kernel (half the time of this one at M = 1; its statistics are summed in another order,
// so its gamma may differ from this kernel's in the last bit).
cudaError_t launch_gemv_batch(const GemvArgs& g, int64_t M, cudaStream_t s) {
  if (M == 1 && g.K <= 32768) return launch_gemv_decode(g, s);
  const size_t xsz = g.xt == BL_F32 ? 4 : 2, ysz = g.yt == BL_F32 ? 4 : 2;
  for (int64_t m0 = 0; m0 < M; m0 += kBatchTokens) {
    BatchArgs a;
    a.x = reinterpret_cast<const char*>(g.x) + (size_t)m0 * (size_t)g.K * xsz;
    a.M = (int)(M - m0 < kBatchTokens ? M - m0 : kBatchTokens);
    a.K = g.K; a.N = g.N; a.G = g.G; a.mode = (int)g.mode; a.ln_eps = g.ln_eps; a.eta_correction = g.eta_correction;
    a.W_packed = g.W_packed; a.beta = g.beta; a.rowsum = g.rowsum;
    a.y = reinterpret_cast<char*>(g.y) + (size_t)m0 * (size_t)g.N * ysz;
    a.stage_tokens = 0;
    a.inv_kg = 1.0 / (double)(g.K / g.G);
    a.clear_status = m0 == 0 ? g.clear_status : nullptr;
    a.pre_codes = nullptr; a.pre_gamma = nullptr; a.pre_csum = nullptr;
    cudaError_t e = cudaErrorInvalidValue;
    switch (g.xt) {
      case BL_F32: e = run1<float>(a, g.yt, s); break;
      case BL_F16: e = run1<__half>(a, g.yt, s); break;
      case BL_BF16: e = run1<__nv_bfloat16>(a, g.yt, s); break;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// One launch for up to 8 tokens (one group) whose codes [M][K], gamma [M] and code sums [M] an earlier
// kernel on the stream has written.
cudaError_t launch_gemv_batch_pre(const GemvArgs& g, int64_t M, const int8_t* codes, const float* gamma, const int* csum,
                                  cudaStream_t s) {
  if (M < 1 || M > kBatchTokens || g.G != 1) return cudaErrorInvalidValue;
  BatchArgs a;
  a.x = g.x; a.M = (int)M;
  a.K = g.K; a.N = g.N; a.G = 1; a.mode = (int)g.mode; a.ln_eps = g.ln_eps; a.eta_correction = 0;
  a.W_packed = g.W_packed; a.beta = g.beta; a.rowsum = g.rowsum; a.y = g.y;
  a.stage_tokens = 0;
  a.inv_kg = 1.0 / (double)g.K;
  a.clear_status = nullptr;
  a.pre_codes = codes; a.pre_gamma = gamma; a.pre_csum = csum;
  switch (g.xt) {
    case BL_F32: return run1<float>(a, g.yt, s);
    case BL_F16: return run1<__half>(a, g.yt, s);
    case BL_BF16: return run1<__nv_bfloat16>(a, g.yt, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl
