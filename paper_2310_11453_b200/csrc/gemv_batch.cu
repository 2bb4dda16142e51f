// Small-batch decode: up to 8 tokens share one pass over the packed weights (Eq. 7, 11 with
// per-token gamma), LN + Quant of the tokens (Eq. 12, 4-6) fused in front.  Bound by streaming the
// packed weights (N*K/8 bytes) once; the tokens and outputs are a few hundred KB.
//
// Shape of one call.  A CTA has 8 warps.
//   1. Every warp loads the packed weights of its first two batches of K blocks into registers
//      (they do not depend on x), lets the next kernel on the stream be scheduled and waits for
//      everything earlier on the stream (programmatic dependent launch).
//   2. Warp t normalises and quantises token t (every CTA does all tokens: 8 x K values out of
//      L2, cheaper than a separate launch) and leaves the int8 codes in shared memory, one padded
//      row per token, with the per-group sums of the codes, gamma and eta.  A group segment of up
//      to 8 KB is first copied to the warp's staging slot with all its asynchronous copies in
//      flight at once, so the two passes over it (statistics, codes) run at shared-memory
//      latency; longer segments are read from L2 twice.
//   3. Per 16 rows, the warp runs the 1-bit x 8-bit product on the tensor cores without ever
//      expanding the weights to bytes.  DECODE layout puts weight q of a 32-weight word at bit
//      q/4 + 8*(q%4), so word & (0x01010101 << j) is four bytes that are 0 or 2^j, the
//      weights 4j..4j+3 of the word.  Eight such words of a row (256 weights) are one 16 x 32
//      byte A operand per bit plane j (one logic instruction per register), the tokens' matching
//      codes the 32 x 8 B operand, and mma.sync m16n8k32 (s8 x s8 -> s32) accumulates
//      2^j * sum_{bit = 1} x~ for 16 rows x 8 tokens (-2^7 for plane 7, whose byte 0x80 reads as
//      -128).  Planes keep separate accumulators (eight independent chains); a group's result is
//      sum_j |acc_j| >> j, exact, and sum_k W~ x~ = 2 * (that) - sum_k x~.
#include "quant_rows.cuh"

namespace bl {

namespace {

using namespace rows;

constexpr int kBatchTokens = 8;          // tokens per launch = columns of the MMA
constexpr int kBatchWarps = 8;
constexpr int kTileRows = 16;            // output rows per warp tile = rows of the MMA
constexpr int kBlockK = 256;             // weights per row and MMA step: 8 words of 32
constexpr int kPreload = 8;              // K blocks per batch; two batches are held in registers (2 x 8 x 4 words)
constexpr int kRowPad = 16;              // bytes between token rows beyond K (bank spread of the B loads)
constexpr int kZeroBytes = 64;           // zero area read by the lanes of absent tokens
constexpr int kStageBytes = 8192;        // per-warp staging slot for one group segment of a token

struct BatchShared {
  int csum[kBatchTokens][BL_MAX_GROUPS];
  float gamma[kBatchTokens][BL_MAX_GROUPS];
  float eta[kBatchTokens][BL_MAX_GROUPS];
};

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
  const int blocks_per_group = Kg / kBlockK;
  const int64_t stride = a.K + kRowPad;                      // bytes between token rows of codes
  uint4* slot = reinterpret_cast<uint4*>(smem + kZeroBytes + (size_t)warp * kStageBytes);
  int8_t* codes = reinterpret_cast<int8_t*>(smem + kZeroBytes + (size_t)kBatchWarps * kStageBytes);
  const int64_t words_per_row = a.K / 32;
  const uint32_t* W32 = reinterpret_cast<const uint32_t*>(a.W_packed);
  const int64_t tiles = a.N / kTileRows;

  // 1. the warp's first two batches of weight blocks into registers; these loads read only the
  //    static weights.  Work items are (tile, batch): a batch is up to kPreload K blocks of one group.
  const int nbg = (blocks_per_group + kPreload - 1) / kPreload;   // batches per group
  const int nbt = a.G * nbg;                                      // batches per tile
  const int64_t tile_step = (int64_t)gridDim.x * kBatchWarps;
  struct Item { int64_t tile; int t; };
  auto valid = [&](const Item& it) { return it.tile < tiles; };
  auto next = [&](const Item& it) {
    Item n = it;
    if (++n.t == nbt) { n.t = 0; n.tile += tile_step; }
    return n;
  };
  // first K block and number of K blocks of a batch
  auto first_block = [&](const Item& it) { return (it.t / nbg) * blocks_per_group + (it.t % nbg) * kPreload; };
  auto num_blocks = [&](const Item& it) {
    const int left = blocks_per_group - (it.t % nbg) * kPreload;
    return left < kPreload ? left : kPreload;
  };
  auto load_item = [&](const Item& it, uint32_t (&w)[kPreload][4]) {
    const uint32_t* lo = W32 + (it.tile * kTileRows + g8) * words_per_row;
    const uint32_t* hi = lo + 8 * words_per_row;
    const int b0 = first_block(it), nb = num_blocks(it);
#pragma unroll
    for (int i = 0; i < kPreload; ++i)
      if (i < nb) load_block(lo, hi, b0 + i, qd, w[i]);
  };
  Item cur{(int64_t)blockIdx.x + (int64_t)gridDim.x * warp, 0};
  Item nxt = next(cur);
  uint32_t wa[kPreload][4], wb[kPreload][4];
  if (valid(cur)) load_item(cur, wa);
  if (valid(nxt)) load_item(nxt, wb);
  if (threadIdx.x < kZeroBytes / 4) reinterpret_cast<uint32_t*>(smem)[threadIdx.x] = 0u;
  pdl_launch_dependents();
  pdl_wait();

  // 2. LN + Quant of token `warp`
  if (warp < a.M) {
    const TX* xt = reinterpret_cast<const TX*>(a.x) + (int64_t)warp * a.K;
    const int ni = Kg / 256;
    const double inv_kg = 1.0 / (double)Kg;
    const int pieces = Kg * (int)sizeof(TX) / 512;             // 16-byte pieces per lane
    const bool staged = Kg * (int)sizeof(TX) <= kStageBytes;
    for (int g = 0; g < a.G; ++g) {
      const uint4* seg = reinterpret_cast<const uint4*>(xt + (int64_t)g * Kg);
      if (staged) {
        __syncwarp();                                           // the previous group's reads are done
        for (int i = 0; i < pieces; ++i) cp_async16(slot + lane + 32 * i, seg + lane + 32 * i);
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncwarp();
        seg = slot;
      }
      const RowStats st = row_stats<TX>(seg, ni, lane, a.ln_eps, inv_kg);
      const double lo = ((double)st.xlo - st.mean) * st.rstd, hi = ((double)st.xhi - st.mean) * st.rstd;
      double gam, et;
      scope_gamma_eta(a.mode, lo, hi, gam, et);
      const RowMap map = row_map(a.mode, st.mean, st.rstd, gam, et, st.xlo, st.xhi);
      int8_t* dst = codes + warp * stride + (int64_t)g * Kg;
      row_store_codes<TX>(seg, ni, lane, map, dst);
      __syncwarp();
      int cs = 0;
      for (int i = 0; i < ni; ++i) {
        const uint2 c = *reinterpret_cast<const uint2*>(dst + (size_t)(lane + 32 * i) * 8);
        cs = __dp4a((int)c.x, 0x01010101, cs);
        cs = __dp4a((int)c.y, 0x01010101, cs);
      }
      cs = warp_sum(cs);
      if (lane == 0) { sh.csum[warp][g] = cs; sh.gamma[warp][g] = (float)gam; sh.eta[warp][g] = (float)et; }
    }
  }
  __syncthreads();

  // 3. rows.  Lanes of absent tokens read zeros.
  const bool tok_ok = g8 < a.M;
  const unsigned char* brow = tok_ok ? reinterpret_cast<const unsigned char*>(codes) + g8 * stride : smem;
  const uint32_t bmask = tok_ok ? 0xFFFFFFFFu : (uint32_t)(kZeroBytes - 1);
  const bool correct = a.eta_correction != 0;
  TY* y = reinterpret_cast<TY*>(a.y);
  float out[4] = {0.f, 0.f, 0.f, 0.f};
  int acc[8][4];
  while (valid(cur)) {
    const Item nn = next(nxt);
    const int64_t r0 = cur.tile * kTileRows;
    const int g = cur.t / nbg;
    const int b0 = first_block(cur), nb = num_blocks(cur);
    if (cur.t % nbg == 0) {                                    // a group starts
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[j][c] = 0;
    }
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
        for (int j = 0; j < 8; ++j) {
          const uint32_t m = 0x01010101u << j;
          const uint32_t af[4] = {wa[i][0] & m, wa[i][1] & m, wa[i][2] & m, wa[i][3] & m};
          mma_s8s8(acc[j], af, bl[j], bh[j]);
        }
      }
    }
    // the next item's weights move up; the one after it starts loading
#pragma unroll
    for (int i = 0; i < kPreload; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) wa[i][c] = wb[i][c];
    if (valid(nn)) load_item(nn, wb);
    if (cur.t % nbg == nbg - 1) {                              // the group is complete: fold and rescale
      const float beta_g = a.beta[g];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int s = 0;
#pragma unroll
        for (int j = 0; j < 7; ++j) s += acc[j][c] >> j;
        s -= acc[7][c] >> 7;                                   // plane 7's bytes are 0x80 = -128 as s8
        const int tok = 2 * qd + (c & 1);
        if (tok < a.M) {
          const int dot = 2 * s - sh.csum[tok][g];
          const int64_t n = r0 + g8 + 8 * (c >> 1);
          out[c] += dequant_term(dot, beta_g, sh.gamma[tok][g], correct ? sh.eta[tok][g] : 0.f,
                                 correct ? a.rowsum[n * a.G + g] : 0, correct);
        }
      }
    }
    if (cur.t == nbt - 1) {                                    // the tile is complete
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int tok = 2 * qd + (c & 1);
        if (tok < a.M) y[(int64_t)tok * a.N + r0 + g8 + 8 * (c >> 1)] = out_cast<TY>(out[c]);
        out[c] = 0.f;
      }
    }
    cur = nxt; nxt = nn;
  }
}

template <typename TX, typename TY>
cudaError_t run2(const BatchArgs& a, cudaStream_t s) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const int64_t tiles = a.N / kTileRows;
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  const size_t smem = kZeroBytes + (size_t)kBatchWarps * kStageBytes + (size_t)a.M * (size_t)(a.K + kRowPad);
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
         kZeroBytes + (size_t)kBatchWarps * kStageBytes +
                 (size_t)(M < kBatchTokens ? M : kBatchTokens) * (size_t)(K + kRowPad) <= 220 * 1024;
}

// M tokens in launches of up to 8; later launches find the weights in L2.
cudaError_t launch_gemv_batch(const GemvArgs& g, int64_t M, cudaStream_t s) {
  const size_t xsz = g.xt == BL_F32 ? 4 : 2, ysz = g.yt == BL_F32 ? 4 : 2;
  for (int64_t m0 = 0; m0 < M; m0 += kBatchTokens) {
    BatchArgs a;
    a.x = reinterpret_cast<const char*>(g.x) + (size_t)m0 * (size_t)g.K * xsz;
    a.M = (int)(M - m0 < kBatchTokens ? M - m0 : kBatchTokens);
    a.K = g.K; a.N = g.N; a.G = g.G; a.mode = (int)g.mode; a.ln_eps = g.ln_eps; a.eta_correction = g.eta_correction;
    a.W_packed = g.W_packed; a.beta = g.beta; a.rowsum = g.rowsum;
    a.y = reinterpret_cast<char*>(g.y) + (size_t)m0 * (size_t)g.N * ysz;
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

}  // namespace bl
