// Decode for a small batch of tokens on the 5th-generation tensor cores (Sec. 2.1 per-token
// inference: Eq. 12 and 4-6 per token, Eq. 7 and 11 for the product), for callers that can lend a
// workspace.  Two kernels per call:
//
//   decode_quant_kernel   one CTA per token: LN statistics, gamma / eta and the 8-bit codes
//                         (the arithmetic of the single-token decode kernel: fp32 sums around a
//                         pilot value, one FMA per element, an exact decision near a tie),
//                         written to the workspace already in the order and swizzle in which the
//                         second kernel's MMAs read them, with gamma and the sum of the codes.
//                         Every CTA of the product kernel used to quantise every token itself:
//                         that, not the product, was most of a small-batch call.
//
//   gemv_tc_kernel        the product, transposed: y^T = W~ x~^T.  A CTA owns up to 128 weight
//                         rows (the M side of tcgen05.mma kind::i8, 128 x 16 x 32) and all of K;
//                         up to 16 (or 32) tokens are the columns.  The weights never pass through
//                         shared memory: a thread owns one row (= one lane of tensor memory),
//                         reads 256 of its weights (32 bytes) from global memory / L2, and for
//                         bit plane j forms word & (0x01010101 << j) - in DECODE layout that is
//                         four weights as bytes 0 or 2^j, one logic operation per four weights -
//                         and stores the eight registers of a plane to tensor memory
//                         (tcgen05.st), where they are the A operand (32 bytes of K per lane) of
//                         one MMA.  Each plane has its own int32 accumulator columns, so plane j
//                         sums 2^j (-128 for j = 7) times the codes under its set bits; the
//                         epilogue adds acc_j >> j over the planes (exact) and applies
//                         sum_k W~ x~ = 2 sum_{bit=1} x~ - sum x~ and the Eq. 11 rescale.
//                         The B operand (the tokens x 32 codes per MMA) comes from shared memory,
//                         copied there in one piece from the workspace.
//
// Issue rate.  One thread issues a tcgen05.mma in about 63 clocks and a commit in about 67
// whatever the shape, and several warps issue in parallel, so four issuer threads share the
// work (two planes each, every chunk), each plane's accumulator written by one thread only.
// The expanders are two groups of four warps (one warp per lane quarter): group g forms planes
// 4g..4g+3 of every chunk of 256 weights, two chunks per slot of its ring in tensor memory (three
// slots with 16 tokens, two with 32, where the accumulators take twice the columns).  The weights
// are constants of the model, so the rings are filled and the CTA's weights are requested into L2
// before the stream-order wait.  tcgen05.st moves 128 bytes per clock and SM: the 454 KB of
// expanded weights of a CTA (K 4096, 111 rows) are 3 550 clocks, the floor of this form.
//
// Waits: every mbarrier wait is bounded (tc_common.cuh); one that runs out raises the CTA's abort
// flag, everybody falls through to the end, the status word of the workspace gets BL_ERR_TIMEOUT,
// tensor memory is freed, and y is then not valid.
#include <algorithm>
#include <atomic>

#include "quant_rows.cuh"
#include "tc_common.cuh"

namespace bl {

namespace {

using namespace tc;

                                         // tokens per pass (MMA N): 16, or 32 where their codes fit in shared memory
constexpr int kQuantThreads = 256;        // with the product kernel's 384 threads on the same SM: registers for both
constexpr int kQuantWarps = kQuantThreads / 32;
constexpr int kMaxOctets = 6;            // 8-feature pieces per thread of the quantising kernel: K <= 12288
constexpr int kTcThreads = 384;          // warps 0-7 expand (0-3 also run the epilogue), 8-11 issue
constexpr int kSlotsMax = 3;             // A ring: slots per expander group (3 for 16 tokens, 2 for 32), two chunks x four planes per slot
constexpr int kSlotCols = 64;            // 2 chunks x 4 planes x 8 columns (32 bytes of K per lane and plane)
                                         // accumulators: columns [plane 8][token NT]; the A ring [group 2][slot] behind them
constexpr uint32_t kTmemCols = 512;
constexpr size_t kStatusBytes = 256;
constexpr uint32_t kCopyPiece = 16384;

// a pass: the codes of nt tokens, then gamma[nt] (float) and csum[nt] (int)
__host__ __device__ inline size_t pass_bytes(int64_t K, int nt) { return (size_t)nt * ((size_t)K + 8); }

// Where the code of feature k of token n sits in a pass's code block.  The block is B tiles of 8
// token rows x 128 bytes, [token half n / 8][tile K / 128][row n % 8][128 bytes], 128-byte swizzled
// (16-byte piece p of row n at piece p ^ (n & 7)); the MMA's descriptor strides from the tile of
// rows 0..7 to that of rows 8..15, and a pass of at most 8 tokens only moves the first half.  Inside a chunk of 256 features (8 words of 32 weights) the MMA of plane j reads,
// as its 32 bytes of K, byte i of word u at 4u + i, which is feature 32u + 4j + i: so a tile holds
// four planes of one half of a chunk.
__device__ __forceinline__ uint32_t code_offset4(int k, int n, int tiles) {   // k % 4 == 0: four codes at once
  const int c = k >> 8, u = (k >> 5) & 7, j = (k >> 2) & 7;
  const int tile = 2 * c + (j >> 2);
  const int b = 32 * (j & 3) + 4 * u;
  return (uint32_t)((((n >> 3) * tiles + tile) * 8 + (n & 7)) * 128 + ((((b >> 4) ^ (n & 7)) << 4) | (b & 15)));
}

struct QuantTokArgs {
  const void* x; int64_t K; int mode; float ln_eps;
  float inv_k; double inv_k_d;
  int nt;                   // tokens per pass
  int row_major;            // codes as plain rows [token][K] (for the bit-plane kernel) instead of MMA tiles
  uint8_t* passes;          // workspace behind the status block
  uint32_t* status;         // cleared here (in stream order); the product kernels only ever raise it
};

struct __align__(16) WarpStats { float s1, s2, lo, hi; };
constexpr float kRoundMagic = 12582912.f;   // 1.5 * 2^23: x + magic - magic is rne(x) for |x| < 2^22

// The rare element whose fp32 image f of (x - c) Q_b / span is too close to a rounding tie for fp32 to
// decide: (x - c) Q_b is compared with (n + 1/2) span in fp64, where both products are exact (x,
// span and, in the eta form, c are floats; Q_b is a power of two).  No division; an exact tie goes to
// the even neighbour.  (The same routine as in the single-token kernel.)
__device__ __noinline__ int exact_code(float x, float f, double c, double span) {
  const float nf = rintf(f - 0.5f);
  const int n = (int)nf;
  const double lhs = ((double)x - c) * (double)kQb;
  const double h = ((double)nf + 0.5) * span;
  if (lhs > h) return n + 1;
  if (lhs < h) return n;
  return n + (n & 1);
}
__device__ __noinline__ float rstd_outside_fp32(float v) { return v > 0.f ? (float)(1.0 / sqrt((double)v)) : 0.f; }

// One CTA per token.  The arithmetic of the single-token decode kernel: the codes do not need the
// variance, rne((x^ - eta) Q_b / gamma) = rne((x - c) A) with c = mean, A = Q_b / max|x - mean| (absmax)
// or c = min x, A = Q_b / (max x - min x) (eta form), all in fp32 with the sums taken around a pilot
// value; an element within the tie window is settled exactly; gamma (which does need 1/sqrt(Var + eps))
// only scales the output.
// kOct: 8-feature pieces per thread (2, 4 or 6: K up to 4096, 8192, 12288), kept in registers.
template <typename TX, int kOct>
__global__ void __launch_bounds__(kQuantThreads, 2) decode_quant_kernel(QuantTokArgs a) {
  __shared__ WarpStats red[kQuantWarps];
  __shared__ int red_c[kQuantWarps];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t m = blockIdx.x;
  const int n = (int)(m % a.nt);
  uint8_t* region = a.passes + (size_t)(m / a.nt) * pass_bytes(a.K, a.nt);
  // The product kernel may start on the weights.  Measured: the bit-plane kernel does best released at
  // once, the tensor-core kernel released once this kernel's own stream-order wait has returned (its 148
  // CTAs then do not set up and prefetch while the kernel before this one is still finishing).
  if (a.row_major) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (!a.row_major) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (m == 0 && threadIdx.x == 0) *a.status = 0u;
  const uint4* slot = reinterpret_cast<const uint4*>(reinterpret_cast<const TX*>(a.x) + m * a.K);
  const int octets = (int)(a.K / 8);
  const bool ln = a.ln_eps >= 0.f;

  // ---- Eq. 12 sums around a pilot value (mean of the first 8 features), raw extremes -----------------
  float xv[kOct][8];
  float pilot;
  {
    rows::Chunk<TX> ch; float v[8];
    ch.load(slot, 0); ch.unpack(v);
    pilot = 0.125f * (((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7])));
    if (!ln) pilot = 0.f;
  }
  float s1 = 0.f, s2 = 0.f, mn = INFINITY, mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < kOct; ++i) {
    const int c = threadIdx.x + kQuantThreads * i;
    if (c < octets) {
      rows::Chunk<TX> ch;
      ch.load(slot, c); ch.unpack(xv[i]);
      float d[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) { d[j] = xv[i][j] - pilot; mn = fminf(mn, xv[i][j]); mx = fmaxf(mx, xv[i][j]); }
      s1 += ((d[0] + d[1]) + (d[2] + d[3])) + ((d[4] + d[5]) + (d[6] + d[7]));
      float p0 = d[0] * d[0], p1 = d[1] * d[1];
#pragma unroll
      for (int j = 2; j < 8; j += 2) { p0 = fmaf(d[j], d[j], p0); p1 = fmaf(d[j + 1], d[j + 1], p1); }
      s2 += p0 + p1;
    }
  }
  s1 = warp_sum(s1); s2 = warp_sum(s2); mn = warp_min(mn); mx = warp_max(mx);
  if (lane == 0) red[warp] = WarpStats{s1, s2, mn, mx};
  __syncthreads();
  float t1 = 0.f, t2 = 0.f, xlo = INFINITY, xhi = -INFINITY;
  {
    float4 w[kQuantWarps];
#pragma unroll
    for (int i = 0; i < kQuantWarps; ++i) w[i] = *reinterpret_cast<const float4*>(&red[i]);
#pragma unroll
    for (int i = 0; i < kQuantWarps; i += 4) {               // a fixed order, the same in every thread
      t1 += (w[i].x + w[i + 1].x) + (w[i + 2].x + w[i + 3].x);
      t2 += (w[i].y + w[i + 1].y) + (w[i + 2].y + w[i + 3].y);
      xlo = fminf(xlo, fminf(fminf(w[i].z, w[i + 1].z), fminf(w[i + 2].z, w[i + 3].z)));
      xhi = fmaxf(xhi, fmaxf(fmaxf(w[i].w, w[i + 1].w), fmaxf(w[i + 2].w, w[i + 3].w)));
    }
  }
  // ---- the code map ------------------------------------------------------------------------------------
  const float off = ln ? t1 * a.inv_k : 0.f;            // mean - pilot
  const float mean_f = pilot + off;
  const float cf = (a.mode == BL_ABSMAX) ? mean_f : xlo;
  const float span_f = (a.mode == BL_ABSMAX) ? fmaxf(fabsf(xlo - mean_f), fabsf(xhi - mean_f)) : xhi - xlo;
  float Af = 0.f;                                        // a constant token has gamma = 0: all codes are 0
  if (span_f > 0.f) {
    const float y = __frcp_rn(span_f);
    Af = (float)kQb * (y * (2.f - span_f * y));
  }
  const float Bf = -cf * Af;
  const float tau = 1e-6f * (fabsf(Af) * fmaxf(fabsf(xlo), fabsf(xhi)) + fabsf(Bf) + 1.0f);
  const float near = 0.5f - tau;
  const float lo_f = (a.mode == BL_ABSMAX) ? -(float)kCodeMax : 0.f;

  // ---- Eq. 4 / 6: codes, written where the product kernel's MMAs read them ---------------------------
  int csum = 0;
#pragma unroll
  for (int i = 0; i < kOct; ++i) {
    const int c = threadIdx.x + kQuantThreads * i;
    if (c < octets) {
      uint32_t tb[8];
      bool near_tie = false;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float f = fminf(fmaxf(fmaf(xv[i][j], Af, Bf), lo_f), (float)kCodeMax);   // the clip commutes with rne
        const float t = f + kRoundMagic;
        tb[j] = __float_as_uint(t);
        near_tie |= fabsf(f - (t - kRoundMagic)) > near;
      }
      if (near_tie && span_f > 0.f) {                                    // rare: settle the close ones exactly
        const double mean = (double)pilot + (ln ? (double)t1 * a.inv_k_d : 0.0);
        const double cd = (a.mode == BL_ABSMAX) ? mean : (double)xlo;
        const double span = (a.mode == BL_ABSMAX) ? fmax(fabs((double)xlo - mean), fabs((double)xhi - mean))
                                                  : (double)xhi - (double)xlo;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float f = fmaf(xv[i][j], Af, Bf);                        // unclipped: a clipped one is never close
          if (f > lo_f && f < (float)kCodeMax && fabsf(f - rintf(f)) > near)
            tb[j] = (uint32_t)max((int)lo_f, min(kCodeMax, exact_code(xv[i][j], f, cd, span)));
        }
      }
      const uint32_t w0 = __byte_perm(__byte_perm(tb[0], tb[1], 0x0040), __byte_perm(tb[2], tb[3], 0x0040), 0x5410);
      const uint32_t w1 = __byte_perm(__byte_perm(tb[4], tb[5], 0x0040), __byte_perm(tb[6], tb[7], 0x0040), 0x5410);
      if (a.row_major) {
        *reinterpret_cast<uint2*>(region + (size_t)n * (size_t)a.K + (size_t)c * 8) = make_uint2(w0, w1);
      } else {
        const uint32_t offb = code_offset4(8 * c, n, (int)(a.K / 128));     // features 8c..8c+3; 8c+4..8c+7 are the next plane, 32 bytes on
        *reinterpret_cast<uint32_t*>(region + offb) = w0;
        *reinterpret_cast<uint32_t*>(region + (offb ^ 32u)) = w1;
      }
      csum = __dp4a((int)w0, 0x01010101, csum);
      csum = __dp4a((int)w1, 0x01010101, csum);
    }
  }
  csum = __reduce_add_sync(0xFFFFFFFFu, csum);
  if (lane == 0) red_c[warp] = csum;
  if (threadIdx.x == kQuantThreads - 32) {          // (a warp that does not close the kernel)
    // gamma of Eq. 5 / 6 on x^ = (x - mean) rstd: only the final rescale reads it
    float rstd = 1.f;
    if (ln) {
      const float var_f = fmaxf(fmaf(-off, off, t2 * a.inv_k), 0.f);
      const float vv = var_f + a.ln_eps;
      if (vv > 1e-30f && vv < 1e30f) {
        const float y = rsqrtf(vv);
        rstd = y * (1.5f - 0.5f * vv * y * y);
      } else {
        rstd = rstd_outside_fp32(vv);
      }
    }
    reinterpret_cast<float*>(region + (size_t)a.nt * (size_t)a.K)[n] = span_f * rstd;
  }
  __syncthreads();
  if (warp == 0) {
    const int t = __reduce_add_sync(0xFFFFFFFFu, lane < kQuantWarps ? red_c[lane] : 0);
    if (lane == 0) reinterpret_cast<int*>(region + (size_t)a.nt * (size_t)a.K)[a.nt + n] = t;
  }
}

// ---- the product ------------------------------------------------------------------------------------
struct TcArgs {
  const uint8_t* W; int64_t K, N; int rows_per_cta;
  const uint8_t* region;     // codes of this pass | gamma[NT] | csum[NT]
  const float* beta;
  void* y; int64_t m0; int mcount;
  uint32_t* status;
};

struct TcShared {
  unsigned long long full[2][kSlotsMax], empty[2][kSlotsMax], codes_full, acc_full;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// D (tensor memory) += A (tensor memory: one row of 32 bytes per lane) x B (shared memory descriptor)
__device__ __forceinline__ void mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// K-major tile with 128-byte rows and 128-byte swizzle whose 8-row groups lie `sbo` bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128_sbo(uint32_t addr, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// NT: tokens per pass, 16 or 32.
template <typename TY, int NT>
__global__ void __launch_bounds__(kTcThreads, 1) gemv_tc_kernel(TcArgs a) {
  // kind::i8 instruction descriptor: s32 accumulate, s8 x s8, both operands K-major, 128 x NT.
  constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NT >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  constexpr uint32_t kColA = 8u * NT;
  constexpr int kSlots = (int)((kTmemCols - kColA) / (2 * kSlotCols));
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* codes = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ TcShared sh;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  volatile int* abort_flag = &sh.abort_flag;
  const int64_t Kb = a.K / 8;
  const int nchunks = (int)(a.K / 256);
  const int npairs = (nchunks + 1) >> 1;
  const int64_t row_begin = (int64_t)blockIdx.x * a.rows_per_cta;
  const int rows_cta = (int)min((int64_t)a.rows_per_cta, a.N - row_begin);
  const uint32_t half_bytes = 8u * (uint32_t)a.K;          // the codes of 8 tokens: all tiles of rows 0..7, then of rows 8..15, ...

  if (threadIdx.x == 0) {
    for (int g = 0; g < 2; ++g)
      for (int i = 0; i < kSlots; ++i) { mbar_init(smem_u32(&sh.full[g][i]), 4); mbar_init(smem_u32(&sh.empty[g][i]), 2); }
    mbar_init(smem_u32(&sh.codes_full), 1);
    mbar_init(smem_u32(&sh.acc_full), 4);
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // ---- ahead of stream order: the CTA's weights on their way into L2, tensor memory, the A ring ----
  {
    const uint8_t* base = a.W + row_begin * Kb;
    const int64_t total = (int64_t)rows_cta * Kb;
    for (int64_t off = (int64_t)threadIdx.x * kCopyPiece; off < total; off += (int64_t)kTcThreads * kCopyPiece) {
      const uint32_t sz = (uint32_t)min((int64_t)kCopyPiece, total - off);
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(base + off), "r"(sz) : "memory");
    }
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&sh.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp < 8) {
    // ------------------------------------------------------------------ expanders: one weight row per thread;
    // group g (warps 4g..4g+3, one per lane quarter) writes planes 4g..4g+3 of every chunk, two chunks per slot
    const int qtr = warp & 3, g = warp >> 2;
    const int row = qtr * 32 + lane;
    const uint8_t* wrow = a.W + (row_begin + min(row, rows_cta - 1)) * Kb;
    const uint32_t lane_base = (uint32_t)(qtr * 32) << 16;
    uint32_t mask[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) mask[jj] = 0x01010101u << (4 * g + jj);
    uint4 cur[4], nxt[4];
    auto fetch = [&](int p, uint4 (&v)[4]) {
#pragma unroll
      for (int i = 0; i < 4; ++i) v[i] = make_uint4(0u, 0u, 0u, 0u);
      if (2 * p < nchunks) {
        v[0] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)p * 64));
        v[1] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)p * 64 + 16));
      }
      if (2 * p + 1 < nchunks) {
        v[2] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)p * 64 + 32));
        v[3] = __ldg(reinterpret_cast<const uint4*>(wrow + (size_t)p * 64 + 48));
      }
    };
    fetch(0, cur);
    int slot = 0; uint32_t phase = 0;
    for (int p = 0; p < npairs; ++p) {
      fetch(p + 1, nxt);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(smem_u32(&sh.empty[g][slot]), phase ^ 1u, abort_flag);
      ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      const uint32_t abase = tmem_base + lane_base + kColA + (uint32_t)(g * kSlots + slot) * kSlotCols;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const uint32_t w[8] = {cur[2 * cc].x, cur[2 * cc].y, cur[2 * cc].z, cur[2 * cc].w,
                               cur[2 * cc + 1].x, cur[2 * cc + 1].y, cur[2 * cc + 1].z, cur[2 * cc + 1].w};
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          uint32_t r[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) r[u] = w[u] & mask[jj];
          tmem_st8(abase + (uint32_t)(cc * 32 + jj * 8), r);
        }
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh.full[g][slot]));
#pragma unroll
      for (int i = 0; i < 4; ++i) cur[i] = nxt[i];
      if (++slot == kSlots) { slot = 0; phase ^= 1u; }
    }
  } else if (lane == 0) {
    // ------------------------------------------------------------------ issuers: two planes each, every chunk
    const int i = warp - 8, g = i >> 1, j0 = 4 * g + 2 * (i & 1);
    const uint32_t copy_bytes = (uint32_t)((a.mcount + 7) >> 3) * half_bytes;
    if (i == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");              // the codes are the work of the kernel before
      mbar_arrive_expect_tx(smem_u32(&sh.codes_full), copy_bytes);
      for (uint32_t off = 0; off < copy_bytes; off += kCopyPiece) {
        const uint32_t sz = min(kCopyPiece, copy_bytes - off);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(codes + off)), "l"(a.region + off), "r"(sz), "r"(smem_u32(&sh.codes_full)) : "memory");
      }
    }
    bool ok = mbar_wait(smem_u32(&sh.codes_full), 0u, abort_flag);
    const uint32_t codes_addr = smem_u32(codes);
    int slot = 0; uint32_t phase = 0;
    for (int p = 0; ok && p < npairs; ++p) {
      ok = mbar_wait(smem_u32(&sh.full[g][slot]), phase, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t abase = tmem_base + kColA + (uint32_t)(g * kSlots + slot) * kSlotCols;
#pragma unroll
      for (int cc = 0; cc < 2; ++cc) {
        const int c = 2 * p + cc;
        if (c < nchunks) {
          // planes 4g..4g+3 of chunk c are tile 2c + g: 32 bytes of K per plane
          const uint64_t bdesc = smem_desc_sw128_sbo(codes_addr + (uint32_t)(2 * c + g) * 1024u, half_bytes);
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const int j = j0 + t;
            mma_i8_ts(tmem_base + (uint32_t)(j * NT), abase + (uint32_t)(cc * 32 + (j & 3) * 8),
                      bdesc + (uint64_t)(2 * (j & 3)), kIdesc, c > 0 ? 1u : 0u);
          }
        }
      }
      mma_commit(smem_u32(&sh.empty[g][slot]));
      if (++slot == kSlots) { slot = 0; phase ^= 1u; }
    }
    mma_commit(smem_u32(&sh.acc_full));
  }
  __syncwarp();

  if (warp < 4) {
    // ------------------------------------------------------------------ epilogue: thread = weight row
    asm volatile("griddepcontrol.wait;" ::: "memory");                // gamma, csum; y in stream order
    // lane n holds what token n needs (fetched while the last MMAs run)
    const float* tail = reinterpret_cast<const float*>(a.region + (uint32_t)NT * (uint32_t)a.K);
    const float my_scale = __ldg(a.beta) * tail[lane & (NT - 1)] * kInvQb;
    const int my_csum = reinterpret_cast<const int*>(tail)[NT + (lane & (NT - 1))];
    bool ok = true;
    if (lane == 0) ok = mbar_wait(smem_u32(&sh.acc_full), 0u, abort_flag);
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    tc_fence_after();
    if (ok) {
      const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
      const int row = warp * 32 + lane;
      TY* y = reinterpret_cast<TY*>(a.y);
#pragma unroll 1
      for (int n0 = 0; n0 < NT && n0 < a.mcount; n0 += 16) {         // 16 tokens (accumulator columns) at a time
        int S[16];
#pragma unroll
        for (int n = 0; n < 16; ++n) S[n] = 0;
#pragma unroll
        for (int jb = 0; jb < 8; jb += 4) {
          uint32_t d[4][16];
#pragma unroll
          for (int t = 0; t < 4; ++t) tmem_ld16_nowait(tmem_base + lane_base + (uint32_t)((jb + t) * NT + n0), d[t]);
          tmem_ld_wait();
          // plane j holds 2^j * (sum of the codes under its set bits); the byte 0x80 of plane 7 is -128
#pragma unroll
          for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int n = 0; n < 16; ++n) S[n] += (jb + t < 7) ? ((int)d[t][n] >> (jb + t)) : -((int)d[t][n] >> 7);
        }
#pragma unroll
        for (int n = 0; n < 16; ++n) {
          const float sc = __shfl_sync(0xFFFFFFFFu, my_scale, n0 + n);
          const int cs = __shfl_sync(0xFFFFFFFFu, my_csum, n0 + n);
          // Eq. 7 and 11: (2 S - sum x~) beta gamma / Q_b
          if (n0 + n < a.mcount && row < rows_cta)
            y[(a.m0 + n0 + n) * a.N + row_begin + row] = out_cast<TY>((float)(2 * S[n] - cs) * sc);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (sh.abort_flag) {
    // something gave up: let what may still be in flight finish (bounded), then report
    if (threadIdx.x == 256) {
      mbar_wait(smem_u32(&sh.codes_full), 0u, abort_flag);
      mbar_wait(smem_u32(&sh.acc_full), 0u, abort_flag);
      atomicExch(a.status, (uint32_t)BL_ERR_TIMEOUT);
    }
    __syncthreads();
    tc_fence_after();
  }
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

template <typename Kern, typename Args>
cudaError_t launch_pdl(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, args);
}

template <typename TX, typename TY>
cudaError_t run(const GemvArgs& a, int64_t M, void* ws, cudaStream_t s) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  // One product CTA per SM at a time: a CTA holds all of the SM's tensor memory until it ends, so a
  // second one on the same SM (the next call's, or one displaced from an SM that is full) would sit in
  // tcgen05.alloc behind it and then start with an empty ring.  Asking for more than half of the
  // shared memory keeps them apart; a waiting CTA then takes the first SM that frees up.
  const int nt = (M > 16 && (size_t)32 * (size_t)a.K + 1024 <= 200 * 1024) ? 32 : 16;
  const size_t smem = std::max<size_t>((size_t)nt * (size_t)a.K + 1024, 116 * 1024);
  static std::atomic<int> configured[64];
  if (dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    e = cudaFuncSetAttribute(gemv_tc_kernel<TY, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemv_tc_kernel<TY, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024);
    if (e != cudaSuccess) return e;
    if (dev < 64) configured[dev].store(1, std::memory_order_release);
  }
  uint8_t* base = reinterpret_cast<uint8_t*>(ws);
  QuantTokArgs qa{a.x, a.K, (int)a.mode, a.ln_eps, (float)(1.0 / (double)a.K), 1.0 / (double)a.K, nt, 0, base + kStatusBytes,
                  reinterpret_cast<uint32_t*>(base)};
  const int64_t per_thread = (a.K / 8 + kQuantThreads - 1) / kQuantThreads;
  if (per_thread <= 2) e = launch_pdl(decode_quant_kernel<TX, 2>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  else if (per_thread <= 4) e = launch_pdl(decode_quant_kernel<TX, 4>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  else e = launch_pdl(decode_quant_kernel<TX, 6>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  if (e != cudaSuccess) return e;
  const int rows_per_cta = (int)std::min<int64_t>(128, (a.N + sms - 1) / sms);
  const unsigned grid = (unsigned)((a.N + rows_per_cta - 1) / rows_per_cta);
  for (int64_t m0 = 0; m0 < M; m0 += nt) {
    TcArgs ta{a.W_packed, a.K, a.N, rows_per_cta, base + kStatusBytes + (size_t)(m0 / nt) * pass_bytes(a.K, nt), a.beta,
              a.y, m0, (int)std::min<int64_t>(nt, M - m0), reinterpret_cast<uint32_t*>(base)};
    e = nt == 32 ? launch_pdl(gemv_tc_kernel<TY, 32>, dim3(grid), dim3(kTcThreads), smem, s, ta)
                 : launch_pdl(gemv_tc_kernel<TY, 16>, dim3(grid), dim3(kTcThreads), smem, s, ta);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Up to 8 tokens: the same quantising kernel (codes as plain rows), then the bit-plane kernel of
// gemv_batch.cu told to take codes, gamma and the code sums from the workspace instead of computing them
// in every CTA.
template <typename TX>
cudaError_t run_small(const GemvArgs& a, int64_t M, void* ws, cudaStream_t s) {
  uint8_t* base = reinterpret_cast<uint8_t*>(ws);
  uint8_t* region = base + kStatusBytes;
  QuantTokArgs qa{a.x, a.K, (int)a.mode, a.ln_eps, (float)(1.0 / (double)a.K), 1.0 / (double)a.K, (int)M, 1, region,
                  reinterpret_cast<uint32_t*>(base)};
  const int64_t per_thread = (a.K / 8 + kQuantThreads - 1) / kQuantThreads;
  cudaError_t e;
  if (per_thread <= 2) e = launch_pdl(decode_quant_kernel<TX, 2>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  else if (per_thread <= 4) e = launch_pdl(decode_quant_kernel<TX, 4>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  else e = launch_pdl(decode_quant_kernel<TX, 6>, dim3((unsigned)M), dim3(kQuantThreads), 0, s, qa);
  if (e != cudaSuccess) return e;
  const float* gamma = reinterpret_cast<const float*>(region + (size_t)M * (size_t)a.K);
  return launch_gemv_batch_pre(a, M, reinterpret_cast<const int8_t*>(region), gamma, reinterpret_cast<const int*>(gamma) + M, s);
}

template <typename TX>
cudaError_t run1(const GemvArgs& a, int64_t M, void* ws, cudaStream_t s) {
  if (M <= 8) return run_small<TX>(a, M, ws, s);
  switch (a.yt) {
    case BL_F32: return run<TX, float>(a, M, ws, s);
    case BL_F16: return run<TX, __half>(a, M, ws, s);
    case BL_BF16: return run<TX, __nv_bfloat16>(a, M, ws, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

bool gemv_tc_supported(int64_t M, int64_t K, int64_t N, int G, int eta_correction) {
  return M >= 2 && G == 1 && !eta_correction && K % 256 == 0 && N % 16 == 0 && N > 0 &&
         K <= (int64_t)kMaxOctets * kQuantThreads * 8 && (M > 8 || gemv_batch_supported(M, K, N, G));
}

size_t gemv_tc_ws_bytes(int64_t M, int64_t K) {
  return kStatusBytes + (size_t)((M + 31) / 32) * pass_bytes(K, 32);      // covers passes of 16 as well
}

cudaError_t launch_gemv_tc(const GemvArgs& a, int64_t M, void* ws, cudaStream_t s) {
  switch (a.xt) {
    case BL_F32: return run1<float>(a, M, ws, s);
    case BL_F16: return run1<__half>(a, M, ws, s);
    case BL_BF16: return run1<__nv_bfloat16>(a, M, ws, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl
