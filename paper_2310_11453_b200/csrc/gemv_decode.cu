// Batch-1 decode: LN + Quant of the single token (Eq. 12, 4-6) and the 1-bit x 8-bit product
// with its rescale (Eq. 7, 11) in one kernel.  Bound by streaming the packed weights
// (N*K/8 bytes) once from HBM; everything else is a few KB.
//
// A call is short (microseconds), so what sits between two calls on a stream decides the rate.
// The kernel is therefore split at griddepcontrol.wait (programmatic dependent launch):
//
//   ahead of stream order, while the call before it is still computing, a CTA brings its whole
//   slice of the packed weights on chip: bulk copies (cp.async.bulk, no multicast) into a ring of
//   shared-memory stages, each completing on an mbarrier.  The weights are constants of the
//   model, which is what makes reading them early legal; x, beta, rowsum and y are only touched
//   after the wait.  The token's cache lines are requested into L2 (a hint, no architectural effect).
//
//   in stream order: x -> fp32 in shared memory with the sums and extremes taken on the way; one
//   block barrier; codes = rne((x - c) A) with c, A from mean and extremes only (see below); a
//   second block barrier; each lane takes the 128 codes of its chunk into registers and walks the
//   rows of its warp out of shared memory; results go straight to y.
//
// The codes do not depend on the variance:
//   rne((x^ - eta) Q_b / gamma) = rne((x - c) A),  c = mean, A = Q_b / max|x - mean|  (absmax)
//                                                  c = min x, A = Q_b / (max x - min x) (eta form)
// so the chain from x to the codes is one block reduction, one reciprocal and one FMA per element;
// gamma and eta (which do need 1/sqrt(Var + eps)) are only used by the final rescale.
//
// Row product.  DECODE layout: row-major like CANONICAL, but inside every 32-weight word weight q
// sits at bit q/4 + 8*(q%4).  Then word & (0x01010101 << j) holds weights 4j..4j+3 as bytes that
// are 0 or 2^j, and one dp4a against the matching four codes adds 2^j * (their masked sum): two
// instructions per four weights (a logic op and a dot product, on different pipes).  The eight
// partial sums of a chunk are folded as sum_j acc_j * 2^(7-j) = 128 * (masked sum), and
// sum_k W~[n,k] x~[k] = 2 * sum_{bit=1} x~[k] - sum_k x~[k].
//
// Work split.  The grid splits the N rows evenly over the SMs.  Inside a CTA a row of more than
// 4096 weights is shared by several warps (slices of 4096), so the 8 warps form `rowslots` row
// slots; the CTA's rows are cut into stages of rpw <= 8 consecutive rows per row slot, one stage
// per ring slot.  A warp takes its rows one per iteration of a loop that is not unrolled: the kernel
// runs every instruction only a few times per call, so fetching them is what costs, and the body of
// this loop is the one part that repeats.
//
// Waits.  The only spin in the kernel is the wait for a stage's barrier.  It is bounded; when the
// limit runs out the warp reads that stage (and every later one) directly from global memory
// instead, so the result is the same, and before the CTA exits one thread waits, again with a
// limit, for the copies that were still in flight.
#include <algorithm>
#include <atomic>

#include "quant_core.cuh"

namespace bl {

namespace {

constexpr int kGemvThreads = 256;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kBatchRows = 8;            // most rows per warp and stage
constexpr int kSlice = 4096;             // weights per warp slice = 32 lanes x 128
constexpr int kMaxStages = 4;            // most ring slots
constexpr uint32_t kRingBytes = 64 * 1024;
constexpr float kRoundMagic = 12582912.f;   // 1.5 * 2^23: x + magic - magic is rne(x) for |x| < 2^22
constexpr unsigned long long kDrainNs = 2000000000ull;   // limit of the wait for copies in flight at exit
constexpr unsigned long long kStageWaitNs = 1000000000ull;   // limit of the wait for one stage
constexpr uint32_t kStagePolls = 1u << 22;               // and its limit in polls

// Profiling hook, compiled out unless BL_GEMV_STAMPS is defined: thread 0 of two CTAs records the
// SM clock at the points marked BL_STAMP(i) (and the global timer at entry, after the stream-order
// wait and at the end), one record per launch in a small ring, read back by a debug accessor.
#ifdef BL_GEMV_STAMPS
constexpr int kStampSlots = 64, kStampPoints = 32;
struct StampRecord { unsigned long long ns[3]; long long clk[kStampPoints]; };
__device__ StampRecord g_stamps[2][kStampSlots];
__device__ unsigned int g_stamp_launch[2];
#define BL_STAMP_DECL \
  const int stamp_cta = blockIdx.x == 0 ? 0 : (blockIdx.x == gridDim.x / 2 ? 1 : -1); \
  StampRecord* stamp_rec = nullptr; \
  if (stamp_cta >= 0 && threadIdx.x == 0) \
    stamp_rec = &g_stamps[stamp_cta][atomicAdd(&g_stamp_launch[stamp_cta], 1u) % kStampSlots];
#define BL_STAMP(i) do { if (stamp_rec) stamp_rec->clk[i] = clock64(); } while (0)
#define BL_STAMP_NS(i) do { if (stamp_rec) stamp_rec->ns[i] = global_ns(); } while (0)
#else
#define BL_STAMP_DECL
#define BL_STAMP(i) do {} while (0)
#define BL_STAMP_NS(i) do {} while (0)
#endif

struct __align__(16) WarpStats { float s1, s2, lo, hi; };   // read back as one 16-byte word
struct GroupStats { double mean; float mean_f, span_f, xlo, t2; };

struct GemvShared {
  WarpStats red[kGemvWarps];
  unsigned long long full[kMaxStages];   // one mbarrier per ring slot: the stage's bytes have landed
  int done[kMaxStages];                  // warps that have finished reading the slot's current stage
  int issued[kMaxStages];                // copies issued into the slot so far
  int abandon;                           // a wait ran out: no further copies, read from global memory
  GroupStats grp[BL_MAX_GROUPS];
  float gamma[BL_MAX_GROUPS], eta[BL_MAX_GROUPS];
  int csum[BL_MAX_GROUPS];               // sum of the codes of a group
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
// The rare element whose fp32 image f of (x - c) Q_b / span is too close to a rounding tie for fp32 to
// decide: f lies within the tie window of n + 1/2, and (x - c) Q_b is compared with (n + 1/2) span in
// fp64, where both products are exact (x, span and, in the eta form, c are floats; Q_b is a power of
// two).  No division; an exact tie goes to the even neighbour.  Out of line: the common path
// should not have to be fetched around it.
__device__ __noinline__ int exact_code(float x, float f, double c, double span) {
  const float nf = rintf(f - 0.5f);
  const int n = (int)nf;
  const double lhs = ((double)x - c) * (double)kQb;
  const double h = ((double)nf + 0.5) * span;
  if (lhs > h) return n + 1;
  if (lhs < h) return n;
  return n + (n & 1);
}

// 1 / sqrt(v) for v outside the range where the fp32 approximation is safe (out of line: rare).
__device__ __noinline__ float rstd_outside_fp32(float v) { return v > 0.f ? (float)(1.0 / sqrt((double)v)) : 0.f; }

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

// ---- ring of weight stages ---------------------------------------------------------------------------
__device__ unsigned int g_fallbacks;          // warps whose wait for a weight stage ran out (since last read)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool bar_poll(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// At most `polls` further polls after the first one, and at most kStageWaitNs on the clock; false
// when the phase has still not completed.
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, uint32_t polls) {
  if (bar_poll(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t it = 0; it < polls; ++it) {
    if (bar_poll(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kStageWaitNs) return false;
    }
  }
  return false;
}

struct GemvGeom {            // decided on the host
  int rows_per_cta, rpw, nstages, nslices, rowslots;
  int depth;                 // ring slots in use (<= kMaxStages)
  uint32_t stage_stride;     // bytes between ring slots (a multiple of 128)
  uint32_t ring_bytes;       // depth * stage_stride
  uint32_t wait_polls;       // polls of a stage barrier before the warp falls back to global loads (0: at once)
  uint32_t inv_nslices, inv_group_chunks;   // ceil(2^16 / d): (v * inv) >> 16 == v / d for v < 256
  double inv_kg;
};

template <typename TX, typename TY>
__global__ void __launch_bounds__(kGemvThreads, 2)
gemv_decode_kernel(GemvArgs a, GemvGeom geo) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ GemvShared sh;
  unsigned char* ring = smem_raw;                                                  // [depth][stage_stride]
  float* xf = reinterpret_cast<float*>(smem_raw + geo.ring_bytes);                 // [K] raw x
  int8_t* codes = reinterpret_cast<int8_t*>(smem_raw + geo.ring_bytes + a.K * sizeof(float));   // [nslices * 4096]
  const int K = (int)a.K, G = a.G, Kg = K / G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t Kb = a.K / 8;
  const int rpw = geo.rpw, nslices = geo.nslices, rowslots = geo.rowslots, depth = geo.depth;
  const int stage_rows = rpw * rowslots;
  const int64_t row_begin = (int64_t)blockIdx.x * geo.rows_per_cta;
  const int64_t row_end = min((int64_t)a.N, row_begin + geo.rows_per_cta);
  const int rows_cta = (int)(row_end - row_begin);
  // stages that hold rows of this CTA (the last CTA has fewer rows than the others): a stage without
  // rows gets no copy, so nobody may wait for one
  const int nstages = min(geo.nstages, (rows_cta + stage_rows - 1) / stage_rows);
  const uint8_t* wslice = a.W_packed + row_begin * Kb;

  // Copy of stage st into its ring slot; called by one thread once every reader of the slot's
  // previous stage is done with it.
  auto issue_stage = [&](int st) {
    const int slot = st % depth;
    const int rows = min(stage_rows, rows_cta - st * stage_rows);
    if (rows <= 0) return;
    const uint32_t bytes = (uint32_t)rows * (uint32_t)Kb;                          // a multiple of 32
    const uint32_t bar = smem_u32(&sh.full[slot]);
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");                   // earlier reads of the slot come first
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(ring + (size_t)slot * geo.stage_stride)), "l"(wslice + (int64_t)st * stage_rows * Kb),
          "r"(bytes), "r"(bar), "l"(policy) : "memory");
    sh.issued[slot] += 1;
  };

  BL_STAMP_DECL
  BL_STAMP_NS(0);
  BL_STAMP(0);
  // ---- ahead of stream order: this CTA's weights on their way into shared memory --------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh.full[i])));
      sh.done[i] = 0;
      sh.issued[i] = 0;
    }
    sh.abandon = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int st = 0; st < depth && st < nstages; ++st) issue_stage(st);
  }
  if (threadIdx.x < BL_MAX_GROUPS) sh.csum[threadIdx.x] = 0;
  if (blockIdx.x < 4) {
    const char* xb = reinterpret_cast<const char*>(a.x);
    for (int64_t off = (int64_t)threadIdx.x * 128; off < a.K * (int64_t)sizeof(TX); off += (int64_t)kGemvThreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(xb + off));
  }
  BL_STAMP(1);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  BL_STAMP_NS(1);
  BL_STAMP(2);

  // ---- x first (the chain to the codes hangs on it), staged as fp32 ------------------------------
  const TX* x = reinterpret_cast<const TX*>(a.x);
  float s1 = 0.f, s2 = 0.f;
  float mn = INFINITY, mx = -INFINITY;
  // two chunks of a thread are in flight before either is used (one L2 round trip for K <= 4096)
#pragma unroll 1
  for (int k = threadIdx.x * 8; k < K; k += 2 * kGemvThreads * 8) {
    const int k2 = k + kGemvThreads * 8;
    float v[8], u[8];
    Elem<TX>::load8(x + k, v);
    if (k2 < K) Elem<TX>::load8(x + k2, u);
    *reinterpret_cast<float4*>(xf + k) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(xf + k + 4) = make_float4(v[4], v[5], v[6], v[7]);
    if (G == 1) accumulate8(v, s1, s2, mn, mx);
    if (k2 < K) {
      *reinterpret_cast<float4*>(xf + k2) = make_float4(u[0], u[1], u[2], u[3]);
      *reinterpret_cast<float4*>(xf + k2 + 4) = make_float4(u[4], u[5], u[6], u[7]);
      if (G == 1) accumulate8(u, s1, s2, mn, mx);
    }
  }

  BL_STAMP(3);
  // ---- work split inside the CTA --------------------------------------------------------------------
  const int rowslot = (int)(((uint32_t)warp * geo.inv_nslices) >> 16);   // rows side by side
  const int slice = warp - rowslot * nslices;                            // warps that share a row
  const int chunk = slice * 32 + lane;                                   // 128-weight chunk of this lane
  const bool warp_on = rowslot < rowslots;                               // 8 is not a multiple of every slice count
  const bool active = chunk * 128 < K && warp_on;
  const int my_group = active ? (int)(((uint32_t)chunk * geo.inv_group_chunks) >> 16) : 0;
  const float beta_mine = __ldg(a.beta + my_group);

  // ---- steps 1-2 on the token: LN per group, gamma/eta, codes ------------------------------------
  const bool ln = a.ln_eps >= 0.f;
  if (G == 1) {
    s1 = warp_sum(s1); s2 = warp_sum(s2); mn = warp_min(mn); mx = warp_max(mx);
    if (lane == 0) sh.red[warp] = WarpStats{s1, s2, mn, mx};
  }
  __syncthreads();                                     // raw x (and, for one group, the warp totals) visible
  BL_STAMP(4);
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
      s1 = warp_sum(s1); s2 = warp_sum(s2); mn = warp_min(mn); mx = warp_max(mx);
      if (lane == 0) sh.red[warp] = WarpStats{s1, s2, mn, mx};
      __syncthreads();
    }
    WarpStats ws[kGemvWarps];
#pragma unroll
    for (int w = 0; w < kGemvWarps; ++w) {
      const float4 t = *reinterpret_cast<const float4*>(&sh.red[w]);
      ws[w] = WarpStats{t.x, t.y, t.z, t.w};
    }
    double t1 = 0.0;
#pragma unroll
    for (int w = 0; w < kGemvWarps; w += 4)
      t1 += ((double)ws[w].s1 + (double)ws[w + 1].s1) + ((double)ws[w + 2].s1 + (double)ws[w + 3].s1);
    float xlo = ws[0].lo, xhi = ws[0].hi;
#pragma unroll
    for (int w = 1; w < kGemvWarps; ++w) { xlo = fminf(xlo, ws[w].lo); xhi = fmaxf(xhi, ws[w].hi); }
    // location c and slope A of the code map (see the header).  The fast path only needs fp32
    // images of A and B = -c A (its error is covered by the tie window tau); the exact fp64
    // values are rebuilt inside the slow path.
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
    int csum = 0;
    // four elements per thread and iteration, not unrolled: the loop body is fetched once
#pragma unroll 1
    for (int k = threadIdx.x * 4; k < Kg; k += kGemvThreads * 4) {
      const float4 p = *reinterpret_cast<const float4*>(seg + k);
      const float v[4] = {p.x, p.y, p.z, p.w};
      int code[4];
      bool near_tie = false;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float f = fmaf(v[i], Af, Bf);
        const float t = f + kRoundMagic;                               // rne(f) in the low mantissa bits
        const float r = t - kRoundMagic;
        code[i] = __float_as_int(t) - __float_as_int(kRoundMagic);
        near_tie |= fabsf(fabsf(f - r) - 0.5f) < tau;
      }
      if (near_tie && span_f > 0.f) {                                  // rare: settle the close ones exactly
        const double c = (a.mode == BL_ABSMAX) ? mean : (double)xlo;
        const double span = (a.mode == BL_ABSMAX) ? fmax(fabs((double)xlo - mean), fabs((double)xhi - mean))
                                                  : (double)xhi - (double)xlo;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float f = fmaf(v[i], Af, Bf);
          if (fabsf(fabsf(f - rintf(f)) - 0.5f) < tau) code[i] = exact_code(v[i], f, c, span);
        }
      }
      uint32_t wq = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) wq |= (uint32_t)(max(code_lo, min(kCodeMax, code[i])) & 0xFF) << (8 * i);
      *reinterpret_cast<uint32_t*>(codes + code_slot(g * Kg + k)) = wq;
      csum = __dp4a((int)wq, 0x01010101, csum);
    }
    csum = __reduce_add_sync(0xFFFFFFFFu, csum);
    if (lane == 0 && csum != 0) atomicAdd(&sh.csum[g], csum);
    if (threadIdx.x == 0) {
      float t2 = 0.f;
#pragma unroll
      for (int w = 0; w < kGemvWarps; w += 4) t2 += (ws[w].s2 + ws[w + 1].s2) + (ws[w + 2].s2 + ws[w + 3].s2);
      sh.grp[g] = GroupStats{mean, mean_f, span_f, xlo, t2};
    }
    if (G > 1) __syncthreads();                        // sh.red is rewritten by the next group
  }
  BL_STAMP(5);
  __syncthreads();                                     // codes, code sums and group statistics visible
  BL_STAMP(6);

  // gamma and eta of Eq. 5 / 6 on x^ = (x - mean) rstd; only the final rescale reads them, so fp32
  // is enough unless the mean dwarfs the spread (then the variance is formed in fp64)
  auto group_scale = [&](int g, float& gamma, float& eta) {
    const GroupStats q = sh.grp[g];
    float rstd = 1.f;
    if (ln) {
      const float inv_f = (float)geo.inv_kg;
      const float var_f = fmaf(-q.mean_f, q.mean_f, q.t2 * inv_f);
      double var = (double)var_f;
      if (!(q.mean_f * q.mean_f <= 16.f * var_f)) var = (double)q.t2 * geo.inv_kg - q.mean * q.mean;
      if (var < 0.0) var = 0.0;
      rstd = rsqrt_scale(var + (double)a.ln_eps);
    }
    gamma = q.span_f * rstd;
    eta = (a.mode == BL_ABSMAX) ? 0.f : (q.xlo - q.mean_f) * rstd;
  };
  const bool row_terms = a.eta_correction || nslices > 1;   // rows are finished by a second pass over shared memory
  if (row_terms) {
    if (threadIdx.x < G) group_scale(threadIdx.x, sh.gamma[threadIdx.x], sh.eta[threadIdx.x]);
    __syncthreads();
  }
  float gamma_mine, eta_mine;
  group_scale(my_group, gamma_mine, eta_mine);
  const float lane_scale = beta_mine * gamma_mine * kInvQb;           // inactive lanes: group 0, sums 0

  // ---- this lane's 128 codes -------------------------------------------------------------------------
  uint32_t xr[32];
  int lane_csum = 0;                                    // several groups: the lane's own share of sum x~
  if (active) {
    const uint4* src = reinterpret_cast<const uint4*>(codes + slice * kSlice) + lane;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint4 v = src[i * 32];
      xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
    }
    if (G > 1) {
      int cs[4] = {0, 0, 0, 0};
#pragma unroll
      for (int i = 0; i < 32; ++i) cs[i & 3] = __dp4a((int)xr[i], 0x01010101, cs[i & 3]);
      lane_csum = (cs[0] + cs[1]) + (cs[2] + cs[3]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) xr[i] = 0;
  }
  const int total_csum = sh.csum[0];                    // one group: sum x~ over the whole token
  BL_STAMP(7);

  // ---- the rows of this CTA, stage by stage ------------------------------------------------------------
  TY* y = reinterpret_cast<TY*>(a.y);
  const bool refill = nstages > depth;
  bool from_global = false;                             // sticky: a wait of this warp ran out
  const uint8_t* wlane_g = wslice + (int64_t)chunk * 16;
  for (int st = 0; st < nstages; ++st) {
    const int slot = st % depth;
    if (!from_global) {
      if (*reinterpret_cast<volatile int*>(&sh.abandon)) from_global = true;
      else if (geo.wait_polls == 0 || !bar_wait(smem_u32(&sh.full[slot]), (uint32_t)(st / depth) & 1u, geo.wait_polls)) {
        from_global = true;
        if (lane == 0) { atomicExch(&sh.abandon, 1); __threadfence_block(); atomicAdd(&g_fallbacks, 1u); }
      }
    }
    if (st == 0) BL_STAMP(8);
    const int row0 = st * stage_rows + rowslot * rpw;   // first row of this warp in the stage (CTA-local)
    const unsigned char* wlane_s = ring + (size_t)slot * geo.stage_stride + (size_t)(rowslot * rpw) * Kb + (size_t)chunk * 16;
    float (&part)[kGemvWarps][8] = sh.partial[st & 1];
    // rows past the end read as all-zero bits
    auto load_w = [&](int r) -> uint4 {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (active && r < rpw && row0 + r < rows_cta)
        v = from_global ? __ldcs(reinterpret_cast<const uint4*>(wlane_g + (int64_t)(row0 + r) * Kb))
                        : *reinterpret_cast<const uint4*>(wlane_s + (size_t)r * Kb);
      return v;
    };
    // Row r of the warp summed over its lanes, then Eq. 7 and 11 (one group: (2 S - sum x~) beta gamma / Q_b)
    // straight to y, or the warp's share for the second pass (one group: kept as an integer, so that the
    // slices add up exactly; sum x~ comes off there).  r = -1: nothing to write.
    auto finish = [&](int r, int vi, float vf) {
      if (G == 1) {
        vi = __reduce_add_sync(0xFFFFFFFFu, vi);
        vf = (float)(vi - total_csum) * lane_scale;
        if (row_terms) vf = __int_as_float(vi);
      } else {
        vf = warp_sum(vf);
      }
      if (lane == 0 && r >= 0 && warp_on) {
        if (row_terms) part[warp][r] = vf;
        else if (row0 + r < rows_cta) y[row_begin + row0 + r] = out_cast<TY>(vf);
      }
    };
    // One row per iteration, not unrolled (the body stays in the instruction cache); the sum across
    // the lanes of row r - 1 is taken while row r is multiplied.
    uint4 wcur = load_w(0);
    int pend_i = 0;
    float pend_f = 0.f;
#pragma unroll 1
    for (int r = 0; r < rpw; ++r) {
      const uint4 wnext = load_w(r + 1);
      const int twice_s = active ? (chunk_dot128(wcur, xr) >> 6) : 0;           // 2 S of this lane's chunk
      finish(r - 1, pend_i, pend_f);
      pend_i = twice_s;
      if (G > 1) pend_f = (float)(twice_s - lane_csum) * lane_scale;
      wcur = wnext;
    }
    finish(rpw - 1, pend_i, pend_f);
    if (st == 0) BL_STAMP(9);
    if (refill) {
      // the warp that finishes a stage last starts the copy of the stage that reuses its slot
      __syncwarp();
      if (lane == 0) {
        const int c = atomicAdd(&sh.done[slot], 1);
        if (c == kGemvWarps - 1) {
          atomicExch(&sh.done[slot], 0);
          if (st + depth < nstages && !*reinterpret_cast<volatile int*>(&sh.abandon)) issue_stage(st + depth);
        }
      }
    }
    if (row_terms) {
      __syncthreads();
      // fold the K slices of each row, add the row terms and write y (one thread per row of the stage)
      if (threadIdx.x < rowslots * 8) {
        const int rs = threadIdx.x >> 3, r = threadIdx.x & 7;
        const int row = st * stage_rows + rs * rpw + r;
        if (r < rpw && row < rows_cta) {
          const int64_t n = row_begin + row;
          float v = 0.f;
          if (G == 1) {
            int t = -total_csum;                                       // Eq. 7: 2 S - sum x~
            for (int s = 0; s < nslices; ++s) t += __float_as_int(part[rs * nslices + s][r]);
            v = (float)t * (a.beta[0] * sh.gamma[0] * kInvQb);
          } else {
            for (int s = 0; s < nslices; ++s) v += part[rs * nslices + s][r];
          }
          if (a.eta_correction) {
            for (int g = 0; g < G; ++g) v += sh.eta[g] * a.beta[g] * (float)a.rowsum[n * G + g];
          }
          y[n] = out_cast<TY>(v);
        }
      }
    }
  }

  BL_STAMP(10);
  // ---- a wait ran out somewhere: let the copies that are still in flight finish before the exit -------
  __syncthreads();
  BL_STAMP(11);
  BL_STAMP_NS(2);
  if (threadIdx.x == 0 && blockIdx.x == 0 && a.clear_status != nullptr) *a.clear_status = 0u;
  if (threadIdx.x == 0 && sh.abandon) {
    const unsigned long long t0 = global_ns();
    for (int slot = 0; slot < depth; ++slot) {
      if (sh.issued[slot] == 0) continue;
      const uint32_t bar = smem_u32(&sh.full[slot]);
      const uint32_t parity = (uint32_t)(sh.issued[slot] - 1) & 1u;
      while (!bar_wait(bar, parity, 1024u) && global_ns() - t0 < kDrainNs) {}
    }
  }
}


// ====================================================================================================
// The common case: one group, Eq. 11 as printed (no row terms).  K is taken in slices of 4096; the
// last one may be partial.
//
// Measured on this kernel family: every instruction of a call runs only a handful of times, two
// warps per scheduler hide little, and a conditional branch inside the row loop costs more than the
// arithmetic it guards.  So here a warp owns whole rows (all slices of K), the row loop has no
// branch but its own, no predicate and no reduction across lanes: a lane's partial sum goes to a
// warp-private array in shared memory, and once per stage the warp adds the 32 partial sums of each
// of its rows (four lanes per row, eight loads each, two shuffles).  Rows past the end of the CTA's
// slice are multiplied like the others (on whatever bytes the ring slot holds) and dropped at the
// store.  The LN sums are taken around a pilot value (the mean of the first eight features) in fp32.
struct FastGeom {            // decided on the host
  int rows_per_cta, rpw, nstages, nslices, depth;
  uint32_t stage_stride;     // bytes between ring slots (a multiple of 128)
  uint32_t ring_bytes;       // depth * stage_stride
  uint32_t wait_polls;
  int x_in_smem;             // more than one slice and not kept in registers: raw x as fp32 in shared memory
  float inv_k;
  double inv_k_d;
};

constexpr int kAccStride = 33;                           // words per row of partial sums (bank spread)
constexpr int kAccWarpWords = kBatchRows * kAccStride;   // per warp

struct FastShared {
  WarpStats red[kGemvWarps];
  unsigned long long full[kMaxStages];
  int done[kMaxStages];
  int issued[kMaxStages];
  int abandon;
  int csum;
  int acc[kGemvWarps][kAccWarpWords];
};

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// The rows of one warp in one stage, slice s of K: lane partial sums to (or onto) the warp's array.
// kFirst: first slice (store), else add to what is there.  kGlobal: weights straight from global
// memory (the stage's copy did not arrive in time); rows past the end then re-read the last row.
template <bool kFirst, bool kGlobal>
__device__ __forceinline__ void warp_rows(const uint32_t (&xr)[32], int rpw, uint32_t wsm, const uint8_t* wgl,
                                          int64_t Kb, int rows_left, int* acc_lane) {
  uint4 wcur;
  if (kGlobal) wcur = __ldcs(reinterpret_cast<const uint4*>(wgl));
  else wcur = lds128(wsm);
#pragma unroll 1
  for (int r = 0; r < rpw; ++r) {
    uint4 wnext;
    if (kGlobal) {
      const int rn = min(r + 1, rows_left - 1);
      wnext = __ldcs(reinterpret_cast<const uint4*>(wgl + (int64_t)rn * Kb));
    } else {
      wnext = lds128(wsm + (uint32_t)(r + 1) * (uint32_t)Kb);      // one row past the warp's last: still inside the ring
    }
    int p = chunk_dot128(wcur, xr) >> 6;                           // 2 S of this lane's chunk
    if (!kFirst) p += acc_lane[r * kAccStride];
    acc_lane[r * kAccStride] = p;
    wcur = wnext;
  }
}

// Eight 16-bit inputs (one 16-byte load) as floats.
template <typename T> __device__ __forceinline__ void unpack8(const uint4& r, float (&v)[8]);
template <> __device__ __forceinline__ void unpack8<__half>(const uint4& r, float (&v)[8]) {
  const __half2* h = reinterpret_cast<const __half2*>(&r);
#pragma unroll
  for (int i = 0; i < 4; ++i) { const float2 f = __half22float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
}
template <> __device__ __forceinline__ void unpack8<__nv_bfloat16>(const uint4& r, float (&v)[8]) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}
template <> __device__ __forceinline__ void unpack8<float>(const uint4&, float (&)[8]) {}   // never called

constexpr int kRawSlices = 4;            // most slices of a 16-bit token that a thread keeps in registers (32 of them)

// kSingle: K <= 4096 (one slice).  The thread's 16 features then stay in registers between the two passes, no
// raw copy of x is kept in shared memory, and three CTAs fit on an SM (the call in progress and two
// calls staging their weights behind it, or three independent calls).
// kPartial: K does not fill its last slice; only then does the code test features for presence.
template <typename TX, typename TY, bool kSingle, bool kPartial>
__global__ void __launch_bounds__(kGemvThreads, kSingle ? 3 : 2)
gemv_decode_fast_kernel(GemvArgs a, FastGeom geo) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ FastShared sh;
  unsigned char* ring = smem_raw;                                                  // [depth][stage_stride] (+ one row)
  const int K = (int)a.K, Kp = geo.nslices * kSlice;                               // K rounded up to whole slices
  const uint32_t ring_alloc = geo.ring_bytes + (uint32_t)(a.K / 8) + 512u;         // lanes of a partial slice read past a row's end
  float* xf = reinterpret_cast<float*>(smem_raw + ring_alloc);                     // [Kp] raw x (not for kSingle)
  int8_t* codes = reinterpret_cast<int8_t*>(smem_raw + ring_alloc + (geo.x_in_smem ? (size_t)Kp * sizeof(float) : 0));   // [Kp]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t Kb = a.K / 8;
  const int rpw = geo.rpw, nslices = geo.nslices, depth = geo.depth;
  const int stage_rows = rpw * kGemvWarps;
  const int64_t row_begin = (int64_t)blockIdx.x * geo.rows_per_cta;
  const int64_t row_end = min((int64_t)a.N, row_begin + geo.rows_per_cta);
  const int rows_cta = (int)(row_end - row_begin);
  // stages that hold rows of this CTA (the last CTA has fewer rows than the others): a stage without
  // rows gets no copy, so nobody may wait for one
  const int nstages = min(geo.nstages, (rows_cta + stage_rows - 1) / stage_rows);
  const uint8_t* wslice = a.W_packed + row_begin * Kb;

  auto issue_stage = [&](int st, int slot) {
    const int rows = min(stage_rows, rows_cta - st * stage_rows);
    if (rows <= 0) return;
    const uint32_t bytes = (uint32_t)rows * (uint32_t)Kb;                          // a multiple of 512
    const uint32_t bar = smem_u32(&sh.full[slot]);
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");                   // earlier reads of the slot come first
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(ring + (size_t)slot * geo.stage_stride)), "l"(wslice + (int64_t)st * stage_rows * Kb),
          "r"(bytes), "r"(bar), "l"(policy) : "memory");
    sh.issued[slot] += 1;
  };

  BL_STAMP_DECL
  BL_STAMP_NS(0);
  BL_STAMP(0);
  // ---- ahead of stream order: this CTA's weights on their way into shared memory --------------------
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&sh.full[i])));
      sh.done[i] = 0;
      sh.issued[i] = 0;
    }
    sh.abandon = 0;
    sh.csum = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int st = 0; st < depth && st < nstages; ++st) issue_stage(st, st);
  }
  if (blockIdx.x < 4) {
    const char* xb = reinterpret_cast<const char*>(a.x);
    for (int64_t off = (int64_t)threadIdx.x * 128; off < a.K * (int64_t)sizeof(TX); off += (int64_t)kGemvThreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(xb + off));
  }
  BL_STAMP(1);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  asm volatile("griddepcontrol.wait;" ::: "memory");
  BL_STAMP_NS(1);
  BL_STAMP(2);

  // ---- x: 16 features per thread and slice, sums around the pilot, raw values to shared memory -------
  const TX* x = reinterpret_cast<const TX*>(a.x);
  const float beta = __ldg(a.beta);
  float pilot;
  {
    float h[8];
    Elem<TX>::load8(x, h);
    pilot = (((h[0] + h[1]) + (h[2] + h[3])) + ((h[4] + h[5]) + (h[6] + h[7]))) * 0.125f;
  }
  const bool ln = a.ln_eps >= 0.f;
  if (!ln) pilot = 0.f;
  float s1 = 0.f, s2 = 0.f, mn = INFINITY, mx = -INFINITY;
  float xv[16];                                         // kSingle: this thread's features
  // Features past K (K need not fill its last slice of 4096) are absent: they add nothing to the
  // sums, are read as copies of real features for the extremes, get code 0, and the lanes that own them multiply zeros.
  // sums of 16 raw features around the pilot, and their extremes
  auto moments16 = [&](int i, const float (&v)[16]) {
    const int k = i * kSlice + threadIdx.x * 8;
    const bool have[2] = {!kPartial || k < K, !kPartial || k + kSlice / 2 < K};
    float d[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) { d[j] = have[j >> 3] ? v[j] - pilot : 0.f; mn = fminf(mn, v[j]); mx = fmaxf(mx, v[j]); }
    s1 += (((d[0] + d[1]) + (d[2] + d[3])) + ((d[4] + d[5]) + (d[6] + d[7]))) +
          (((d[8] + d[9]) + (d[10] + d[11])) + ((d[12] + d[13]) + (d[14] + d[15])));
    float p2 = 0.f, q2 = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) { p2 = fmaf(d[j], d[j], p2); q2 = fmaf(d[8 + j], d[8 + j], q2); }
    s2 += p2 + q2;
  };
  // features k..k+7 and k+2048..k+2055 of slice i
  auto load16 = [&](int i, float (&v)[16]) {
    const int k = i * kSlice + threadIdx.x * 8;
    float lo8[8], hi8[8];
    // (absent features: the last eight real ones once more, which leaves the extremes alone)
    Elem<TX>::load8(x + (kPartial ? min(k, K - 8) : k), lo8);
    Elem<TX>::load8(x + (kPartial ? min(k + kSlice / 2, K - 8) : k + kSlice / 2), hi8);
#pragma unroll
    for (int j = 0; j < 8; ++j) { v[j] = lo8[j]; v[8 + j] = hi8[j]; }
  };
  // A 16-bit token of up to kRawSlices slices stays in registers as loaded (all loads issued at once,
  // converted once for the sums and once more for the codes); longer or fp32 tokens go through shared
  // memory as fp32, one slice at a time.
  constexpr bool kRaw16 = !kSingle && sizeof(TX) == 2;
  uint4 raw[kRaw16 ? kRawSlices : 1][2];
  const bool in_regs = kRaw16 && !geo.x_in_smem;
  auto from_raw = [&](int i, float (&v)[16]) {
    float lo8[8], hi8[8];
    unpack8<TX>(raw[kRaw16 ? i : 0][0], lo8);
    unpack8<TX>(raw[kRaw16 ? i : 0][1], hi8);
#pragma unroll
    for (int j = 0; j < 8; ++j) { v[j] = lo8[j]; v[8 + j] = hi8[j]; }
  };
  if (kSingle) {
    load16(0, xv);
    moments16(0, xv);
  } else if (in_regs) {
#pragma unroll
    for (int i = 0; i < kRawSlices; ++i) {
      if (i < nslices) {
        const int k = i * kSlice + threadIdx.x * 8;
        raw[kRaw16 ? i : 0][0] = __ldg(reinterpret_cast<const uint4*>(x + (kPartial ? min(k, K - 8) : k)));
        raw[kRaw16 ? i : 0][1] = __ldg(reinterpret_cast<const uint4*>(x + (kPartial ? min(k + kSlice / 2, K - 8) : k + kSlice / 2)));
      }
    }
#pragma unroll
    for (int i = 0; i < kRawSlices; ++i) {
      if (i < nslices) {
        float v[16];
        from_raw(i, v);
        moments16(i, v);
      }
    }
  } else {
#pragma unroll 1
    for (int i = 0; i < nslices; ++i) {
      const int k = i * kSlice + threadIdx.x * 8;
      float v[16];
      load16(i, v);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        *reinterpret_cast<float4*>(xf + k + h * (kSlice / 2)) = make_float4(v[8 * h], v[8 * h + 1], v[8 * h + 2], v[8 * h + 3]);
        *reinterpret_cast<float4*>(xf + k + h * (kSlice / 2) + 4) = make_float4(v[8 * h + 4], v[8 * h + 5], v[8 * h + 6], v[8 * h + 7]);
      }
      moments16(i, v);
    }
  }
  BL_STAMP(3);
  s1 = warp_sum(s1); s2 = warp_sum(s2); mn = warp_min(mn); mx = warp_max(mx);
  if (lane == 0) sh.red[warp] = WarpStats{s1, s2, mn, mx};
  __syncthreads();
  BL_STAMP(4);

  // ---- code map from the eight warp totals (every thread the same arithmetic) ----------------------
  float t1, t2, xlo, xhi;
  {
    float4 w8[kGemvWarps];
#pragma unroll
    for (int w = 0; w < kGemvWarps; ++w) w8[w] = *reinterpret_cast<const float4*>(&sh.red[w]);
    t1 = ((w8[0].x + w8[1].x) + (w8[2].x + w8[3].x)) + ((w8[4].x + w8[5].x) + (w8[6].x + w8[7].x));
    t2 = ((w8[0].y + w8[1].y) + (w8[2].y + w8[3].y)) + ((w8[4].y + w8[5].y) + (w8[6].y + w8[7].y));
    xlo = fminf(fminf(fminf(w8[0].z, w8[1].z), fminf(w8[2].z, w8[3].z)), fminf(fminf(w8[4].z, w8[5].z), fminf(w8[6].z, w8[7].z)));
    xhi = fmaxf(fmaxf(fmaxf(w8[0].w, w8[1].w), fmaxf(w8[2].w, w8[3].w)), fmaxf(fmaxf(w8[4].w, w8[5].w), fmaxf(w8[6].w, w8[7].w)));
  }
  const float off = ln ? t1 * geo.inv_k : 0.f;          // mean - pilot
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
  BL_STAMP(5);

  // ---- codes of this thread's features -----------------------------------------------------------------
  int csum = 0;
  // Eq. 4 / 6 for 16 features of slice i (k..k+7, k+2048..k+2055), codes to their slots
  auto quant16 = [&](int i, const float (&v)[16]) {
    const int k = i * kSlice + threadIdx.x * 8;
    uint32_t tb[16];
    bool near_tie = false;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float f = fminf(fmaxf(fmaf(v[j], Af, Bf), lo_f), (float)kCodeMax);   // the clip of Eq. 4 / 6 commutes with rne
      const float t = f + kRoundMagic;                                 // rne(f) in the low mantissa bits
      tb[j] = __float_as_uint(t);
      near_tie |= fabsf(f - (t - kRoundMagic)) > near;
    }
    if (near_tie && span_f > 0.f) {                                    // rare: settle the close ones exactly
      const double mean = (double)pilot + (ln ? (double)t1 * geo.inv_k_d : 0.0);
      const double c = (a.mode == BL_ABSMAX) ? mean : (double)xlo;
      const double span = (a.mode == BL_ABSMAX) ? fmax(fabs((double)xlo - mean), fabs((double)xhi - mean))
                                                : (double)xhi - (double)xlo;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float f = fmaf(v[j], Af, Bf);                            // unclipped: a clipped one is never close
        if (f > lo_f && f < (float)kCodeMax && fabsf(f - rintf(f)) > near)
          tb[j] = (uint32_t)max((int)lo_f, min(kCodeMax, exact_code(v[j], f, c, span)));
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t w0 = __byte_perm(__byte_perm(tb[8 * h], tb[8 * h + 1], 0x0040), __byte_perm(tb[8 * h + 2], tb[8 * h + 3], 0x0040), 0x5410);
      uint32_t w1 = __byte_perm(__byte_perm(tb[8 * h + 4], tb[8 * h + 5], 0x0040), __byte_perm(tb[8 * h + 6], tb[8 * h + 7], 0x0040), 0x5410);
      if (kPartial && k + h * (kSlice / 2) >= K) { w0 = 0u; w1 = 0u; }              // absent features
      *reinterpret_cast<uint2*>(codes + code_slot(k + h * (kSlice / 2))) = make_uint2(w0, w1);
      csum = __dp4a((int)w0, 0x01010101, csum);
      csum = __dp4a((int)w1, 0x01010101, csum);
    }
  };
  if (kSingle) {
    quant16(0, xv);
  } else if (in_regs) {
#pragma unroll
    for (int i = 0; i < kRawSlices; ++i) {
      if (i < nslices) {
        float v[16];
        from_raw(i, v);
        quant16(i, v);
      }
    }
  } else {
#pragma unroll 1
    for (int i = 0; i < nslices; ++i) {
      const int k = i * kSlice + threadIdx.x * 8;
      float v[16];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float4 p = *reinterpret_cast<const float4*>(xf + k + h * (kSlice / 2));
        const float4 q = *reinterpret_cast<const float4*>(xf + k + h * (kSlice / 2) + 4);
        v[8 * h] = p.x; v[8 * h + 1] = p.y; v[8 * h + 2] = p.z; v[8 * h + 3] = p.w;
        v[8 * h + 4] = q.x; v[8 * h + 5] = q.y; v[8 * h + 6] = q.z; v[8 * h + 7] = q.w;
      }
      quant16(i, v);
    }
  }
  csum = __reduce_add_sync(0xFFFFFFFFu, csum);
  if (lane == 0) atomicAdd(&sh.csum, csum);
  BL_STAMP(6);
  __syncthreads();                                     // codes and their sum visible
  BL_STAMP(7);

  // ---- the rows of this CTA, stage by stage ------------------------------------------------------------
  TY* y = reinterpret_cast<TY*>(a.y);
  const int total_csum = sh.csum;
  const bool refill = nstages > depth;
  bool from_global = false;                             // sticky: a wait of this warp ran out
  int* acc_lane = &sh.acc[warp][lane];
  const int* acc_row = &sh.acc[warp][(lane >> 2) * kAccStride + (lane & 3) * 8];
  uint32_t xr[32];
  const uint4* code_src = reinterpret_cast<const uint4*>(codes) + lane;
  auto load_codes = [&](int s) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint4 v = code_src[s * (kSlice / 16) + i * 32];
      xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
    }
  };
  // gamma of Eq. 5 / 6 on x^ = (x - mean) rstd: only the final rescale reads it
  float rstd = 1.f;
  if (ln) {
    const float var_f = fmaxf(fmaf(-off, off, t2 * geo.inv_k), 0.f);
    const float vv = var_f + a.ln_eps;
    if (vv > 1e-30f && vv < 1e30f) {
      const float y = rsqrtf(vv);
      rstd = y * (1.5f - 0.5f * vv * y * y);
    } else {
      rstd = rstd_outside_fp32(vv);
    }
  }
  const float scale = beta * (span_f * rstd) * kInvQb;
  load_codes(0);
  const uint32_t warp_off = (uint32_t)(warp * rpw) * (uint32_t)Kb + lane * 16;
  BL_STAMP(8);
  int slot = 0;                                         // st % depth and the parity of st / depth, kept by hand:
  uint32_t phase = 0u;                                  // a division costs more here than a row
  uint32_t slot_addr = smem_u32(ring);
  for (int st = 0; st < nstages; ++st) {
    if (!from_global) {
      if (*reinterpret_cast<volatile int*>(&sh.abandon)) from_global = true;
      else if (geo.wait_polls == 0 || !bar_wait(smem_u32(&sh.full[slot]), phase, geo.wait_polls)) {
        from_global = true;
        if (lane == 0) { atomicExch(&sh.abandon, 1); __threadfence_block(); atomicAdd(&g_fallbacks, 1u); }
      }
    }
    if (st == 0) BL_STAMP(9);
    const int row0 = st * stage_rows + warp * rpw;      // first row of this warp in the stage (CTA-local)
    const int rows_left = rows_cta - row0;              // may be <= 0: nothing of this warp is stored
    const uint32_t wsm = slot_addr + warp_off;
    const uint8_t* wgl = wslice + (int64_t)min(row0, rows_cta - 1) * Kb;               // only read after a failed wait
    const int rl = max(rows_left, 1);
    if (kSingle) {
      if (!from_global) warp_rows<true, false>(xr, rpw, wsm, wgl, Kb, rl, acc_lane);
      else warp_rows<true, true>(xr, rpw, wsm, wgl + min((int64_t)lane * 16, Kb - 16), Kb, rl, acc_lane);
    } else {
#pragma unroll 1
      for (int s = 0; s < nslices; ++s) {
        if (s > 0 || st > 0) load_codes(s);
        if (!from_global) {
          if (s == 0) warp_rows<true, false>(xr, rpw, wsm, wgl, Kb, rl, acc_lane);
          else warp_rows<false, false>(xr, rpw, wsm + s * 512, wgl, Kb, rl, acc_lane);
        } else {
          // (a lane whose chunk lies past K multiplies zero codes: any bytes of the row will do)
          const uint8_t* wl = wgl + min((int64_t)s * 512 + lane * 16, Kb - 16);
          if (s == 0) warp_rows<true, true>(xr, rpw, wsm, wl, Kb, rl, acc_lane);
          else warp_rows<false, true>(xr, rpw, wsm, wl, Kb, rl, acc_lane);
        }
      }
    }
    if (st == 0) BL_STAMP(10);
    // the 32 partial sums of each row: four lanes per row, eight each
    __syncwarp();
    {
      int t = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) t += acc_row[i];
      t += __shfl_xor_sync(0xFFFFFFFFu, t, 1);
      t += __shfl_xor_sync(0xFFFFFFFFu, t, 2);
      const int r = lane >> 2;
      // Eq. 7 and 11: (2 S - sum x~) beta gamma / Q_b
      if ((lane & 3) == 0 && r < rpw && r < rows_left) y[row_begin + row0 + r] = out_cast<TY>((float)(t - total_csum) * scale);
    }
    __syncwarp();
    if (st == 0) BL_STAMP(11);
    if (refill) {
      // the warp that finishes a stage last starts the copy of the stage that reuses its slot
      if (lane == 0) {
        const int c = atomicAdd(&sh.done[slot], 1);
        if (c == kGemvWarps - 1) {
          atomicExch(&sh.done[slot], 0);
          if (st + depth < nstages && !*reinterpret_cast<volatile int*>(&sh.abandon)) issue_stage(st + depth, slot);
        }
      }
    }
    if (++slot == depth) { slot = 0; slot_addr = smem_u32(ring); phase ^= 1u; }
    else slot_addr += geo.stage_stride;
  }
  BL_STAMP(12);

  // ---- a wait ran out somewhere: let the copies that are still in flight finish before the exit -------
  __syncthreads();
  BL_STAMP(13);
  BL_STAMP_NS(2);
  if (threadIdx.x == 0 && blockIdx.x == 0 && a.clear_status != nullptr) *a.clear_status = 0u;
  if (threadIdx.x == 0 && sh.abandon) {
    const unsigned long long t0 = global_ns();
    for (int slot = 0; slot < depth; ++slot) {
      if (sh.issued[slot] == 0) continue;
      const uint32_t bar = smem_u32(&sh.full[slot]);
      const uint32_t parity = (uint32_t)(sh.issued[slot] - 1) & 1u;
      while (!bar_wait(bar, parity, 1024u) && global_ns() - t0 < kDrainNs) {}
    }
  }
}

template <typename TX, typename TY>
cudaError_t run_fast(const GemvArgs& a, cudaStream_t s, int dev, int sms) {
  FastGeom geo;
  const int64_t Kb = a.K / 8;
  geo.nslices = (int)((a.K + kSlice - 1) / kSlice);
  const int64_t rows_per_cta = (a.N + sms - 1) / sms;
  const int64_t per_warp = (rows_per_cta + kGemvWarps - 1) / kGemvWarps;
  int64_t rmax = std::max<int64_t>(1, std::min<int64_t>(kBatchRows, 32768 / (kGemvWarps * Kb)));
  // long rows: when the CTA's whole slice fits the ring as one stage, take it as one (a warp then loads
  // the codes of a K slice once for all of its rows instead of once per stage)
  if (per_warp > rmax && per_warp <= kBatchRows && per_warp * kGemvWarps * Kb <= (int64_t)kRingBytes) rmax = per_warp;
  const int64_t nstages = (per_warp + rmax - 1) / rmax;
  if (nstages > 0x3FFFFFFF) return cudaErrorInvalidValue;
  geo.rows_per_cta = (int)rows_per_cta;
  geo.nstages = (int)nstages;
  geo.rpw = (int)((per_warp + nstages - 1) / nstages);
  geo.stage_stride = (uint32_t)(geo.rpw * kGemvWarps * Kb);                      // a multiple of 4096, at most 32 KB
  const bool single = geo.nslices == 1;
  const size_t Kp = (size_t)geo.nslices * kSlice;
  geo.x_in_smem = (!single && (sizeof(TX) != 2 || geo.nslices > kRawSlices)) ? 1 : 0;
  const size_t fixed = Kp * (geo.x_in_smem ? sizeof(float) + 1 : 1) + (size_t)Kb + 512;   // (raw x,) codes, slack beyond the ring
  const size_t budget = std::min<size_t>(kRingBytes, 210 * 1024 - fixed);
  const int depth = std::max(1, std::min((int)(budget / geo.stage_stride), kMaxStages));
  geo.depth = (int)std::min<int64_t>(depth, nstages);
  geo.ring_bytes = (uint32_t)geo.depth * geo.stage_stride;
  const long long polls = g_debug_wait_polls.load(std::memory_order_relaxed);
  geo.wait_polls = polls < 0 ? kStagePolls : (uint32_t)std::min<long long>(polls, kStagePolls);
  geo.inv_k_d = 1.0 / (double)a.K;
  geo.inv_k = (float)geo.inv_k_d;
  const unsigned grid = (unsigned)((a.N + rows_per_cta - 1) / rows_per_cta);
  const size_t smem = (size_t)geo.ring_bytes + fixed;
  static std::atomic<int> configured[64];
  cudaError_t e;
  const bool partial = a.K % kSlice != 0;
  auto kern = single ? (partial ? gemv_decode_fast_kernel<TX, TY, true, true> : gemv_decode_fast_kernel<TX, TY, true, false>)
                     : (partial ? gemv_decode_fast_kernel<TX, TY, false, true> : gemv_decode_fast_kernel<TX, TY, false, false>);
  if (dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    for (auto k : {gemv_decode_fast_kernel<TX, TY, true, true>, gemv_decode_fast_kernel<TX, TY, true, false>,
                   gemv_decode_fast_kernel<TX, TY, false, true>, gemv_decode_fast_kernel<TX, TY, false, false>}) {
      e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024);
      if (e != cudaSuccess) return e;
      e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
    }
    if (dev < 64) configured[dev].store(1, std::memory_order_release);
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
  return cudaLaunchKernelEx(&cfg, kern, a, geo);
}

template <typename TX, typename TY>
cudaError_t run2(const GemvArgs& a, cudaStream_t s) {
  int dev = 0, sms = 148;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  if (a.G == 1 && !a.eta_correction) return run_fast<TX, TY>(a, s, dev, sms);
  // One CTA per SM when there are enough rows; every row slot takes its rows in stages of at most
  // kBatchRows, all stages the same height.
  GemvGeom geo;
  const int64_t Kb = a.K / 8;
  geo.nslices = (int)((a.K + kSlice - 1) / kSlice);
  geo.rowslots = kGemvWarps / geo.nslices;
  const int64_t rows_per_cta = (a.N + sms - 1) / sms;
  const int64_t per_slot = (rows_per_cta + geo.rowslots - 1) / geo.rowslots;
  const int64_t nstages = (per_slot + kBatchRows - 1) / kBatchRows;
  if (nstages > 0x3FFFFFFF) return cudaErrorInvalidValue;
  geo.rows_per_cta = (int)rows_per_cta;
  geo.nstages = (int)nstages;
  geo.rpw = (int)((per_slot + nstages - 1) / nstages);
  const uint32_t stage_bytes = (uint32_t)(geo.rpw * geo.rowslots * Kb);          // at most 32 KB
  geo.stage_stride = (stage_bytes + 127u) & ~127u;
  const size_t fixed = (size_t)a.K * sizeof(float) + (size_t)geo.nslices * kSlice;
  const size_t budget = std::min<size_t>(kRingBytes, 216 * 1024 - fixed);
  int depth = (int)(budget / geo.stage_stride);
  depth = std::max(1, std::min(depth, kMaxStages));
  geo.depth = (int)std::min<int64_t>(depth, nstages);
  geo.ring_bytes = (uint32_t)geo.depth * geo.stage_stride;
  const long long polls = g_debug_wait_polls.load(std::memory_order_relaxed);
  geo.wait_polls = polls < 0 ? kStagePolls : (uint32_t)std::min<long long>(polls, kStagePolls);
  geo.inv_kg = 1.0 / (double)(a.K / a.G);
  geo.inv_nslices = (65536u + geo.nslices - 1) / geo.nslices;
  const uint32_t group_chunks = a.G > 1 ? (uint32_t)(a.K / a.G / 128) : 256u;   // G > 1 needs K_g % 128 == 0
  geo.inv_group_chunks = (65536u + group_chunks - 1) / group_chunks;
  const unsigned grid = (unsigned)((a.N + rows_per_cta - 1) / rows_per_cta);
  const size_t smem = (size_t)geo.ring_bytes + fixed;
  // per device: the opt-in shared-memory size, and a carve-out that lets two CTAs share an SM so
  // that the call behind this one can stage its weights while this one computes
  static std::atomic<int> configured[64];
  if (dev >= 64 || configured[dev].load(std::memory_order_acquire) < (int)smem) {
    e = cudaFuncSetAttribute(gemv_decode_kernel<TX, TY>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemv_decode_kernel<TX, TY>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    if (dev < 64) configured[dev].store(216 * 1024, std::memory_order_release);
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

// Reads and clears the count of warps that gave up waiting for a weight stage and read it from
// global memory instead.
cudaError_t gemv_decode_take_fallbacks(unsigned int* out) {
  cudaError_t e = cudaMemcpyFromSymbol(out, g_fallbacks, sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  if (*out) {
    const unsigned int zero = 0;
    e = cudaMemcpyToSymbol(g_fallbacks, &zero, sizeof(zero));
  }
  return e;
}

cudaError_t launch_gemv_decode(const GemvArgs& a, cudaStream_t s) {
  switch (a.xt) {
    case BL_F32: return run1<float>(a, s);
    case BL_F16: return run1<__half>(a, s);
    case BL_BF16: return run1<__nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl

#ifdef BL_GEMV_STAMPS
// Copies the stamp rings to the host: out must hold 2 * 64 records of (3 + 32) 64-bit words.
extern "C" int bitlinear_debug_gemv_stamps(unsigned long long* out, unsigned int* launches) {
  if (cudaDeviceSynchronize() != cudaSuccess) return 1;
  if (cudaMemcpyFromSymbol(out, bl::g_stamps, sizeof(bl::g_stamps)) != cudaSuccess) return 1;
  return cudaMemcpyFromSymbol(launches, bl::g_stamp_launch, sizeof(bl::g_stamp_launch)) != cudaSuccess;
}
#endif
