// Steps 1-2 of BitLinear: LN per token and group (Eq. 12, 15) fused with the 8-bit activation
// quantisation (Eq. 4-6, 14).  HBM-bound: x is read once (per token) or twice (per tensor) with
// 128-bit loads; the normalised row is never written to HBM.
//
// Two implementations.  Segments of up to 16 KB (8192 16-bit, 4096 fp32 features) that are a
// multiple of 256 features take the fast path in the second half of this file: one warp per
// segment, staged in shared memory.  Other segments take one CTA per (token m, group g) segment,
// staged in shared memory as fp32:
//   moments  sum, raw min/max, then sum of squared deviations      (quant_core.cuh)
//   codes    one FMA + round per element, 8 codes per 8-byte store
// Per-tensor scope splits in two kernels: the first leaves each segment's moments in the
// workspace and folds the extremes of x^ into a global atomic min/max on an order-preserving
// encoding (order-independent, hence deterministic); the second re-reads x and writes codes.
#include <algorithm>
#include <atomic>
#include <mutex>
#include <random>
#include <type_traits>

#include "quant_rows.cuh"

namespace bl {

namespace {

using namespace rows;

constexpr int kQuantThreads = 256;

struct SegRecord {                 // per-segment record kept between the two per-tensor kernels
  double mean, rstd;
  float xlo, xhi;                  // raw extremes of the segment
};

struct TensorScope {               // running extremes of x^ per group (long-segment kernels, atomics)
  unsigned long long enc_min[BL_MAX_GROUPS];
  unsigned long long enc_max[BL_MAX_GROUPS];
};
struct ScopePartial {              // one CTA's extremes of x^ for one group (fast path, plain stores)
  unsigned long long lo, hi;
};
constexpr int kMaxStatCtas = 256;  // upper bound on the grid of the persistent fast-path kernels
// Per-tensor workspace:
//   status word (256 bytes reserved) | TensorScope | ScopePartial[kMaxStatCtas][BL_MAX_GROUPS] |
//   arrival tags u64[kMaxStatCtas] | SegRecord[M*G].
constexpr size_t kWsGenOff = 128;     // inside the status block: generation count of the fused kernel's meeting
constexpr size_t kWsScopeOff = 256;
constexpr size_t kWsPartialOff = kWsScopeOff + sizeof(TensorScope);
constexpr size_t kWsTagOff = kWsPartialOff + (size_t)kMaxStatCtas * BL_MAX_GROUPS * sizeof(ScopePartial);
constexpr size_t kWsHeaderBytes = kWsTagOff + (size_t)kMaxStatCtas * sizeof(unsigned long long);

template <typename T>
__device__ __forceinline__ void stage_segment(const T* __restrict__ src, int Kg, float* seg) {
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    float v[8];
    Elem<T>::load8(src + k, v);
    *reinterpret_cast<float4*>(seg + k) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(seg + k + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
  __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
quant_per_token(const T* __restrict__ x, int64_t K, int G, int mode, float ln_eps,
                int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  extern __shared__ __align__(16) float seg[];
  __shared__ QuantRed<kQuantThreads> red;
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t base = m * K + (int64_t)g * Kg;
  stage_segment<T>(x + base, Kg, seg);
  SegMoments mom; float xlo, xhi;
  segment_moments<kQuantThreads>(seg, Kg, ln_eps, red, mom, xlo, xhi);
  const double lo = ((double)xlo - mom.mean) * mom.rstd, hi = ((double)xhi - mom.mean) * mom.rstd;
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const QuantMap map = make_quant_map(mode, mom, gam, et, fmaxf(fabsf(xlo), fabsf(xhi)));
  if (threadIdx.x == 0) {
    gamma[m * G + g] = (float)gam;
    if (eta) eta[m * G + g] = (float)et;
  }
  int8_t* dst = x_q + base;
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    const float4 a = *reinterpret_cast<const float4*>(seg + k);
    const float4 b = *reinterpret_cast<const float4*>(seg + k + 4);
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    *reinterpret_cast<uint2*>(dst + k) = quant_pack8(v, map);
  }
}

__global__ void init_scope(TensorScope* sc, uint32_t* status, int clear_status) {
  const int g = threadIdx.x;
  if (g == 0 && clear_status) *status = 0u;                          // these kernels have no device-side wait
  if (g < BL_MAX_GROUPS) { sc->enc_min[g] = ~0ull; sc->enc_max[g] = 0ull; }
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
tensor_stats(const T* __restrict__ x, int64_t K, int G, float ln_eps, TensorScope* sc,
             SegRecord* __restrict__ recs) {
  extern __shared__ __align__(16) float seg[];
  __shared__ QuantRed<kQuantThreads> red;
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  stage_segment<T>(x + m * K + (int64_t)g * Kg, Kg, seg);
  SegMoments mom; float xlo, xhi;
  segment_moments<kQuantThreads>(seg, Kg, ln_eps, red, mom, xlo, xhi);
  if (threadIdx.x == 0) {
    recs[blockIdx.x] = SegRecord{mom.mean, mom.rstd, xlo, xhi};
    atomicMin(&sc->enc_min[g], enc_ordered64(((double)xlo - mom.mean) * mom.rstd));
    atomicMax(&sc->enc_max[g], enc_ordered64(((double)xhi - mom.mean) * mom.rstd));
  }
}

template <typename T>
__global__ void __launch_bounds__(kQuantThreads)
tensor_codes(const T* __restrict__ x, int64_t K, int G, int mode, const TensorScope* __restrict__ sc,
             const SegRecord* __restrict__ recs, int8_t* __restrict__ x_q,
             float* __restrict__ gamma, float* __restrict__ eta) {
  const int Kg = (int)(K / G);
  const int64_t m = blockIdx.x / G;
  const int g = blockIdx.x % G;
  const int64_t base = m * K + (int64_t)g * Kg;
  const SegRecord rec = recs[blockIdx.x];
  const double lo = dec_ordered64(sc->enc_min[g]), hi = dec_ordered64(sc->enc_max[g]);
  double gam, et;
  scope_gamma_eta(mode, lo, hi, gam, et);
  const QuantMap map = make_quant_map(mode, SegMoments{rec.mean, rec.rstd}, gam, et, fmaxf(fabsf(rec.xlo), fabsf(rec.xhi)));
  if (m == 0 && threadIdx.x == 0) {
    gamma[g] = (float)gam;
    if (eta) eta[g] = (float)et;
  }
  const T* src = x + base;
  int8_t* dst = x_q + base;
  for (int k = threadIdx.x * 8; k < Kg; k += kQuantThreads * 8) {
    float v[8];
    Elem<T>::load8(src + k, v);
    *reinterpret_cast<uint2*>(dst + k) = quant_pack8(v, map);
  }
}


// ================================================================================================
// Fast path: one warp per (token, group) segment, the segment staged in shared memory.
//
// Used when a segment is a whole number of 256-element pieces and at most 16 KB, which covers
// every hidden size of the paper's model table and the FFN width up to the 1.3B model.  The
// kernels are persistent: one CTA per SM; CTA c owns the contiguous segment range
// [c*S/grid, (c+1)*S/grid) and its warps draw segments from it through a shared counter.  Each warp
// has 16 KB of shared memory.  For segments of up to 8 KB these are two slots: while the warp works
// on one, the asynchronous copies (cp.async, 16 bytes per lane and instruction) of its next
// segment land in the other, so every warp keeps a segment's worth of HBM traffic outstanding
// whatever it is computing.  A longer segment takes the whole area; its successor is copied after
// the work on it, and the other warps keep the memory system busy meanwhile.  Waiting is
// cp.async.wait_group: no barrier objects, no spin loops.  A warp walks its segment in chunks of
// 8 elements per lane (a short rolled loop: small code, few registers), with warp shuffles for
// the reductions and no block barrier inside the loop.  Sums are fp32 inside a lane and fp64
// across lanes, in one pass over deviations from a pilot value.  Reciprocals and the inverse
// square root are hardware seeds refined by Newton steps in fp64 (below one ulp of fp64 after two
// steps), which keeps fp64 division and square-root routines out of the kernels.
constexpr int kRowWarps = 14;              // as many as shared memory holds: 14 x 16 KB of staging + 2.3 KB static
constexpr int kSlotBytes = 8192;
constexpr int kRowStage = kRowWarps * 2 * kSlotBytes;
static_assert(kRowStage + 3 * 1024 <= 227 * 1024, "staging plus the kernels' static shared memory must fit one SM");
template <typename T> struct RowTraits {                      // chunk = 8 consecutive elements
  static constexpr int kVecPerChunk = sizeof(T) == 4 ? 2 : 1; // 16-byte pieces per chunk
  static constexpr int kMaxKg = 2 * kSlotBytes / (int)sizeof(T);   // a warp's whole staging area
};

// ---- segment ranges and staging --------------------------------------------------------------------
struct RowRange { int64_t begin, end; };
__device__ __forceinline__ RowRange cta_range(int64_t segments) {
  RowRange r;
  r.begin = segments * (int64_t)blockIdx.x / (int64_t)gridDim.x;
  r.end = segments * ((int64_t)blockIdx.x + 1) / (int64_t)gridDim.x;
  return r;
}
// 16-byte asynchronous copy with an L2 eviction policy for the line it reads.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;"
               ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc), "l"(policy) : "memory");
}
// keep = true: the lines are read again soon (first per-tensor pass); false: this is their last use.
__device__ __forceinline__ uint64_t l2_policy(bool keep) {
  uint64_t p;
  if (keep) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  else asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// All of this thread's copy groups but the newest are complete; __syncwarp() makes the other
// lanes' pieces visible too.
__device__ __forceinline__ void cp_async_wait_but_newest() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// ---- bulk copies ---------------------------------------------------------------------------------------
// With a status word to report through, a segment travels as ONE bulk copy issued by lane 0 and
// completing on an mbarrier of the warp's slot: the 16 (or 32) cp.async per lane it replaces cost a
// warp about 1000 clocks of issue per 8 KB.  The wait for it is bounded; a limit that runs out is
// recorded in the status word and the kernel goes on (its outputs are then undefined), so nothing
// can hang.  Without a status word the per-lane copies are used: their wait is not a spin loop.
constexpr unsigned kMeetSpins = 1u << 22;                     // polls of a barrier or of the arrival tags
constexpr unsigned long long kMeetNs = 2000000000ull;         // and a 2 s limit on the clock
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// One lane, after the warp has finished reading dst.  bytes is a multiple of 16.
__device__ __forceinline__ void bulk_issue(void* dst, const void* src, uint32_t bytes, unsigned long long* bar,
                                           uint64_t policy) {
  const uint32_t b = smem_u32(bar);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the lanes' reads of the slot come first
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory");
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(b), "l"(policy) : "memory");
}
// Waits for phase `ph` of the barrier; false when the limit ran out first.
__device__ __forceinline__ bool bulk_wait(unsigned long long* bar, uint32_t ph) {
  const uint32_t b = smem_u32(bar);
  auto poll = [&]() {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(b), "r"(ph) : "memory");
    return ok != 0;
  };
  bool ok = poll();
  if (!ok) {
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (unsigned it = 0; it < kMeetSpins && !ok; ++it) {
      ok = poll();
      if (!ok && (it & 255u) == 255u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (now - t0 > kMeetNs) break;
      }
    }
  }
  return ok;
}

// A warp's staging area: 16 KB of shared memory (two slots, or one long one) and one mbarrier per slot.
struct Staging {
  uint4* slots;
  unsigned long long* bars;
  uint32_t* status;                                              // nullptr: per-lane cp.async
  uint32_t parity;                                               // bit c: phase of slot c's barrier to wait for
  __device__ __forceinline__ uint4* slot(int c) const { return slots + c * (kSlotBytes / 16); }
};
// Called by every thread before the kernel's first block barrier.
__device__ __forceinline__ Staging staging_init(unsigned char* stage, unsigned long long (*bars)[2], uint32_t* status) {
  const int warp = threadIdx.x >> 5;
  Staging sg{reinterpret_cast<uint4*>(stage + (size_t)warp * 2 * kSlotBytes), bars[warp], status, 0u};
  if ((threadIdx.x & 31) == 0) {
    for (int c = 0; c < 2; ++c) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[warp][c])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  return sg;
}
__device__ __forceinline__ void staging_wait(Staging& sg, int c, bool newest_pending, int lane) {
  if (sg.status) {
    if (!bulk_wait(&sg.bars[c], (sg.parity >> c) & 1u) && lane == 0) atomicExch(sg.status, (uint32_t)BL_ERR_TIMEOUT);
    sg.parity ^= 1u << c;
  } else if (newest_pending) {
    cp_async_wait_but_newest();
  } else {
    asm volatile("cp.async.wait_all;" ::: "memory");
  }
  __syncwarp();
}

// Draws the warp's next segment (-1 when the CTA's range is used up) and starts its copy into
// slot c (per-lane copies: also closes the copy group, an empty one when there is nothing left).
// reverse walks the range from its end: the second per-tensor pass then begins with the rows the
// first pass read last, the ones most likely still in L2.
template <typename T>
__device__ __forceinline__ int64_t stage_next(const T* __restrict__ x, const RowRange& rg, int64_t K, int G, int Kg,
                                              bool reverse, uint64_t policy, int* counter, const Staging& sg, int c,
                                              int lane) {
  int r = 0;
  if (lane == 0) r = atomicAdd(counter, 1);
  r = __shfl_sync(0xFFFFFFFFu, r, 0);
  int64_t seg = -1;
  if (rg.begin + r < rg.end) {
    seg = reverse ? rg.end - 1 - r : rg.begin + r;
    const T* src = x + (seg / G) * K + (seg % G) * (int64_t)Kg;
    if (sg.status) {
      if (lane == 0) bulk_issue(sg.slot(c), src, (uint32_t)(Kg * sizeof(T)), &sg.bars[c], policy);
    } else {
      const uint4* src16 = reinterpret_cast<const uint4*>(src);
      const int nv = Kg / 256 * RowTraits<T>::kVecPerChunk;    // 16-byte pieces per lane
#pragma unroll 4
      for (int i = 0; i < nv; ++i) cp_async16(sg.slot(c) + lane + 32 * i, src16 + lane + 32 * i, policy);
    }
  }
  if (!sg.status) cp_async_commit();
  return seg;
}

// The warp loop shared by the three kernels: body(seg, slot) runs with the segment staged and
// the next one already on its way.
template <typename T, typename Body>
__device__ __forceinline__ void for_each_segment(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg,
                                                 bool reverse, uint64_t policy, int* counter, Staging& sg,
                                                 int64_t first_seg, Body body) {
  const int lane = threadIdx.x & 31;
  const RowRange rg = cta_range(segments);
  // A segment of up to kSlotBytes leaves room for two slots (the next copy overlaps this body); a
  // longer one (up to 2 * kSlotBytes) fills the warp's whole area and its successor is copied after
  // the body, the other warps' copies and bodies covering for it.
  const bool two_slots = Kg * (int)sizeof(T) <= kSlotBytes;
  int cur = 0;
  int64_t seg = first_seg;
  while (seg >= 0) {
    int64_t next = -1;
    if (two_slots) next = stage_next<T>(x, rg, K, G, Kg, reverse, policy, counter, sg, cur ^ 1, lane);
    staging_wait(sg, cur, two_slots, lane);
    body(seg, sg.slot(cur));
    __syncwarp();                                    // every lane is done with the slot before it is refilled
    if (two_slots) cur ^= 1;
    else next = stage_next<T>(x, rg, K, G, Kg, reverse, policy, counter, sg, 0, lane);
    seg = next;
  }
}
// First draw of a warp (into slot 0), split off so that a kernel can put work between it and the loop.
template <typename T>
__device__ __forceinline__ int64_t first_segment(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg,
                                                 bool reverse, uint64_t policy, int* counter, const Staging& sg) {
  return stage_next<T>(x, cta_range(segments), K, G, Kg, reverse, policy, counter, sg, 0, threadIdx.x & 31);
}

template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 1)
rows_per_token(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, int mode, float ln_eps,
               double inv_kg, uint32_t* status, int clear_status, int8_t* __restrict__ x_q,
               float* __restrict__ gamma, float* __restrict__ eta) {
  extern __shared__ __align__(16) unsigned char stage[];
  __shared__ int counter;
  __shared__ unsigned long long copy_bar[kRowWarps][2];
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) counter = 0;
  Staging sg = staging_init(stage, copy_bar, status);
  pdl_launch_dependents();
  __syncthreads();
  pdl_wait();
  if (status && clear_status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0u;   // a timeout comes seconds later
  const int ni = Kg / 256;
  const uint64_t pol = l2_policy(false);
  const int64_t first = first_segment<T>(x, segments, K, G, Kg, false, pol, &counter, sg);
  for_each_segment<T>(x, segments, K, G, Kg, false, pol, &counter, sg, first, [&](int64_t seg, const uint4* slot) {
    const RowStats st = row_stats<T>(slot, ni, lane, ln_eps, inv_kg);
    const double lo = ((double)st.xlo - st.mean) * st.rstd, hi = ((double)st.xhi - st.mean) * st.rstd;
    double gam, et;
    scope_gamma_eta(mode, lo, hi, gam, et);
    const RowMap map = row_map(mode, st.mean, st.rstd, gam, et, st.xlo, st.xhi);
    if (lane == 0) {
      gamma[seg] = (float)gam;
      if (eta) eta[seg] = (float)et;
    }
    row_store_codes<T>(slot, ni, lane, map, x_q + (seg / G) * K + (seg % G) * (int64_t)Kg);
  });
}

// Per-tensor scope, first pass: the segment records, and per CTA and group the extremes of x^ on
// the order-preserving encoding (plain stores: every CTA writes its own G entries, the second pass
// folds them; no atomics on global memory and nothing to initialise).
template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 1)
rows_tensor_stats(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, float ln_eps, double inv_kg,
                  ScopePartial* __restrict__ partials, SegRecord* __restrict__ recs, uint32_t* status,
                  int clear_status) {
  extern __shared__ __align__(16) unsigned char stage[];
  __shared__ int counter;
  __shared__ unsigned long long part_lo[BL_MAX_GROUPS], part_hi[BL_MAX_GROUPS];
  __shared__ unsigned long long copy_bar[kRowWarps][2];
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) counter = 0;
  Staging sg = staging_init(stage, copy_bar, status);
  if (threadIdx.x < BL_MAX_GROUPS) { part_lo[threadIdx.x] = ~0ull; part_hi[threadIdx.x] = 0ull; }
  __syncthreads();
  pdl_wait();
  // Only now may the second pass be scheduled: its CTAs read x before their own wait, which is
  // safe because every CTA of this kernel has by then seen x complete.
  pdl_launch_dependents();
  if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0u;   // a timeout comes seconds later
  const int ni = Kg / 256;
  const uint64_t pol = l2_policy(true);                  // the second pass reads x again
  const int64_t first = first_segment<T>(x, segments, K, G, Kg, false, pol, &counter, sg);
  for_each_segment<T>(x, segments, K, G, Kg, false, pol, &counter, sg, first, [&](int64_t seg, const uint4* slot) {
    const RowStats st = row_stats<T>(slot, ni, lane, ln_eps, inv_kg);
    if (lane == 0) {
      const int g = (int)(seg % G);
      recs[seg] = SegRecord{st.mean, st.rstd, st.xlo, st.xhi};
      atomicMin(&part_lo[g], enc_ordered64(((double)st.xlo - st.mean) * st.rstd));
      atomicMax(&part_hi[g], enc_ordered64(((double)st.xhi - st.mean) * st.rstd));
    }
  });
  __syncthreads();
  if (threadIdx.x < G)
    partials[(size_t)blockIdx.x * G + threadIdx.x] = ScopePartial{part_lo[threadIdx.x], part_hi[threadIdx.x]};
}

// Second pass: folds the first pass's `stat_ctas` partial extremes into gamma / eta per group,
// then writes the codes.
template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 1)
rows_tensor_codes(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, int mode, int stat_ctas,
                  const ScopePartial* __restrict__ partials, const SegRecord* __restrict__ recs, uint32_t* status,
                  int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  extern __shared__ __align__(16) unsigned char stage[];
  __shared__ int counter;
  __shared__ double gam_s[BL_MAX_GROUPS], eta_s[BL_MAX_GROUPS];
  __shared__ unsigned long long copy_bar[kRowWarps][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) counter = 0;
  Staging sg = staging_init(stage, copy_bar, status);
  pdl_launch_dependents();
  __syncthreads();
  const int ni = Kg / 256;
  const uint64_t pol = l2_policy(false);
  // x was complete before the first pass let this kernel be scheduled (see there), so the first
  // copies start before the wait for the first pass's records and extremes.
  const int64_t first = first_segment<T>(x, segments, K, G, Kg, true, pol, &counter, sg);
  pdl_wait();
  for (int g = warp; g < G; g += kRowWarps) {
    unsigned long long lo = ~0ull, hi = 0ull;
    for (int c = lane; c < stat_ctas; c += 32) {
      const ScopePartial p = partials[(size_t)c * G + g];
      lo = min(lo, p.lo); hi = max(hi, p.hi);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    }
    if (lane == 0) {
      double gam, et;
      scope_gamma_eta(mode, dec_ordered64(lo), dec_ordered64(hi), gam, et);
      gam_s[g] = gam; eta_s[g] = et;
      if (blockIdx.x == 0) {
        gamma[g] = (float)gam;
        if (eta) eta[g] = (float)et;
      }
    }
  }
  __syncthreads();
  for_each_segment<T>(x, segments, K, G, Kg, true, pol, &counter, sg, first, [&](int64_t seg, const uint4* slot) {
    const SegRecord rec = recs[seg];
    const int g = (int)(seg % G);
    const RowMap map = row_map(mode, rec.mean, rec.rstd, gam_s[g], eta_s[g], rec.xlo, rec.xhi);
    row_store_codes<T>(slot, ni, lane, map, x_q + (seg / G) * K + g * (int64_t)Kg);
  });
}

// ---- per-tensor scope in one kernel ------------------------------------------------------------------
// Both passes in one cooperative launch (every CTA is resident, so they can wait for one another).
// Pass 1 as in rows_tensor_stats, except that the last two segments of every warp are handed out
// statically: they are still in the warp's two slots when the pass ends.  Then the CTAs meet: each
// publishes a tag (unique to the call, so the array needs no clearing) after its partial extremes,
// and waits, with a limit, until all tags of the grid show it.  Pass 2 codes the retained segments
// straight from shared memory (two per warp that are not read from HBM again) and then the rest of
// its range backwards, as rows_tensor_codes does.
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

template <typename T>
__global__ void __launch_bounds__(kRowWarps * 32, 1)
rows_tensor_fused(const T* __restrict__ x, int64_t segments, int64_t K, int G, int Kg, int mode, float ln_eps,
                  double inv_kg, ScopePartial* __restrict__ partials, SegRecord* __restrict__ recs,
                  unsigned long long* __restrict__ tags, unsigned long long* __restrict__ generation,
                  unsigned long long tag, unsigned long long wait_tag,
                  unsigned meet_polls, uint32_t* __restrict__ status, int clear_status, int8_t* __restrict__ x_q, float* __restrict__ gamma, float* __restrict__ eta) {
  extern __shared__ __align__(16) unsigned char stage[];
  __shared__ int counter1, counter2;
  __shared__ unsigned long long part_lo[BL_MAX_GROUPS], part_hi[BL_MAX_GROUPS];
  __shared__ double gam_s[BL_MAX_GROUPS], eta_s[BL_MAX_GROUPS];
  __shared__ unsigned long long copy_bar[kRowWarps][2];        // one mbarrier per warp and slot
  __shared__ unsigned long long gen_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { counter1 = 0; counter2 = 0; }
  Staging sg = staging_init(stage, copy_bar, status);
  if (threadIdx.x < BL_MAX_GROUPS) { part_lo[threadIdx.x] = ~0ull; part_hi[threadIdx.x] = 0ull; }
  __syncthreads();
  pdl_wait();
  pdl_launch_dependents();
  // The tag is a launch parameter, so a captured graph replays it; the workspace's generation count,
  // which CTA 0 advances after every meeting, makes what is published differ from launch to launch all
  // the same.  Any starting value will do: all CTAs of a launch read the same one (it only changes after
  // their meeting).  Visible to the whole CTA by the barriers ahead of the meeting.
  if (threadIdx.x == 0) gen_s = *generation;
  if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0u;   // a timeout (seconds later) overwrites it

  const RowRange rg = cta_range(segments);
  const int n = (int)(rg.end - rg.begin);
  const int n_keep = n < 2 * kRowWarps ? n : 2 * kRowWarps;     // handed out statically, stay in the slots
  const int n_dyn = n - n_keep;                                 // drawn through the counters
  const int ni = Kg / 256;
  auto slot_of = [&](int c) { return sg.slot(c); };
  const uint32_t seg_bytes = (uint32_t)(Kg * sizeof(T));
  auto issue = [&](int64_t seg, int c, uint64_t policy) {
    if (seg >= 0 && lane == 0)
      bulk_issue(sg.slot(c), x + (seg / G) * K + (seg % G) * (int64_t)Kg, seg_bytes, &sg.bars[c], policy);
  };
  auto arrived = [&](int c) { staging_wait(sg, c, false, lane); };

  // ---- pass 1
  bool dyn_done = n_dyn == 0;
  int statics = 0;
  auto draw1 = [&]() -> int64_t {
    if (!dyn_done) {
      int r = 0;
      if (lane == 0) r = atomicAdd(&counter1, 1);
      r = __shfl_sync(0xFFFFFFFFu, r, 0);
      if (r < n_dyn) return rg.begin + r;
      dyn_done = true;
    }
    const int j = warp + kRowWarps * statics;
    if (j < n_keep) { ++statics; return rg.begin + n_dyn + j; }
    return -1;
  };
  const uint64_t keep = l2_policy(true), last_use = l2_policy(false);
  int cur = 0;
  int64_t seg = draw1();
  issue(seg, 0, keep);
  int64_t seg_last = -1, seg_prev = -1;
  RowStats st_last = {0.0, 0.0, 0.f, 0.f}, st_prev = st_last;
  while (seg >= 0) {
    const int64_t next = draw1();
    issue(next, cur ^ 1, next >= rg.begin + n_dyn ? last_use : keep);
    arrived(cur);
    const RowStats st = row_stats<T>(slot_of(cur), ni, lane, ln_eps, inv_kg);
    if (lane == 0) {
      const int g = (int)(seg % G);
      recs[seg] = SegRecord{st.mean, st.rstd, st.xlo, st.xhi};
      atomicMin(&part_lo[g], enc_ordered64(((double)st.xlo - st.mean) * st.rstd));
      atomicMax(&part_hi[g], enc_ordered64(((double)st.xhi - st.mean) * st.rstd));
    }
    __syncwarp();
    seg_prev = seg_last; st_prev = st_last;
    seg_last = seg; st_last = st;
    seg = next;
    if (seg >= 0) cur ^= 1;                                     // cur stays on the last segment's slot
  }
  // retained: seg_last in slot cur, and (if the warp had two static draws) seg_prev in slot cur ^ 1
  const int kept = statics;                                      // 0, 1 or 2
  __syncthreads();
  if (threadIdx.x < G)
    partials[(size_t)blockIdx.x * G + threadIdx.x] = ScopePartial{part_lo[threadIdx.x], part_hi[threadIdx.x]};
  __syncthreads();

  // ---- the CTAs meet
  const unsigned long long mix = gen_s * 0x9E3779B97F4A7C15ull;
  tag ^= mix;
  wait_tag ^= mix;
  if (threadIdx.x == 0) { __threadfence(); st_release_u64(tags + blockIdx.x, tag); }
  bool here = true;
  if (threadIdx.x < gridDim.x) {
    here = false;
    unsigned long long t0 = 0;
    for (unsigned it = 0; it <= meet_polls; ++it) {
      if (ld_acquire_u64(tags + threadIdx.x) == wait_tag) { here = true; break; }
      if ((it & 63u) == 63u) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        else if (now - t0 > kMeetNs) break;
      }
      __nanosleep(64);
    }
  }
  if (!__syncthreads_and(here)) {                                // someone never arrived: codes are not written
    if (threadIdx.x == 0) atomicExch(status, (uint32_t)BL_ERR_TIMEOUT);
    return;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) *generation = gen_s + 1;   // every CTA has read it: all have arrived

  // ---- gamma / eta of every group from all CTAs' extremes
  for (int g = warp; g < G; g += kRowWarps) {
    unsigned long long lo = ~0ull, hi = 0ull;
    for (int c = lane; c < (int)gridDim.x; c += 32) {
      const ScopePartial p = partials[(size_t)c * G + g];
      lo = min(lo, p.lo); hi = max(hi, p.hi);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, o));
    }
    if (lane == 0) {
      double gam, et;
      scope_gamma_eta(mode, dec_ordered64(lo), dec_ordered64(hi), gam, et);
      gam_s[g] = gam; eta_s[g] = et;
      if (blockIdx.x == 0) {
        gamma[g] = (float)gam;
        if (eta) eta[g] = (float)et;
      }
    }
  }
  __syncthreads();

  // ---- pass 2
  auto code = [&](int64_t sg, const RowStats& st, const uint4* slot) {
    const int g = (int)(sg % G);
    const RowMap map = row_map(mode, st.mean, st.rstd, gam_s[g], eta_s[g], st.xlo, st.xhi);
    row_store_codes<T>(slot, ni, lane, map, x_q + (sg / G) * K + g * (int64_t)Kg);
  };
  auto draw2 = [&]() -> int64_t {
    int r = 0;
    if (lane == 0) r = atomicAdd(&counter2, 1);
    r = __shfl_sync(0xFFFFFFFFu, r, 0);
    return r < n_dyn ? rg.begin + n_dyn - 1 - r : -1;           // backwards: the rows read last first
  };
  if (kept >= 1) code(seg_last, st_last, slot_of(cur));
  __syncwarp();
  seg = n_dyn > 0 ? draw2() : -1;
  issue(seg, cur, last_use);                                     // overlaps the second retained segment
  if (kept >= 2) code(seg_prev, st_prev, slot_of(cur ^ 1));
  __syncwarp();
  while (seg >= 0) {
    const int64_t next = draw2();
    issue(next, cur ^ 1, last_use);
    const SegRecord rec = recs[seg];
    arrived(cur);
    code(seg, RowStats{rec.mean, rec.rstd, rec.xlo, rec.xhi}, slot_of(cur));
    __syncwarp();
    seg = next; cur ^= 1;
  }
}

// Unique, never zero, per call: high half drawn once per process, low half a call counter.
inline unsigned long long next_tag() {
  static const unsigned long long high = [] {
    std::random_device rd;
    return ((unsigned long long)rd() << 32) ^ ((unsigned long long)rd() << 13);
  }();
  static std::atomic<unsigned long long> calls{1};
  const unsigned long long t = (high & 0xFFFFFFFF00000000ull) | (calls.fetch_add(1) & 0xFFFFFFFFull);
  return t ? t : 1;
}

// cudaErrorNotSupported: the device or context cannot launch cooperatively (the caller falls back).
template <typename T>
cudaError_t launch_fused(const QuantArgs& a, cudaStream_t s, const T* x, int64_t segments, int Kg, double inv_kg,
                         unsigned grid, ScopePartial* partials, SegRecord* recs, uint32_t* status) {
  int dev = 0, coop = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return cudaErrorNotSupported;
  auto kern = rows_tensor_fused<T>;
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kRowStage)) != cudaSuccess) return e;
  // CTAs that can be resident at once on this device (cached per device ordinal)
  static std::atomic<int> resident[64] = {};
  int cap = dev < 64 ? resident[dev].load() : 0;
  if (cap == 0) {
    int per_sm = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kRowWarps * 32, kRowStage) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || per_sm < 1)
      return cudaErrorNotSupported;
    cap = per_sm * sms;
    if (dev < 64) resident[dev].store(cap);
  }
  if ((int64_t)grid > (int64_t)cap) grid = (unsigned)cap;
  unsigned long long* tags = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(a.ws) + kWsTagOff);
  unsigned long long* generation = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(a.ws) + kWsGenOff);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kRowWarps * 32);
  cfg.dynamicSmemBytes = kRowStage;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  static std::atomic<int> with_pdl{1};                          // dropped for good if the pair is refused once
  cfg.numAttrs = with_pdl.load() ? 2 : 1;
  const unsigned long long tag = next_tag();
  // test hook: a smaller poll limit, and a tag to wait for that no CTA publishes (the complement of this
  // call's tag: the array holds this call's tag or those of earlier calls, whose high half is the same)
  const long long dbg_polls = g_debug_wait_polls.load(std::memory_order_relaxed);
  const unsigned meet_polls = dbg_polls < 0 ? kMeetSpins : (unsigned)std::min<long long>(dbg_polls, kMeetSpins);
  const unsigned long long wait_tag = g_debug_meet_skew.load(std::memory_order_relaxed) ? ~tag : tag;
  const int clear = a.keep_status ? 0 : 1;
  e = cudaLaunchKernelEx(&cfg, kern, x, segments, a.K, a.G, Kg, (int)a.mode, a.ln_eps, inv_kg, partials, recs, tags,
                         generation, tag, wait_tag, meet_polls, status, clear, a.x_q, a.gamma, a.eta);
  if (e != cudaSuccess && cfg.numAttrs == 2) {
    (void)cudaGetLastError();
    with_pdl.store(0);
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, x, segments, a.K, a.G, Kg, (int)a.mode, a.ln_eps, inv_kg, partials, recs, tags,
                           generation, tag, wait_tag, meet_polls, status, clear, a.x_q, a.gamma, a.eta);
  }
  return e;
}

// Grid of the persistent kernels: one CTA per SM, never more CTAs than segments.
inline cudaError_t rows_grid(int64_t segments, unsigned* grid) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  int64_t g = sms < kMaxStatCtas ? sms : kMaxStatCtas;
  if (g > segments) g = segments;
  *grid = (unsigned)(g < 1 ? 1 : g);
  return cudaSuccess;
}

template <typename T>
cudaError_t run_rows(const QuantArgs& a, cudaStream_t s) {
  const T* x = reinterpret_cast<const T*>(a.x);
  const int Kg = (int)(a.K / a.G);
  const int64_t segments = a.M * a.G;
  const double inv_kg = 1.0 / (double)Kg;
  constexpr int kThreads = kRowWarps * 32;
  unsigned grid = 1;
  cudaError_t e = rows_grid(segments, &grid);
  if (e != cudaSuccess) return e;
  const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  const int clear = a.keep_status ? 0 : 1;
  if (a.gran == BL_PER_TOKEN) {                                  // a.status may be nullptr: per-lane copies then
    if ((e = cudaFuncSetAttribute(rows_per_token<T>, attr, kRowStage)) != cudaSuccess) return e;
    return launch_pdl(rows_per_token<T>, grid, kThreads, kRowStage, s, x, segments, a.K, a.G, Kg, (int)a.mode,
                      a.ln_eps, inv_kg, a.status, clear, a.x_q, a.gamma, a.eta);
  }
  ScopePartial* partials = reinterpret_cast<ScopePartial*>(reinterpret_cast<char*>(a.ws) + kWsPartialOff);
  SegRecord* recs = reinterpret_cast<SegRecord*>(reinterpret_cast<char*>(a.ws) + kWsHeaderBytes);
  uint32_t* status = a.status ? a.status : reinterpret_cast<uint32_t*>(a.ws);
  if (Kg * (int)sizeof(T) <= kSlotBytes) {                       // two slots per warp: both passes in one kernel
    e = launch_fused<T>(a, s, x, segments, Kg, inv_kg, grid, partials, recs, status);
    if (e != cudaErrorNotSupported) return e;                    // no cooperative launch here: two kernels
    (void)cudaGetLastError();
  }
  if ((e = cudaFuncSetAttribute(rows_tensor_stats<T>, attr, kRowStage)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(rows_tensor_codes<T>, attr, kRowStage)) != cudaSuccess) return e;
  e = launch_pdl(rows_tensor_stats<T>, grid, kThreads, kRowStage, s, x, segments, a.K, a.G, Kg, a.ln_eps, inv_kg,
                 partials, recs, status, clear);
  if (e != cudaSuccess) return e;
  return launch_pdl(rows_tensor_codes<T>, grid, kThreads, kRowStage, s, x, segments, a.K, a.G, Kg, (int)a.mode,
                    (int)grid, (const ScopePartial*)partials, (const SegRecord*)recs, status, a.x_q, a.gamma, a.eta);
}

constexpr size_t kStaticSmemSlack = 4096;   // more than any kernel here declares statically

template <typename T>
cudaError_t run(const QuantArgs& a, cudaStream_t s) {
  const T* x = reinterpret_cast<const T*>(a.x);
  const int64_t Kg = a.K / a.G;
  const size_t smem = (size_t)Kg * sizeof(float);
  const unsigned grid = (unsigned)(a.M * a.G);
  cudaError_t e;
  if (Kg % 256 == 0 && Kg <= RowTraits<T>::kMaxKg)               // whole chunks per lane, segment fits a slot
    return run_rows<T>(a, s);
  if (a.gran == BL_PER_TOKEN) {
    // no device-side wait in this kernel: the word is only cleared for whoever reads it afterwards
    if (a.status && !a.keep_status && (e = cudaMemsetAsync(a.status, 0, sizeof(uint32_t), s)) != cudaSuccess) return e;
    if (smem + kStaticSmemSlack > 48 * 1024) {      // the 48 KB default covers static and dynamic together
      e = cudaFuncSetAttribute(quant_per_token<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    quant_per_token<T><<<grid, kQuantThreads, smem, s>>>(x, a.K, a.G, (int)a.mode, a.ln_eps, a.x_q,
                                                        a.gamma, a.eta);
    return cudaGetLastError();
  }
  TensorScope* sc = reinterpret_cast<TensorScope*>(reinterpret_cast<char*>(a.ws) + kWsScopeOff);
  SegRecord* recs = reinterpret_cast<SegRecord*>(reinterpret_cast<char*>(a.ws) + kWsHeaderBytes);
  if (smem + kStaticSmemSlack > 48 * 1024) {
    e = cudaFuncSetAttribute(tensor_stats<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  init_scope<<<1, BL_MAX_GROUPS, 0, s>>>(sc, a.status ? a.status : reinterpret_cast<uint32_t*>(a.ws),
                                         a.keep_status ? 0 : 1);
  tensor_stats<T><<<grid, kQuantThreads, smem, s>>>(x, a.K, a.G, a.ln_eps, sc, recs);
  tensor_codes<T><<<grid, kQuantThreads, 0, s>>>(x, a.K, a.G, (int)a.mode, sc, recs, a.x_q, a.gamma, a.eta);
  return cudaGetLastError();
}

}  // namespace

size_t quant_ws_bytes(int64_t M, int G) {
  return kWsHeaderBytes + (size_t)M * (size_t)G * sizeof(SegRecord);
}

// ---- built-in scratch of bitlinear_quant_act_noalloc -------------------------------------------
// Room for the per-tensor statistics of up to BL_NOALLOC_MAX_SEGMENTS (token, group) segments.
// The array lives in the library image: every GPU that loads the library holds these bytes until
// the process exits.  Host code must not hand the symbol itself to a kernel (on the host the name
// is only a stand-in); it asks the runtime for the device address once per device.
constexpr size_t kNoAllocBytes = kWsHeaderBytes + (size_t)BL_NOALLOC_MAX_SEGMENTS * sizeof(SegRecord);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Device address of the built-in scratch on the current device (cached per device ordinal).
static cudaError_t noalloc_scratch_address(void** out) {
  constexpr int kMaxDevices = 64;
  static void* cached[kMaxDevices] = {};
  static std::mutex guard;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(guard);
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    cached[dev] = p;
  }
  *out = cached[dev];
  return cudaSuccess;
}

cudaError_t launch_quant_act(const QuantArgs& a, cudaStream_t s) {
  switch (a.xt) {
    case BL_F32: return run<float>(a, s);
    case BL_F16: return run<__half>(a, s);
    case BL_BF16: return run<__nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl

extern "C" bl_status bitlinear_quant_act_noalloc(const void* x, bl_dtype xt, int64_t M, int64_t K, int G, int b,
                                                 bl_quant_mode mode, bl_gran gran, float ln_eps, int8_t* x_q,
                                                 float* gamma, float* eta, void* stream) {
  // Refuse what the built-in scratch cannot hold before anything else is looked at.
  if (M > 0 && G > 0 && gran == BL_PER_TENSOR && M * (int64_t)G > (int64_t)BL_NOALLOC_MAX_SEGMENTS)
    return BL_ERR_TOO_LARGE;
  void* scratch = nullptr;
  if (bl::noalloc_scratch_address(&scratch) != cudaSuccess) return BL_ERR_CUDA;
  // Same validation and the same kernels as bitlinear_quant_act, with the scratch passed as its
  // workspace.  The first pass rewrites every record and every partial extreme that the second
  // pass reads (the long-segment kernels reset their running extremes first), so nothing of an
  // earlier call survives into this one.
  return bitlinear_quant_act(x, xt, M, K, G, b, mode, gran, ln_eps, x_q, gamma, eta, scratch,
                             bl::kNoAllocBytes, stream);
}

extern "C" bl_status bitlinear_noalloc_status(void* stream) {
  void* scratch = nullptr;
  if (bl::noalloc_scratch_address(&scratch) != cudaSuccess) return BL_ERR_CUDA;
  uint32_t word = 0;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BL_ERR_CUDA;
  if (cudaMemcpy(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return BL_ERR_CUDA;
  return word == 0 ? BL_OK : BL_ERR_TIMEOUT;
}
