// Step 4 of BitLinear on the 5th-generation tensor cores, two SMs per tile: acc = W~ x~ (Eq. 7)
// as tcgen05.mma.cta_group::2 kind::i8 MMAs of 256 x 256 x 32, with the Eq. 11 rescale fused into
// the epilogue.
//
// A cluster of two CTAs owns a tile of 256 tokens x 256 output features.  CTA r (its rank in the
// cluster) holds tokens 128 r .. 128 r + 127 of the tile: their codes arrive by TMA, their
// accumulators live in its own tensor memory, its epilogue warps write their rows of y.  The B
// operand (the weights) is shared by the pair: CTA r expands only rows 128 r .. 128 r + 127 of the
// 256-row weight tile from 1 bit to +-1 bytes into its own shared memory, and the MMA reads both
// halves.  Compared with one SM per tile this halves, per SM, the expansion arithmetic, the
// expansion stores and the tensor core's reads of B.
//
// Roles per CTA:
//   warp 0      TMA producer for this CTA's codes tile
//   warp 1      rank 0: MMA issuer for the pair (one thread); idle in rank 1
//   warp 2      tensor-memory allocation (both CTAs, cta_group::2)
//   warps 4-11  epilogue: warp w reads the tensor-memory lanes of its quarter (w % 4) and takes half
//               of the tile's 256 columns (warps 4-7 the first 128, warps 8-11 the rest)
//   warps 12-19 weight expanders: two groups of 4 warps, group e fills k-block e of every ring slot;
//               thread u of a group owns row u of this CTA's 128-row half of the B tile
// A ring slot holds two k-blocks (256 weights): the MMA issuer, whose serial work per barrier round
// trip bounds the kernel, waits and commits once per slot and issues 8 MMAs in between.
// Barriers.  In every CTA: empty (stage consumed; the issuer commits to both CTAs' copies) and
// tmem_full (accumulator complete; committed to both).  full (rank 0 only): one barrier per slot
// collects the TMA bytes of both CTAs' codes tiles (rank 1's copies complete on rank 0's barrier:
// cp.async.bulk.tensor.cta_group::2) and the expander warps of the pair, so the issuer waits once
// per slot.  tmem_empty (rank 0) takes the 16 epilogue warps of the pair.  Remote arrivals are
// mbarrier.arrive on the mapa address of rank 0's barrier.
//
// Every wait is bounded; a limit that runs out raises the CTA's abort flag, records
// BL_ERR_TIMEOUT and lets every role fall through to the common exit (cluster barrier, tensor
// memory freed).  The partner then runs into its own limits.  No multicast loads are used.
#include <atomic>

#include "tc_common.cuh"

namespace bl {

namespace {

using namespace tc;

constexpr int kBM = 128;                 // tokens per CTA (tensor-memory lanes)
constexpr int kPairM = 256;              // tokens per tile
constexpr int kBN = 256;                 // output features per tile (MMA N)
constexpr int kHalfN = 128;              // weight rows expanded per CTA
constexpr int kBK = 128;                 // weights per k-block (one 128-byte swizzle atom)
constexpr int kSub = 2;                  // k-blocks per ring slot: one barrier round trip per 256 weights
constexpr int kSlots = 3;                // ring slots of kSub x (codes tile + weights half-tile)
constexpr int kGroups = kSub;            // expander groups of 4 warps; group e fills k-block e of every slot
constexpr int kExpandWarp0 = 12;
constexpr int kEpiWarps = 8;             // two per lane quarter; with four, heavier epilogues (residual, ReLU)
                                         // and short K left the MMAs waiting for a free accumulator
constexpr int kThreads = (kExpandWarp0 + 4 * kGroups) * 32;
constexpr int kEpiWarp0 = 4;
constexpr int kABytes = kBM * kBK;       // 16 KB
constexpr int kBBytes = kHalfN * kBK;    // 16 KB
constexpr int kStageBytes = kABytes + kBBytes;   // one k-block
constexpr int kSlotBytes = kSub * kStageBytes;
constexpr int kTmemCols = 512;
constexpr int kMaxCtas = 160;
constexpr size_t kScratchPerCta = (size_t)kBM * kBN * sizeof(float);

struct SharedCtl {
  unsigned long long full[kSlots];       // rank 0: everything a slot needs (see below); rank 1: own TMA bytes
  unsigned long long empty[kSlots];
  unsigned long long tmem_full[2], tmem_empty[2];               // tmem_empty used in rank 0 only
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t kSmemBytes = (size_t)kSlots * kSlotBytes + 1024 + sizeof(SharedCtl) + 64;
static_assert(kSmemBytes <= 232448, "exceeds the shared memory of one CTA");

// kind::i8 instruction descriptor: s32 accumulate, s8 x s8, both operands K-major, 256 x 256.
constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                            ((uint32_t)(kPairM >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same variable in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Waits on barriers that the partner CTA (or a tcgen05.commit of the pair) arrives on use the same
// bounded CTA-scope wait as local ones: what crosses CTAs here is only the barrier count itself;
// the data behind it is read by the tensor core (async proxy), not by this CTA's threads.
__device__ __forceinline__ bool mbar_wait2(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait(bar, parity, abort_flag);
}
// TMA tile load whose completion bytes are counted on a barrier that may live in the partner CTA
// (the destination is always this CTA's shared memory).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t bar_cluster_addr, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on `cluster_addr` (any CTA of the cluster) once all MMAs issued so far have completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_addr)
               : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

struct PairIter {            // tiles of this cluster, in the order every role of both CTAs walks them
  uint32_t t, tiles, m_tiles, stride;
  __device__ PairIter(uint32_t tiles_, uint32_t m_tiles_)
      : t(blockIdx.x >> 1), tiles(tiles_), m_tiles(m_tiles_), stride(gridDim.x >> 1) {}
  __device__ bool valid() const { return t < tiles; }
  __device__ void next() { t += stride; }
  __device__ uint32_t m_tile() const { return t % m_tiles; }
  __device__ uint32_t n_tile() const { return t / m_tiles; }
};

// One ring slot's worth of work: up to kSub consecutive k-blocks of one (tile, group).  Every role
// of both CTAs walks the same sequence of steps.
struct StepIter {
  PairIter it;
  int g, t, G, spg, kbg;                      // group, step in group; groups, steps per group, k-blocks per group
  __device__ StepIter(uint32_t tiles, uint32_t m_tiles, int G_, int kbg_)
      : it(tiles, m_tiles), g(0), t(0), G(G_), spg((kbg_ + kSub - 1) / kSub), kbg(kbg_) {}
  __device__ bool valid() const { return it.valid(); }
  __device__ void next() { if (++t == spg) { t = 0; if (++g == G) { g = 0; it.next(); } } }
  __device__ int nblk() const { const int r = kbg - t * kSub; return r < kSub ? r : kSub; }
  __device__ int kb0() const { return g * kbg + t * kSub; }   // first k-block of the step
  __device__ bool first() const { return t == 0; }
  __device__ bool last() const { return t + 1 == spg; }
};

// kMode 0: write int32 accumulators acc[g,m,n].  kMode 1: write y (Eq. 11).  kMode 2: the same with
// the epilogue options (beta per block of output features, ReLU, residual, row stride of y).
template <int kMode, typename TY>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_x, GemmArgs a, int tx_bytes) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + (size_t)kSlots * kSlotBytes);
  volatile int* abort_flag = &ctl->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;
  pdl_launch_dependents();

  const uint32_t m_tiles = (uint32_t)((a.M + kPairM - 1) / kPairM), n_tiles = (uint32_t)((a.N + kBN - 1) / kBN);
  const uint32_t tiles = m_tiles * n_tiles;
  const int k_blocks = (int)(a.K / kBK);             // stages per tile (all groups)
  const int kb_per_group = k_blocks / a.G;
  const int64_t w_blocks_n = (a.N + 127) / 128;      // 128-row blocks present in W_packed
  const int64_t w_blocks_k = (a.K + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) {
      // rank 0's full barrier collects, per slot: the TMA producers of both CTAs (1 arrival each,
      // plus the bytes of both codes tiles) and the expander warps of both CTAs (2 x kGroups x 4),
      // so the MMA issuer makes one wait per slot.  Rank 1's copy is unused.
      mbar_init(smem_u32(&ctl->full[s]), 2 + 2 * kGroups * (kHalfN / 32));
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 2 * kEpiWarps);
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // both CTAs' barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  // Everything above touched only this cluster's shared and tensor memory, so it may overlap the
  // end of the kernel before this one on the stream; from here on global memory is read.
  pdl_wait();
  if (blockIdx.x == 0 && threadIdx.x == 0 && !a.keep_status) *a.status = 0u;   // a timeout (seconds later) overwrites it

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (own codes)
    if (lane == 0) {
      int slot = 0; uint32_t phase = 0;
      const uint32_t full0 = map_to_rank(smem_u32(&ctl->full[0]), 0);      // both CTAs report to rank 0
      for (StepIter st(tiles, m_tiles, a.G, kb_per_group); st.valid(); st.next()) {
        const int m0 = (int)(st.it.m_tile() * kPairM + rank * kBM);
        if (!mbar_wait2(smem_u32(&ctl->empty[slot]), phase ^ 1u, abort_flag)) break;
        const uint32_t bar = full0 + 8u * (uint32_t)slot;
        const int nblk = st.nblk();
        mbar_arrive_expect_tx_cluster(bar, (uint32_t)(tx_bytes * nblk));
        for (int j = 0; j < nblk; ++j)
          tma_load_2d_pair(smem_u32(smem + (size_t)slot * kSlotBytes + (size_t)j * kStageBytes), &map_x,
                           (st.kb0() + j) * kBK, m0, bar);
        if (++slot == kSlots) { slot = 0; phase ^= 1u; }
      }
      // Every copy issued here is consumed by an MMA before the accumulator it feeds is released,
      // and the epilogue warps of this CTA wait for that release: no copy is in flight at exit.
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- rank 0: MMA issuer for the pair
    if (lane == 0 && leader) {
      int slot = 0; uint32_t phase = 0;
      uint32_t pass = 0;
      uint32_t d_tmem = tmem_base, buf = 0;
      const uint32_t empty0 = map_to_rank(smem_u32(&ctl->empty[0]), 0), empty1 = map_to_rank(smem_u32(&ctl->empty[0]), 1);
      const uint32_t tfull0 = map_to_rank(smem_u32(&ctl->tmem_full[0]), 0), tfull1 = map_to_rank(smem_u32(&ctl->tmem_full[0]), 1);
      for (StepIter st(tiles, m_tiles, a.G, kb_per_group); st.valid(); st.next()) {
        if (st.first()) {                                      // a new (tile, group): next accumulator
          buf = pass & 1u;
          const uint32_t acc_phase = (pass >> 1) & 1u;
          if (!mbar_wait2(smem_u32(&ctl->tmem_empty[buf]), acc_phase ^ 1u, abort_flag)) break;
          tc_fence_after();
          d_tmem = tmem_base + buf * (uint32_t)kBN;
        }
        if (!mbar_wait2(smem_u32(&ctl->full[slot]), phase, abort_flag)) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)slot * kSlotBytes);
        const int nblk = st.nblk();
        for (int b = 0; b < nblk; ++b) {
          const uint64_t adesc = smem_desc_sw128(a_addr + (uint32_t)b * kStageBytes);
          const uint64_t bdesc = smem_desc_sw128(a_addr + (uint32_t)b * kStageBytes + kABytes);
#pragma unroll
          for (int j = 0; j < kBK / 32; ++j)
            mma_i8_pair(d_tmem, adesc + (uint64_t)(2 * j), bdesc + (uint64_t)(2 * j), kIdesc,
                        (!st.first() || b > 0 || j > 0) ? 1u : 0u);
        }
        mma_commit_pair(empty0 + 8u * (uint32_t)slot);
        mma_commit_pair(empty1 + 8u * (uint32_t)slot);
        if (++slot == kSlots) { slot = 0; phase ^= 1u; }
        if (st.last()) {                                       // accumulator of this (tile, group) complete
          mma_commit_pair(tfull0 + 8u * buf);
          mma_commit_pair(tfull1 + 8u * buf);
          ++pass;
        }
      }
    }
  } else if (warp >= kExpandWarp0) {
    // ---------------------------------------------------------------- weight expanders (own half of B)
    const int eg = (warp - kExpandWarp0) >> 2;                       // group: fills k-block eg of every slot
    const int u = (threadIdx.x - kExpandWarp0 * 32) & (kHalfN - 1);  // row of this CTA's half, 0..127
    const uint32_t row_base = smem_u32(smem) + (uint32_t)eg * kStageBytes + (uint32_t)kABytes + (uint32_t)u * 128u +
                              ((uint32_t)(u & 7) << 4);
    int slot = 0; uint32_t phase = 0;
    const uint32_t full0 = map_to_rank(smem_u32(&ctl->full[0]), 0);
    // the 16 bytes of sign bits of the next two steps are prefetched in registers
    StepIter pf(tiles, m_tiles, a.G, kb_per_group);
    auto fetch = [&]() -> uint4 {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (pf.valid()) {
        const int64_t nb = (int64_t)pf.it.n_tile() * 2 + rank;
        if (eg < pf.nblk() && nb < w_blocks_n)
          v = __ldg(reinterpret_cast<const uint4*>(a.W_packed + (nb * w_blocks_k + pf.kb0() + eg) * 2048 + u * 16));
        pf.next();
      }
      return v;
    };
    uint4 b0 = fetch(), b1 = fetch();
    for (StepIter st(tiles, m_tiles, a.G, kb_per_group); st.valid(); st.next()) {
      const uint4 cur = b0;
      b0 = b1;
      b1 = fetch();
      bool got = true;
      if (lane == 0) got = mbar_wait2(smem_u32(&ctl->empty[slot]), phase ^ 1u, abort_flag);
      got = __shfl_sync(0xFFFFFFFFu, got, 0);
      __syncwarp();
      if (!got) break;
      if (eg < st.nblk()) {
        const uint32_t dst = row_base + (uint32_t)slot * (uint32_t)kSlotBytes;
        const uint32_t words[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t wd = words[c >> 1];
          const int j0 = (c & 1) * 4;
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst ^ ((uint32_t)c << 4)),
                       "r"(signs4(wd, j0)), "r"(signs4(wd, j0 + 1)), "r"(signs4(wd, j0 + 2)),
                       "r"(signs4(wd, j0 + 3)) : "memory");
        }
        fence_proxy_async_smem();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(full0 + 8u * (uint32_t)slot);
      if (++slot == kSlots) { slot = 0; phase ^= 1u; }
    }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + kEpiWarps) {
    // ---------------------------------------------------------------- epilogue (own 128 tokens)
    const int q = warp & 3;                                  // lane quarter this warp may read
    const int row = q * 32 + lane;
    uint32_t pass = 0;
    bool ok = true;
    float* run = reinterpret_cast<float*>(reinterpret_cast<char*>(a.scratch) + (size_t)blockIdx.x * kScratchPerCta);
    const bool correct = (kMode >= 1) && a.eta_correction != 0;
    for (PairIter it(tiles, m_tiles); ok && it.valid(); it.next()) {
      const int64_t m = (int64_t)it.m_tile() * kPairM + rank * kBM + row;
      const int64_t n_base = (int64_t)it.n_tile() * kBN;
      const bool m_ok = m < a.M;
      for (int g = 0; g < a.G; ++g, ++pass) {
        const uint32_t buf = pass & 1u, acc_phase = (pass >> 1) & 1u;
        bool got = mbar_wait2(smem_u32(&ctl->tmem_full[buf]), acc_phase, abort_flag);
        got = __all_sync(0xFFFFFFFFu, got);
        if (!got) { ok = false; break; }
        tc_fence_after();
        // one beta for the tile (beta_rows == 0) or one per 32-column chunk, loaded below
        float gamma_m = 0.f, eta_m = 0.f, beta_c = 0.f;
        if (kMode >= 1 && m_ok) {
          const int64_t sc = (a.gran == BL_PER_TOKEN) ? m * a.G + g : g;
          gamma_m = a.gamma[sc];
          if (correct) eta_m = a.eta[sc];
        }
        if (kMode == 1 || (kMode == 2 && a.beta_rows == 0)) beta_c = a.beta[g];
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)kBN;
        const int c_first = ((warp - kEpiWarp0) >> 2) * (kBN / 64);      // this warp's half of the columns
#pragma unroll 1
        for (int c = c_first; c < c_first + kBN / 64; ++c) {
          const int64_t n0 = n_base + c * 32;
          // beta blocks are multiples of 32 output features: one value per chunk, fetched while the
          // accumulators travel from tensor memory
          if (kMode == 2 && a.beta_rows > 0 && n0 < a.N) beta_c = __ldg(a.beta + (n0 / a.beta_rows) * a.G + g);
          uint32_t r[32];
          tmem_ld32(taddr + (uint32_t)(c * 32), r);
          if (n0 >= a.N) continue;                           // uniform across the warp
          if (kMode == 0) {
            if (m_ok) {
              int32_t* dst = a.acc + ((int64_t)g * a.M + m) * a.N + n0;
              if (n0 + 32 <= a.N && (a.N & 3) == 0 && aligned32(dst)) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const uint32_t w[8] = {r[8 * i], r[8 * i + 1], r[8 * i + 2], r[8 * i + 3],
                                         r[8 * i + 4], r[8 * i + 5], r[8 * i + 6], r[8 * i + 7]};
                  st_global_256(dst + 8 * i, w);
                }
              } else if (n0 + 32 <= a.N && (a.N & 3) == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  *reinterpret_cast<uint4*>(dst + 4 * i) = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) if (n0 + i < a.N) dst[i] = (int32_t)r[i];
              }
            }
          } else {
            const float scale = beta_c * gamma_m * kInvQb, eta_beta = eta_m * beta_c;
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              float t = (float)(int32_t)r[i] * scale;
              if (correct) {
                const int64_t n = n0 + i;
                const int rs = (n < a.N) ? __ldg(a.rowsum + n * a.G + g) : 0;
                t += eta_beta * (float)rs;
              }
              v[i] = t;
            }
            if (a.G > 1) {
              float* rp = run + (size_t)(c * 32) * kBM + row;      // [column][row]: coalesced per column
              if (g > 0) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = rp[(size_t)i * kBM] + v[i];
              }
              if (g + 1 < a.G) {
#pragma unroll
                for (int i = 0; i < 32; ++i) rp[(size_t)i * kBM] = v[i];
              }
            }
            if (g + 1 == a.G && m_ok) {
              if (kMode == 2 && a.relu) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = fmaxf(v[i], 0.f);
              }
              if (kMode == 2 && a.residual) {
                const TY* res = reinterpret_cast<const TY*>(a.residual) + m * a.ld_res + n0;
                if (n0 + 32 <= a.N && (a.ld_res * sizeof(TY)) % 16 == 0) {
                  constexpr int kPer = 16 / (int)sizeof(TY);           // elements per 16-byte load
#pragma unroll
                  for (int i = 0; i < 32 / kPer; ++i) {
                    const uint4 w = *reinterpret_cast<const uint4*>(res + i * kPer);
                    const TY* e = reinterpret_cast<const TY*>(&w);
#pragma unroll
                    for (int j = 0; j < kPer; ++j) v[i * kPer + j] += in_cast(e[j]);
                  }
                } else {
#pragma unroll
                  for (int i = 0; i < 32; ++i) if (n0 + i < a.N) v[i] += in_cast(res[i]);
                }
              }
              const int64_t ldy = (kMode == 2 && a.ld_y > 0) ? a.ld_y : a.N;
              TY* dst = reinterpret_cast<TY*>(a.y) + m * ldy + n0;
              const bool vec_ok = (n0 + 32 <= a.N) && ((ldy * sizeof(TY)) % 16 == 0);
              store_row32<TY>(dst, v, n0, a.N, vec_ok);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&ctl->tmem_empty[buf]), 0));
      }
    }
  }

  // ---------------------------------------------------------------- common exit
  if (*abort_flag && threadIdx.x == 0) atomicExch(a.status, (uint32_t)BL_ERR_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // the partner no longer touches this CTA's memory
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

template <int kMode, typename TY>
cudaError_t launch(const GemmArgs& a, cudaStream_t s) {
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap map;
  const cuuint32_t box_m = (cuuint32_t)(a.M < kBM ? a.M : kBM);
  const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
  const cuuint64_t strides[1] = {(cuuint64_t)a.K};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, box_m};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(a.x_q), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  auto kern = gemm_tc2_kernel<kMode, TY>;
  int dev = 0, sms = 148;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  // Per instantiation and device ordinal: 0 until the kernel's shared-memory size has been raised
  // on that device, then the number of clusters that can be resident at once (the persistent grid
  // never has more).  Devices beyond the table are set up on every call.
  constexpr int kMaxDevices = 64;
  static std::atomic<int> resident[kMaxDevices];
  int cap = dev < kMaxDevices ? resident[dev].load(std::memory_order_acquire) : 0;
  const int64_t tiles = ((a.M + kPairM - 1) / kPairM) * ((a.N + kBN - 1) / kBN);
  if (tiles >= (int64_t)1 << 31) return cudaErrorInvalidValue;
  int64_t clusters = (sms < kMaxCtas ? sms : kMaxCtas) / 2;
  if (cap == 0) {
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes)) != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) { (void)cudaGetLastError(); n = (int)clusters; }
    cap = n;
    if (dev < kMaxDevices) resident[dev].store(cap, std::memory_order_release);
  }
  if (cap < clusters) clusters = cap;
  if (tiles < clusters) clusters = tiles;
  return launch_pdl(kern, (unsigned)(2 * clusters), kThreads, kSmemBytes, s, map, a, (int)(box_m * kBK));
}

}  // namespace

bool gemm_tc_supported(int64_t M, int64_t K, int64_t N, int G) {
  return M >= 1 && N >= 1 && G >= 1 && K % kBK == 0 && (K / G) % kBK == 0 && K / kBK < (1 << 24);
}

// Per-CTA fp32 running sums of the grouped epilogue: two CTAs per 256 x 256 tile.
size_t gemm_tc_scratch_bytes(int64_t M, int64_t N, int G) {
  if (G <= 1 || M <= 0 || N <= 0) return 0;
  int64_t ctas = 2 * ((M + kPairM - 1) / kPairM) * ((N + kBN - 1) / kBN);
  if (ctas > kMaxCtas) ctas = kMaxCtas;
  return (size_t)ctas * kScratchPerCta;
}

cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s) {
  if (a.y == nullptr) return launch<0, float>(a, s);
  const bool ext = a.beta_rows > 0 || a.relu || a.residual != nullptr || (a.ld_y > 0 && a.ld_y != a.N);
  switch (a.yt) {
    case BL_F32: return ext ? launch<2, float>(a, s) : launch<1, float>(a, s);
    case BL_F16: return ext ? launch<2, __half>(a, s) : launch<1, __half>(a, s);
    case BL_BF16: return ext ? launch<2, __nv_bfloat16>(a, s) : launch<1, __nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl
