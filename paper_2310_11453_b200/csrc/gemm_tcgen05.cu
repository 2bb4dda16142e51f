// Step 4 of BitLinear on the 5th-generation tensor cores: acc = W~ x~ (Eq. 7) as tcgen05
// kind::i8 MMAs (s8 x s8 -> s32 in tensor memory), with the Eq. 11 rescale fused into the
// epilogue.  The weights stay 1 bit per weight all the way into the SM: each k-step the CTA
// expands a 256 x 128 tile of sign bits into +-1 bytes in shared memory, directly in the
// K-major 128-byte-swizzled layout the MMA's shared-memory descriptor describes, while TMA
// brings the matching 128 x 128 tile of int8 codes.
//
// One persistent CTA per SM, 16 warps, roles fixed per warp:
//   warp 0      TMA producer: codes tile (A operand) of every stage
//   warp 1      MMA issuer (one thread): 4 MMAs of 128x256x32 per stage, tcgen05.commit
//   warp 2      owns the tensor-memory allocation (512 columns = two 128x256 accumulators)
//   warps 4-7   epilogue: tcgen05.ld one accumulator while the MMAs fill the other
//   warps 8-23  weight expanders in two groups of 8 warps that take alternate stages: thread u
//               of a group owns row u of the 256-row B tile; its 16 bytes of bits come straight
//               from global memory (prefetched two owned stages ahead in registers)
// Stage hand-over uses mbarriers: full_a (TMA bytes), full_b (8 expander warps), empty
// (tcgen05.commit), and a full/empty pair per accumulator.  Writes of the expanders are
// generic-proxy stores, so each thread issues fence.proxy.async before its warp arrives.
//
// Every wait is bounded: when a limit runs out the CTA raises a shared abort flag, records
// BL_ERR_TIMEOUT in the status word, lets every role fall through to the common exit and frees
// its tensor memory.  No cluster launch and no multicast loads are used.
//
// PREFILL weight layout read here: blocks of 128 rows x 128 weights, 2048 contiguous bytes,
// row r of the block at byte 16 r; inside each 32-weight word weight q sits at bit
// q/4 + 8*(q%4), so (word >> j) & 0x01010101 holds weights 4j..4j+3 as 0/1 bytes.
//
// Groups (Eq. 13-14) split K, so with G > 1 the int32 accumulator is drained once per group:
// the epilogue keeps the fp32 running sum of a tile in a per-CTA scratch area (L2-resident,
// touched only by the thread that owns the element) and writes y after the last group.
#include <cstdlib>

#include "tc_common.cuh"

namespace bl {

namespace {

using namespace tc;

constexpr int kBM = 128;                 // tokens per tile (MMA M, tensor-memory lanes)
constexpr int kBN = 256;                 // output features per tile (MMA N)
constexpr int kBK = 128;                 // weights per stage (one 128-byte swizzle atom)
constexpr int kStages = 4;
constexpr int kThreads = 768;
constexpr int kExpandWarp0 = 8;          // first expander warp
constexpr int kEpiWarp0 = 4;             // first epilogue warp
constexpr int kABytes = kBM * kBK;       // 16 KB
constexpr int kBBytes = kBN * kBK;       // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTmemCols = 512;
constexpr int kMaxCtas = 160;            // scratch is sized for this many CTAs
constexpr size_t kScratchPerCta = (size_t)kBM * kBN * sizeof(float);

struct SharedCtl {
  unsigned long long full_a[kStages], full_b[kStages], empty[kStages];
  unsigned long long tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 + sizeof(SharedCtl) + 64;

// kind::i8 instruction descriptor: s32 accumulate, s8 x s8, both operands K-major, M x N.
constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) |
                            ((uint32_t)(kBM >> 4) << 24);


struct TileIter {            // tiles of this CTA, in the order every role walks them
  uint32_t t, tiles, m_tiles, stride;
  __device__ TileIter(uint32_t tiles_, uint32_t m_tiles_)
      : t(blockIdx.x), tiles(tiles_), m_tiles(m_tiles_), stride(gridDim.x) {}
  __device__ bool valid() const { return t < tiles; }
  __device__ void next() { t += stride; }
  __device__ uint32_t m_tile() const { return t % m_tiles; }
  __device__ uint32_t n_tile() const { return t / m_tiles; }
};


// kMode 0: write int32 accumulators acc[g,m,n].  kMode 1: write y (Eq. 11).
template <int kMode, typename TY>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_x, GemmArgs a, int tx_bytes) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + (size_t)kStages * kStageBytes);
  volatile int* abort_flag = &ctl->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const uint32_t m_tiles = (uint32_t)((a.M + kBM - 1) / kBM), n_tiles = (uint32_t)((a.N + kBN - 1) / kBN);
  const uint32_t tiles = m_tiles * n_tiles;
  const int k_blocks = (int)(a.K / kBK);             // stages per tile (all groups)
  const int kb_per_group = k_blocks / a.G;
  const int64_t w_blocks_n = (a.N + 127) / 128;      // 128-row blocks present in W_packed
  const int64_t w_blocks_k = (a.K + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&ctl->full_a[s]), 1);
      mbar_init(smem_u32(&ctl->full_b[s]), kBN / 32);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 4);
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (codes)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      uint32_t issued = 0;
      bool ok = true;
      for (TileIter it(tiles, m_tiles); ok && it.valid(); it.next()) {
        const int m0 = (int)(it.m_tile() * kBM);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t bar = smem_u32(&ctl->full_a[stage]);
          mbar_arrive_expect_tx(bar, (uint32_t)tx_bytes);
          tma_load_2d(smem_u32(smem + (size_t)stage * kStageBytes), &map_x, kb * kBK, m0, bar);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      // Copies still in flight must land before the CTA may exit: wait (bounded) for the last
      // copy issued into each stage.  On the normal path these phases completed long ago.
      const uint32_t pending = issued < (uint32_t)kStages ? issued : (uint32_t)kStages;
      for (uint32_t i = 0; i < pending; ++i) {
        if (stage == 0) { stage = kStages; phase ^= 1u; }
        --stage;
        (void)mbar_wait(smem_u32(&ctl->full_a[stage]), phase, abort_flag);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      uint32_t pass = 0;
      bool ok = true;
      for (TileIter it(tiles, m_tiles); ok && it.valid(); it.next()) {
        for (int g = 0; ok && g < a.G; ++g, ++pass) {
          const uint32_t buf = pass & 1u, acc_phase = (pass >> 1) & 1u;
          if (!mbar_wait(smem_u32(&ctl->tmem_empty[buf]), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * (uint32_t)kBN;
          for (int kb = 0; kb < kb_per_group; ++kb) {
            if (!mbar_wait(smem_u32(&ctl->full_a[stage]), phase, abort_flag) ||
                !mbar_wait(smem_u32(&ctl->full_b[stage]), phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = smem_u32(smem + (size_t)stage * kStageBytes);
            const uint64_t adesc = smem_desc_sw128(a_addr);
            const uint64_t bdesc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
            for (int j = 0; j < kBK / 32; ++j)
              mma_i8(d_tmem, adesc + (uint64_t)(2 * j), bdesc + (uint64_t)(2 * j), kIdesc,
                     (kb > 0 || j > 0) ? 1u : 0u);
            mma_commit(smem_u32(&ctl->empty[stage]));
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) mma_commit(smem_u32(&ctl->tmem_full[buf]));
        }
      }
    }
  } else if (warp >= kExpandWarp0) {
    // ---------------------------------------------------------------- weight expanders
    // Two groups of 8 warps take alternate stages, so one group's stores, proxy fence and
    // barrier round trip overlap the other group's arithmetic.
    const int eg = (warp - kExpandWarp0) >> 3;                       // group 0 or 1
    const int u = (threadIdx.x - kExpandWarp0 * 32) & (kBN - 1);     // row of the B tile, 0..255
    // byte offset of chunk position 0 of row u inside a stage, pre-xored with the row's swizzle
    const uint32_t row_base = smem_u32(smem) + (uint32_t)kABytes + (uint32_t)u * 128u + ((uint32_t)(u & 7) << 4);
    int stage = eg; uint32_t phase = 0;
    // flat walk over (tile, k-block); this group owns every second step.  The 16 bytes of
    // bits of the next two owned steps are prefetched in registers.
    TileIter pf_it(tiles, m_tiles);
    int pf_kb = eg;
    const uint8_t* pf_src = nullptr;                                 // row u of the tile's first k-block
    auto seek = [&]() {
      while (pf_it.valid() && pf_kb >= k_blocks) { pf_kb -= k_blocks; pf_it.next(); }
      pf_src = nullptr;
      if (pf_it.valid()) {
        const int64_t nb = (int64_t)pf_it.n_tile() * 2 + (u >> 7);
        if (nb < w_blocks_n) pf_src = a.W_packed + nb * w_blocks_k * 2048 + (u & 127) * 16;
      }
    };
    seek();
    auto fetch = [&]() -> uint4 {
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (pf_it.valid()) {
        if (pf_src) v = __ldg(reinterpret_cast<const uint4*>(pf_src + (size_t)pf_kb * 2048));
        pf_kb += 2;
        if (pf_kb >= k_blocks) seek();
      }
      return v;
    };
    uint4 b0 = fetch(), b1 = fetch();
    // number of steps this group owns: ceil((my_tiles * k_blocks - eg) / 2)
    const uint32_t my_tiles = (tiles > blockIdx.x) ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    const uint64_t flat = (uint64_t)my_tiles * (uint64_t)k_blocks;
    const uint64_t owned = flat > (uint64_t)eg ? (flat - eg + 1) / 2 : 0;
    for (uint64_t i = 0; i < owned; ++i) {
      const uint4 cur = b0;
      b0 = b1;
      b1 = fetch();
      bool got = true;
      if (lane == 0) got = mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag);
      got = __shfl_sync(0xFFFFFFFFu, got, 0);
      __syncwarp();
      if (!got) break;
      const uint32_t dst = row_base + (uint32_t)stage * (uint32_t)kStageBytes;
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
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctl->full_b[stage]));
      stage += 2;
      if (stage >= kStages) { stage -= kStages; phase ^= 1u; }
    }
  } else if (warp >= kEpiWarp0 && warp < kEpiWarp0 + 4) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                                  // lane quarter this warp may read
    const int row = q * 32 + lane;
    uint32_t pass = 0;
    bool ok = true;
    float* run = reinterpret_cast<float*>(reinterpret_cast<char*>(a.scratch) + (size_t)blockIdx.x * kScratchPerCta);
    const bool correct = (kMode == 1) && a.eta_correction != 0;
    for (TileIter it(tiles, m_tiles); ok && it.valid(); it.next()) {
      const int64_t m = (int64_t)it.m_tile() * kBM + row;
      const int64_t n_base = (int64_t)it.n_tile() * kBN;
      const bool m_ok = m < a.M;
      for (int g = 0; g < a.G; ++g, ++pass) {
        const uint32_t buf = pass & 1u, acc_phase = (pass >> 1) & 1u;
        bool got = mbar_wait(smem_u32(&ctl->tmem_full[buf]), acc_phase, abort_flag);
        got = __all_sync(0xFFFFFFFFu, got);
        if (!got) { ok = false; break; }
        tc_fence_after();
        float scale = 0.f, eta_beta = 0.f;
        if (kMode == 1 && m_ok) {
          const int64_t sc = (a.gran == BL_PER_TOKEN) ? m * a.G + g : g;
          const float beta_g = a.beta[g];
          scale = beta_g * a.gamma[sc] * kInvQb;
          if (correct) eta_beta = a.eta[sc] * beta_g;
        }
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)kBN;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + (uint32_t)(c * 32), r);
          const int64_t n0 = n_base + c * 32;
          if (n0 >= a.N) continue;                           // uniform across the warp
          if (kMode == 0) {
            if (m_ok) {
              int32_t* dst = a.acc + ((int64_t)g * a.M + m) * a.N + n0;
              if (n0 + 32 <= a.N && (a.N & 3) == 0) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  *reinterpret_cast<uint4*>(dst + 4 * i) = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
              } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) if (n0 + i < a.N) dst[i] = (int32_t)r[i];
              }
            }
          } else {
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
              TY* dst = reinterpret_cast<TY*>(a.y) + m * a.N + n0;
              const bool vec_ok = (n0 + 32 <= a.N) && ((a.N * sizeof(TY)) % 16 == 0);
              store_row32<TY>(dst, v, n0, a.N, vec_ok);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
      }
    }
  }

  // ---------------------------------------------------------------- common exit
  if (*abort_flag && threadIdx.x == 0) atomicExch(a.status, (uint32_t)BL_ERR_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
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
  static bool attr_set[2][3] = {};
  auto kern = gemm_tc_kernel<kMode, TY>;
  const int ti = kMode == 0 ? 0 : (int)a.yt;
  if (!attr_set[kMode][ti]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[kMode][ti] = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t tiles = ((a.M + kBM - 1) / kBM) * ((a.N + kBN - 1) / kBN);
  if (tiles >= (int64_t)1 << 31) return cudaErrorInvalidValue;
  int64_t grid = sms < kMaxCtas ? sms : kMaxCtas;
  if (tiles < grid) grid = tiles;
  kern<<<(unsigned)grid, kThreads, kSmemBytes, s>>>(map, a, (int)(box_m * kBK));
  return cudaGetLastError();
}

}  // namespace

bool gemm_tc_supported(int64_t M, int64_t K, int64_t N, int G) {
  return M >= 1 && N >= 1 && G >= 1 && K % kBK == 0 && (K / G) % kBK == 0 && K / kBK < (1 << 24);
}

size_t gemm_tc_scratch_bytes(int64_t M, int64_t N, int G) {
  if (G <= 1 || M <= 0 || N <= 0) return 0;
  // enough for either kernel: 128-token tiles, or pairs of CTAs on 256-token tiles
  int64_t ctas = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
  const int64_t pair_ctas = 2 * ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + kBN - 1) / kBN);
  if (pair_ctas > ctas) ctas = pair_ctas;
  if (ctas > kMaxCtas) ctas = kMaxCtas;
  return (size_t)ctas * kScratchPerCta;
}

cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s) {
  static const bool pair = [] { const char* e = getenv("BL_GEMM_PAIR"); return e && e[0] == '1'; }();
  if (pair) return launch_gemm_tc2(a, s);
  if (a.y == nullptr) return launch<0, float>(a, s);
  switch (a.yt) {
    case BL_F32: return launch<1, float>(a, s);
    case BL_F16: return launch<1, __half>(a, s);
    case BL_BF16: return launch<1, __nv_bfloat16>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bl
