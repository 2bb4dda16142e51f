// Dispatch and host-side helpers of the tensor-core GEMM (the kernel itself is in gemm_tc2.cu).
#include "tc_common.cuh"

namespace bl {

namespace {
constexpr int kBM = 128, kBN = 256, kBK = 128;     // tokens per CTA, features per tile, weights per stage
constexpr int kMaxCtas = 160;                      // the scratch is sized for at most this many CTAs
constexpr size_t kScratchPerCta = (size_t)kBM * kBN * sizeof(float);
}  // namespace

bool gemm_tc_supported(int64_t M, int64_t K, int64_t N, int G) {
  return M >= 1 && N >= 1 && G >= 1 && K % kBK == 0 && (K / G) % kBK == 0 && K / kBK < (1 << 24);
}

// Per-CTA fp32 running sums of the grouped epilogue: two CTAs per 256 x 256 tile.
size_t gemm_tc_scratch_bytes(int64_t M, int64_t N, int G) {
  if (G <= 1 || M <= 0 || N <= 0) return 0;
  int64_t ctas = 2 * ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + kBN - 1) / kBN);
  if (ctas > kMaxCtas) ctas = kMaxCtas;
  return (size_t)ctas * kScratchPerCta;
}

cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s) { return launch_gemm_tc2(a, s); }

}  // namespace bl
