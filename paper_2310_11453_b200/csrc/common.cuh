// Shared device helpers and the internal launch interface of the BitLinear CUDA library.
// sm_100a only.  Nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/bitlinear.h"

namespace bl {

// Test hook behind bitlinear_debug_wait_limit (defined in api.cu, read by the launchers when a
// call is made): cap on the polls of the bounded device-side waits (negative: built-in limits),
// and whether the cooperative LN+quant kernel waits for a tag that nobody publishes.
extern std::atomic<long long> g_debug_wait_polls;
extern std::atomic<int> g_debug_meet_skew;

// Programmatic dependent launch.  A kernel launched through launch_pdl() may be scheduled while
// the kernel before it on the stream is still running: it calls pdl_wait() before its first
// access to global memory (after set-up that touches only its own shared memory), which blocks
// until everything earlier on the stream has completed and is visible.  pdl_launch_dependents()
// lets the kernel after this one be scheduled early in the same way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t s,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

constexpr int kQb = 128;             // Q_b = 2^(b-1), b = 8
constexpr int kCodeMax = kQb - 1;    // Clip bound with the paper's eps taken as one code
constexpr float kInvQb = 1.0f / 128.0f;

// ---- element loads: 8 consecutive elements of a 16-byte aligned row as floats ------------
template <typename T> struct Elem;
template <> struct Elem<float> {
  static __device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
  static __device__ __forceinline__ float to_out(float f) { return f; }
};
template <> struct Elem<__half> {
  static __device__ __forceinline__ void load8(const __half* p, float (&v)[8]) {
    uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
    const __half2* h = reinterpret_cast<const __half2*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 f = __half22float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
  }
  static __device__ __forceinline__ __half to_out(float f) { return __float2half_rn(f); }
};
template <> struct Elem<__nv_bfloat16> {
  static __device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ __nv_bfloat16 to_out(float f) { return __float2bfloat16_rn(f); }
};

// ---- order-preserving float <-> uint encoding for atomic min/max ---------------------------
__device__ __forceinline__ uint32_t enc_ordered(float f) {
  uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float dec_ordered(uint32_t e) {
  uint32_t b = (e & 0x80000000u) ? (e & 0x7FFFFFFFu) : ~e;
  return __uint_as_float(b);
}

// ---- warp / block reductions (fixed order, deterministic) ---------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// ---- Quant of one normalised value, Eq. 4-6 (round-half-to-even, then clip) ----------------
// scale = Q_b / gamma (0 when gamma == 0); shift = eta (0 for absmax); lo = -127 or 0.
__device__ __forceinline__ int quant_code(float xhat, float shift, float scale, int lo) {
  int c = __float2int_rn((xhat - shift) * scale);
  return max(lo, min(kCodeMax, c));
}

// ---- Eq. 11 rescale of one group's integer sum (shared by every matmul kernel) --------------
// acc * beta_g * gamma / Q_b, plus eta * beta_g * rowsum when the eta shift is undone.
__device__ __forceinline__ float dequant_term(int acc, float beta_g, float gamma, float eta,
                                              int rowsum, bool correct) {
  float v = (float)acc * (beta_g * gamma * kInvQb);
  if (correct) v += eta * beta_g * (float)rowsum;
  return v;
}

__device__ __forceinline__ float in_cast(float v) { return v; }
__device__ __forceinline__ float in_cast(__half v) { return __half2float(v); }
__device__ __forceinline__ float in_cast(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T out_cast(float f);
template <> __device__ __forceinline__ float out_cast<float>(float f) { return f; }
template <> __device__ __forceinline__ __half out_cast<__half>(float f) { return __float2half_rn(f); }
template <> __device__ __forceinline__ __nv_bfloat16 out_cast<__nv_bfloat16>(float f) { return __float2bfloat16_rn(f); }

// ---- internal launchers (defined one per .cu file) -----------------------------------------
struct PackArgs {
  const void* W; bl_dtype wt; int64_t N, K; int G; bl_layout layout; const float* alpha_in;
  uint8_t* W_packed; float* alpha; float* beta; int32_t* rowsum; void* ws;
};
size_t pack_ws_bytes(int G);
cudaError_t launch_binarize_pack(const PackArgs& a, cudaStream_t s);

struct QuantArgs {
  const void* x; bl_dtype xt; int64_t M, K; int G; bl_quant_mode mode; bl_gran gran; float ln_eps;
  int8_t* x_q; float* gamma; float* eta; void* ws;
  uint32_t* status = nullptr;                      // word for a device-side timeout.  nullptr: per-tensor
                                                   // scope uses the first word of ws, per-token scope runs
                                                   // without bounded waits (per-lane copies)
  int keep_status = 0;                             // an earlier kernel of the call already cleared the word
};
size_t quant_ws_bytes(int64_t M, int G);
cudaError_t launch_quant_act(const QuantArgs& a, cudaStream_t s);

// Integer matmul, optionally with the Eq. 11 rescale fused.  When y != nullptr the kernel
// writes y (dtype yt); otherwise it writes acc [G,M,N].
struct GemmArgs {
  const int8_t* x_q; int64_t M, K, N; int G; const uint8_t* W_packed;
  int32_t* acc;                                    // int32 output, or nullptr
  void* y; bl_dtype yt;                            // dequantised output, or nullptr
  const float* beta; const float* gamma; const float* eta; bl_gran gran;
  const int32_t* rowsum; int eta_correction;
  // Epilogue options of the dequantising kernels (all zero: Eq. 11 as is, dense y).
  int64_t beta_rows;                               // output features per beta block (0: one block);
                                                   // beta is [N/beta_rows, G], rowsum stays [N, G]
  int relu;                                        // y = max(y, 0) before the residual
  const void* residual; int64_t ld_res;            // y += residual[m, n] (dtype yt, row stride ld_res)
  int64_t ld_y;                                    // row stride of y in elements (0: N)
  uint32_t* status;                                // device status word (tensor-core path)
  int keep_status;                                 // the kernel before this one already cleared it
  void* scratch;                                   // gemm_tc_scratch_bytes(G) bytes (tensor-core path)
};
cudaError_t launch_gemm_simple(const GemmArgs& a, cudaStream_t s);
cudaError_t launch_gemm_tc(const GemmArgs& a, cudaStream_t s);      // tcgen05, two SMs per tile (gemm_tc2.cu)
bool gemm_tc_supported(int64_t M, int64_t K, int64_t N, int G);
size_t gemm_tc_scratch_bytes(int64_t M, int64_t N, int G);   // host-only, no device query

struct GemvArgs {
  const void* x; bl_dtype xt; int64_t K, N; int G; bl_quant_mode mode; float ln_eps;
  int eta_correction; const uint8_t* W_packed; const float* beta; const int32_t* rowsum;
  void* y; bl_dtype yt;
  uint32_t* clear_status = nullptr;   // when set: a status word that the call's (first) kernel clears, in stream order
};
cudaError_t launch_gemv_decode(const GemvArgs& a, cudaStream_t s);
cudaError_t gemv_decode_take_fallbacks(unsigned int* out);   // warps that read weights from global memory after a wait ran out
// The same for M tokens (x [M,K], y [M,N]) sharing one pass over the weights per 8 tokens.
cudaError_t launch_gemv_batch(const GemvArgs& a, int64_t M, cudaStream_t s);
bool gemv_batch_supported(int64_t M, int64_t K, int64_t N, int G);
cudaError_t launch_gemv_batch_pre(const GemvArgs& g, int64_t M, const int8_t* codes, const float* gamma, const int* csum,
                                  cudaStream_t s);   // the same kernel on tokens quantised earlier on the stream
// The same with a workspace: tokens quantised once by a kernel of their own, the product on the
// tcgen05 tensor cores, 16 tokens per pass over the weights (gemv_tc.cu).
cudaError_t launch_gemv_tc(const GemvArgs& a, int64_t M, void* ws, cudaStream_t s);
bool gemv_tc_supported(int64_t M, int64_t K, int64_t N, int G, int eta_correction);
size_t gemv_tc_ws_bytes(int64_t M, int64_t K);

// Decoder-block glue (fp16): the causal attention core.
cudaError_t launch_attention_causal(const void* q, const void* k, const void* v, void* o, int batch, int S,
                                    int heads, int64_t ld, int64_t ld_o, cudaStream_t s);

// Host-side layout maps (also exported through bitlinear_layout_index).
int64_t prefill_bytes(int64_t N, int64_t K);
void prefill_index(int64_t K, int64_t n, int64_t k, int64_t* byte_off, int* bit);
void decode_index(int64_t K, int64_t n, int64_t k, int64_t* byte_off, int* bit);

}  // namespace bl
