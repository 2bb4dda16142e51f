// extern "C" entry points: argument validation on the host, workspace carving, launches.
// Nothing here allocates device memory or synchronises (bitlinear_ws_status excepted).
#include "common.cuh"

namespace bl {
std::atomic<long long> g_debug_wait_polls{-1};
std::atomic<int> g_debug_meet_skew{0};
}  // namespace bl

namespace {

using namespace bl;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round256(size_t v) { return (v + 255) & ~size_t(255); }
inline bool valid_dtype(int t) { return t == BL_F32 || t == BL_F16 || t == BL_BF16; }

// Common shape rules: sizes positive, 1 <= G <= BL_MAX_GROUPS, K % (8 G) == 0.
inline bl_status check_kg(int64_t K, int G) {
  if (K <= 0 || G < 1) return BL_ERR_SHAPE;
  if (G > BL_MAX_GROUPS) return BL_ERR_UNSUPPORTED;
  if (K % (8 * (int64_t)G) != 0) return BL_ERR_SHAPE;
  return BL_OK;
}

constexpr size_t kStatusBytes = 256;   // status word lives at the start of a GEMM workspace

// A GEMM workspace is the status word followed by the tensor-core kernel's scratch.
size_t gemm_ws_total(int64_t M, int64_t N, int G) {
  return kStatusBytes + round256(gemm_tc_scratch_bytes(M, N, G));
}

struct BlockWs {                       // carving of the BL_OP_BLOCK_FORWARD workspace
  size_t gemm, codes, gamma, eta, total;
};
BlockWs carve_block(int64_t T, int64_t d, int64_t ffn) {
  BlockWs w;
  size_t off = 0;
  const int64_t widest = ffn > 3 * d ? ffn : 3 * d;       // Q, K, V may run as one [3d, d] GEMM
  w.gemm = off;  off += gemm_ws_total(T, widest, 1);
  w.codes = off; off += round256((size_t)T * (size_t)widest);
  w.gamma = off; off += round256((size_t)T * sizeof(float));
  w.eta = off;   off += round256((size_t)T * sizeof(float));
  w.total = off;
  return w;
}

struct ForwardWs {                     // carving of the BL_OP_FORWARD workspace
  size_t status, codes, gamma, eta, quant, total;
};
ForwardWs carve_forward(int64_t M, int64_t N, int64_t K, int G) {
  ForwardWs w;
  size_t off = 0;
  w.status = off; off += gemm_ws_total(M, N, G);
  w.codes = off;  off += round256((size_t)M * (size_t)K);
  w.gamma = off;  off += round256((size_t)M * (size_t)G * sizeof(float));
  w.eta = off;    off += round256((size_t)M * (size_t)G * sizeof(float));
  w.quant = off;  off += round256(quant_ws_bytes(M, G));
  w.total = off;
  return w;
}

struct LatentWs {                      // carving of the BL_OP_FORWARD_LATENT workspace
  size_t pack, packed, alpha, beta, rowsum, forward, total;
  bl_layout layout;
};
LatentWs carve_latent(int64_t M, int64_t N, int64_t K, int G) {
  LatentWs w;
  w.layout = gemm_tc_supported(M, K, N, G) ? BL_LAYOUT_PREFILL : BL_LAYOUT_CANONICAL;
  size_t off = 0;
  w.pack = off;    off += round256(pack_ws_bytes(G));
  w.packed = off;  off += round256(w.layout == BL_LAYOUT_PREFILL ? (size_t)prefill_bytes(N, K) : (size_t)(N * (K / 8)));
  w.alpha = off;   off += round256((size_t)G * sizeof(float));
  w.beta = off;    off += round256((size_t)G * sizeof(float));
  w.rowsum = off;  off += round256((size_t)N * (size_t)G * sizeof(int32_t));
  w.forward = off; off += carve_forward(M, N, K, G).total;
  w.total = off;
  return w;
}

bl_status check_layout_for_gemm(bl_layout layout, int64_t M, int64_t K, int64_t N, int G) {
  if (layout == BL_LAYOUT_CANONICAL) return BL_OK;
  if (layout == BL_LAYOUT_PREFILL) return gemm_tc_supported(M, K, N, G) ? BL_OK : BL_ERR_SHAPE;
  return BL_ERR_UNSUPPORTED;
}

}  // namespace

extern "C" {

const char* bitlinear_status_string(bl_status st) {
  switch (st) {
    case BL_OK: return "ok";
    case BL_ERR_NULL: return "null pointer";
    case BL_ERR_SHAPE: return "invalid shape";
    case BL_ERR_ALIGN: return "pointer not 16-byte aligned";
    case BL_ERR_UNSUPPORTED: return "unsupported option";
    case BL_ERR_WORKSPACE: return "workspace missing or too small";
    case BL_ERR_CUDA: return "CUDA runtime error";
    case BL_ERR_TIMEOUT: return "device-side wait timed out";
    case BL_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
  }
  return "unknown status";
}

size_t bitlinear_workspace_bytes(bl_op op, int64_t M, int64_t N, int64_t K, int G) {
  if (check_kg(K, G) != BL_OK) return 0;
  switch (op) {
    case BL_OP_BINARIZE_PACK: return round256(pack_ws_bytes(G));
    case BL_OP_QUANT_ACT: return M > 0 ? round256(quant_ws_bytes(M, G)) : 0;
    case BL_OP_FORWARD: return (M > 0 && N > 0) ? carve_forward(M, N, K, G).total : 0;
    case BL_OP_MATMUL_I32:
    case BL_OP_MATMUL_DEQUANT: return (M > 0 && N > 0) ? gemm_ws_total(M, N, G) : 0;
    case BL_OP_BLOCK_FORWARD: return (M > 0 && N > 0) ? carve_block(M, K, N).total : 0;
    case BL_OP_FORWARD_LATENT: return (M > 0 && N > 0) ? carve_latent(M, N, K, G).total : 0;
    case BL_OP_GEMV_DECODE_BATCH: return M > 0 ? round256(gemv_tc_ws_bytes(M, K)) : 0;
  }
  return 0;
}

size_t bitlinear_packed_bytes(bl_layout layout, int64_t N, int64_t K) {
  if (N <= 0 || K <= 0 || K % 8 != 0) return 0;
  switch (layout) {
    case BL_LAYOUT_CANONICAL: return (size_t)(N * (K / 8));
    case BL_LAYOUT_PREFILL: return K % 16 == 0 ? (size_t)prefill_bytes(N, K) : 0;
    case BL_LAYOUT_DECODE: return (K % 256 == 0 && N % 16 == 0) ? (size_t)(N * (K / 8)) : 0;
  }
  return 0;
}

bl_status bitlinear_layout_index(bl_layout layout, int64_t N, int64_t K, int64_t n, int64_t k,
                                 int64_t* byte_offset, int* bit) {
  if (!byte_offset || !bit) return BL_ERR_NULL;
  if (bitlinear_packed_bytes(layout, N, K) == 0 || n < 0 || n >= N || k < 0 || k >= K)
    return BL_ERR_SHAPE;
  switch (layout) {
    case BL_LAYOUT_CANONICAL: *byte_offset = n * (K / 8) + k / 8; *bit = (int)(k % 8); break;
    case BL_LAYOUT_PREFILL: prefill_index(K, n, k, byte_offset, bit); break;
    case BL_LAYOUT_DECODE: decode_index(K, n, k, byte_offset, bit); break;
  }
  return BL_OK;
}

bl_status bitlinear_binarize_pack(const void* W, bl_dtype wt, int64_t N, int64_t K, int G,
                                  bl_layout layout, const float* alpha_in, uint8_t* W_packed,
                                  float* alpha, float* beta, int32_t* rowsum, void* ws,
                                  size_t ws_bytes, void* stream) {
  if (!W || !W_packed || !alpha || !beta) return BL_ERR_NULL;
  if (N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (!valid_dtype(wt)) return BL_ERR_UNSUPPORTED;
  if (layout != BL_LAYOUT_CANONICAL && layout != BL_LAYOUT_PREFILL && layout != BL_LAYOUT_DECODE)
    return BL_ERR_UNSUPPORTED;
  if (bitlinear_packed_bytes(layout, N, K) == 0) return BL_ERR_SHAPE;
  if (layout == BL_LAYOUT_PREFILL && (K / G) % 128 != 0) return BL_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(W_packed)) return BL_ERR_ALIGN;
  if (!ws || ws_bytes < bitlinear_workspace_bytes(BL_OP_BINARIZE_PACK, 1, N, K, G)) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  PackArgs a{W, wt, N, K, G, layout, alpha_in, W_packed, alpha, beta, rowsum, ws};
  return launch_binarize_pack(a, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_quant_act(const void* x, bl_dtype xt, int64_t M, int64_t K, int G, int b,
                              bl_quant_mode mode, bl_gran gran, float ln_eps, int8_t* x_q,
                              float* gamma, float* eta, void* ws, size_t ws_bytes, void* stream) {
  if (!x || !x_q || !gamma) return BL_ERR_NULL;
  if (mode == BL_ETA && !eta) return BL_ERR_NULL;
  if (M <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (b != 8 || !valid_dtype(xt)) return BL_ERR_UNSUPPORTED;
  if (mode != BL_ABSMAX && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (gran != BL_PER_TENSOR && gran != BL_PER_TOKEN) return BL_ERR_UNSUPPORTED;
  if ((K / G) * sizeof(float) > 200 * 1024) return BL_ERR_SHAPE;   // one segment must fit in shared memory
  if (M * (int64_t)G > 0x7FFFFFFF) return BL_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(x_q)) return BL_ERR_ALIGN;
  if (gran == BL_PER_TENSOR) {
    if (!ws || ws_bytes < bitlinear_workspace_bytes(BL_OP_QUANT_ACT, M, 1, K, G)) return BL_ERR_WORKSPACE;
    if (!aligned16(ws)) return BL_ERR_ALIGN;
  }
  QuantArgs a{x, xt, M, K, G, mode, gran, ln_eps, x_q, gamma, eta, ws};
  // per-token scope needs no workspace; given one, its first word serves as the status word and the
  // kernel may then use copies whose wait is bounded and reported there
  if (gran == BL_PER_TOKEN && ws && ws_bytes >= kStatusBytes && aligned16(ws)) a.status = reinterpret_cast<uint32_t*>(ws);
  return launch_quant_act(a, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_matmul_i32(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                               const uint8_t* W_packed, bl_layout layout, int32_t* acc, void* ws,
                               size_t ws_bytes, void* stream) {
  if (!x_q || !W_packed || !acc) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  st = check_layout_for_gemm(layout, M, K, N, G);
  if (st != BL_OK) return st;
  if (!aligned16(x_q) || !aligned16(W_packed) || !aligned16(acc)) return BL_ERR_ALIGN;
  if (!ws || ws_bytes < gemm_ws_total(M, N, G)) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  cudaStream_t s = (cudaStream_t)stream;
  // the tensor-core kernel clears the status word itself; the CUDA-core kernel never writes it
  if (layout != BL_LAYOUT_PREFILL && cudaMemsetAsync(ws, 0, kStatusBytes, s) != cudaSuccess) return BL_ERR_CUDA;
  GemmArgs a{};
  a.x_q = x_q; a.M = M; a.K = K; a.N = N; a.G = G; a.W_packed = W_packed; a.acc = acc;
  a.y = nullptr; a.gran = BL_PER_TENSOR; a.status = reinterpret_cast<uint32_t*>(ws);
  a.scratch = reinterpret_cast<char*>(ws) + kStatusBytes;
  cudaError_t e = (layout == BL_LAYOUT_PREFILL) ? launch_gemm_tc(a, s) : launch_gemm_simple(a, s);
  return e == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_matmul_dequant_ex(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                                      bl_gran gran, const float* gamma, const float* eta,
                                      int eta_correction, const uint8_t* W_packed, bl_layout layout,
                                      const float* beta, const int32_t* rowsum, const bl_epilogue* epi,
                                      void* y, bl_dtype yt, void* ws, size_t ws_bytes, void* stream) {
  if (!x_q || !W_packed || !beta || !gamma || !y) return BL_ERR_NULL;
  if (eta_correction && (!rowsum || !eta)) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (!valid_dtype(yt)) return BL_ERR_UNSUPPORTED;
  if (gran != BL_PER_TENSOR && gran != BL_PER_TOKEN) return BL_ERR_UNSUPPORTED;
  st = check_layout_for_gemm(layout, M, K, N, G);
  if (st != BL_OK) return st;
  bl_epilogue o{};
  if (epi) o = *epi;
  if (o.beta_rows < 0 || (o.beta_rows > 0 && (N % o.beta_rows != 0 || o.beta_rows % 32 != 0))) return BL_ERR_SHAPE;
  if (o.ld_y < 0 || (o.ld_y > 0 && o.ld_y < N)) return BL_ERR_SHAPE;
  if (o.residual && o.ld_res < N) return BL_ERR_SHAPE;
  if (!aligned16(x_q) || !aligned16(W_packed) || !aligned16(y) || !aligned16(o.residual)) return BL_ERR_ALIGN;
  if (!ws || ws_bytes < gemm_ws_total(M, N, G)) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  cudaStream_t s = (cudaStream_t)stream;
  // the tensor-core kernel clears the status word itself; the CUDA-core kernel never writes it
  if (layout != BL_LAYOUT_PREFILL && cudaMemsetAsync(ws, 0, kStatusBytes, s) != cudaSuccess) return BL_ERR_CUDA;
  GemmArgs a{};
  a.x_q = x_q; a.M = M; a.K = K; a.N = N; a.G = G; a.W_packed = W_packed; a.acc = nullptr;
  a.y = y; a.yt = yt; a.beta = beta; a.gamma = gamma; a.eta = eta; a.gran = gran;
  a.rowsum = rowsum; a.eta_correction = eta_correction ? 1 : 0;
  a.beta_rows = o.beta_rows; a.relu = o.relu ? 1 : 0; a.residual = o.residual; a.ld_res = o.ld_res; a.ld_y = o.ld_y;
  a.status = reinterpret_cast<uint32_t*>(ws);
  a.scratch = reinterpret_cast<char*>(ws) + kStatusBytes;
  cudaError_t e = (layout == BL_LAYOUT_PREFILL) ? launch_gemm_tc(a, s) : launch_gemm_simple(a, s);
  return e == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_matmul_dequant(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                                   bl_gran gran, const float* gamma, const float* eta,
                                   int eta_correction, const uint8_t* W_packed, bl_layout layout,
                                   const float* beta, const int32_t* rowsum, void* y, bl_dtype yt,
                                   void* ws, size_t ws_bytes, void* stream) {
  return bitlinear_matmul_dequant_ex(x_q, M, K, N, G, gran, gamma, eta, eta_correction, W_packed, layout, beta,
                                     rowsum, nullptr, y, yt, ws, ws_bytes, stream);
}

bl_status bitlinear_binarize_pack_nsplit(const void* W, bl_dtype wt, int64_t N, int64_t K, int G, int NB,
                                         bl_layout layout, const float* alpha_in, uint8_t* W_packed,
                                         float* alpha, float* beta, int32_t* rowsum, void* ws,
                                         size_t ws_bytes, void* stream) {
  if (NB <= 0 || N <= 0 || N % NB != 0) return BL_ERR_SHAPE;
  if (!valid_dtype(wt)) return BL_ERR_UNSUPPORTED;
  const int64_t rows = N / NB;
  if (layout == BL_LAYOUT_PREFILL && NB > 1 && rows % 128 != 0) return BL_ERR_SHAPE;
  const size_t block_bytes = bitlinear_packed_bytes(layout, rows, K);
  if (block_bytes == 0) return BL_ERR_SHAPE;
  const size_t esz = wt == BL_F32 ? 4 : 2;
  for (int j = 0; j < NB; ++j) {
    const bl_status st = bitlinear_binarize_pack(
        reinterpret_cast<const char*>(W) + (size_t)j * (size_t)rows * (size_t)K * esz, wt, rows, K, G, layout,
        alpha_in ? alpha_in + (size_t)j * G : nullptr, W_packed ? W_packed + (size_t)j * block_bytes : nullptr,
        alpha ? alpha + (size_t)j * G : nullptr, beta ? beta + (size_t)j * G : nullptr,
        rowsum ? rowsum + (size_t)j * (size_t)rows * G : nullptr, ws, ws_bytes, stream);
    if (st != BL_OK) return st;
  }
  return BL_OK;
}

bl_status bitlinear_forward(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                            int b, bl_quant_mode mode, bl_gran gran, float ln_eps,
                            int eta_correction, const uint8_t* W_packed, bl_layout layout,
                            const float* beta, const int32_t* rowsum, void* y, bl_dtype yt,
                            void* ws, size_t ws_bytes, void* stream) {
  if (!x || !W_packed || !beta || !y) return BL_ERR_NULL;
  if (eta_correction && !rowsum) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (b != 8 || !valid_dtype(xt) || !valid_dtype(yt)) return BL_ERR_UNSUPPORTED;
  if (mode != BL_ABSMAX && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (gran != BL_PER_TENSOR && gran != BL_PER_TOKEN) return BL_ERR_UNSUPPORTED;
  if (eta_correction && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  st = check_layout_for_gemm(layout, M, K, N, G);
  if (st != BL_OK) return st;
  if ((K / G) * sizeof(float) > 200 * 1024 || M * (int64_t)G > 0x7FFFFFFF) return BL_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(W_packed) || !aligned16(y)) return BL_ERR_ALIGN;
  const ForwardWs w = carve_forward(M, N, K, G);
  if (!ws || ws_bytes < w.total) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  char* base = reinterpret_cast<char*>(ws);
  cudaStream_t s = (cudaStream_t)stream;
  if (layout != BL_LAYOUT_PREFILL && cudaMemsetAsync(base + w.status, 0, kStatusBytes, s) != cudaSuccess)
    return BL_ERR_CUDA;
  int8_t* codes = reinterpret_cast<int8_t*>(base + w.codes);
  float* gamma = reinterpret_cast<float*>(base + w.gamma);
  float* eta = reinterpret_cast<float*>(base + w.eta);
  QuantArgs q{x, xt, M, K, G, mode, gran, ln_eps, codes, gamma, eta, base + w.quant};
  // One status word for the call: the quant kernels clear it (and may report a timeout of their
  // own), so the GEMM that follows must not clear it again.
  q.status = reinterpret_cast<uint32_t*>(base + w.status);
  if (launch_quant_act(q, s) != cudaSuccess) return BL_ERR_CUDA;
  GemmArgs a{};
  a.keep_status = 1;
  a.x_q = codes; a.M = M; a.K = K; a.N = N; a.G = G; a.W_packed = W_packed; a.acc = nullptr;
  a.y = y; a.yt = yt; a.beta = beta; a.gamma = gamma; a.eta = eta; a.gran = gran;
  a.rowsum = rowsum; a.eta_correction = eta_correction ? 1 : 0;
  a.status = reinterpret_cast<uint32_t*>(base + w.status);
  a.scratch = base + w.status + kStatusBytes;
  cudaError_t e = (layout == BL_LAYOUT_PREFILL) ? launch_gemm_tc(a, s) : launch_gemm_simple(a, s);
  return e == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_forward_latent(const void* x, bl_dtype xt, const void* W, bl_dtype wt, int64_t M, int64_t K,
                                   int64_t N, int G, int b, bl_quant_mode mode, bl_gran gran, float ln_eps,
                                   int eta_correction, float* alpha_out, float* beta_out, void* y, bl_dtype yt,
                                   void* ws, size_t ws_bytes, void* stream) {
  if (!x || !W || !y) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  const LatentWs c = carve_latent(M, N, K, G);
  if (!ws || ws_bytes < c.total) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  char* base = reinterpret_cast<char*>(ws);
  uint8_t* packed = reinterpret_cast<uint8_t*>(base + c.packed);
  float* alpha = reinterpret_cast<float*>(base + c.alpha);
  float* beta = reinterpret_cast<float*>(base + c.beta);
  int32_t* rowsum = reinterpret_cast<int32_t*>(base + c.rowsum);
  st = bitlinear_binarize_pack(W, wt, N, K, G, c.layout, nullptr, packed, alpha, beta, rowsum, base + c.pack,
                               round256(pack_ws_bytes(G)), stream);
  if (st != BL_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  if (alpha_out && cudaMemcpyAsync(alpha_out, alpha, (size_t)G * sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return BL_ERR_CUDA;
  if (beta_out && cudaMemcpyAsync(beta_out, beta, (size_t)G * sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return BL_ERR_CUDA;
  return bitlinear_forward(x, xt, M, K, N, G, b, mode, gran, ln_eps, eta_correction, packed, c.layout, beta, rowsum, y,
                           yt, base + c.forward, c.total - c.forward, stream);
}

bl_status bitlinear_gemv_decode(const void* x, bl_dtype xt, int64_t K, int64_t N, int G, int b,
                                bl_quant_mode mode, float ln_eps, int eta_correction,
                                const uint8_t* W_packed, const float* beta,
                                const int32_t* rowsum, void* y, bl_dtype yt, void* stream) {
  if (!x || !W_packed || !beta || !y) return BL_ERR_NULL;
  if (eta_correction && !rowsum) return BL_ERR_NULL;
  if (N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (b != 8 || !valid_dtype(xt) || !valid_dtype(yt)) return BL_ERR_UNSUPPORTED;
  if (mode != BL_ABSMAX && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (eta_correction && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (K % 256 != 0 || N % 16 != 0 || K > 32768) return BL_ERR_SHAPE;
  if (G > 1 && (K / G) % 128 != 0) return BL_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(W_packed) || !aligned16(y)) return BL_ERR_ALIGN;
  GemvArgs a{x, xt, K, N, G, mode, ln_eps, eta_correction ? 1 : 0, W_packed, beta, rowsum, y, yt};
  return launch_gemv_decode(a, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_gemv_decode_batch(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                                      int b, bl_quant_mode mode, float ln_eps, int eta_correction,
                                      const uint8_t* W_packed, const float* beta, const int32_t* rowsum,
                                      void* y, bl_dtype yt, void* stream) {
  if (!x || !W_packed || !beta || !y) return BL_ERR_NULL;
  if (eta_correction && !rowsum) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (b != 8 || !valid_dtype(xt) || !valid_dtype(yt)) return BL_ERR_UNSUPPORTED;
  if (mode != BL_ABSMAX && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (eta_correction && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (!gemv_batch_supported(M, K, N, G)) return BL_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(W_packed) || !aligned16(y)) return BL_ERR_ALIGN;
  GemvArgs a{x, xt, K, N, G, mode, ln_eps, eta_correction ? 1 : 0, W_packed, beta, rowsum, y, yt};
  return launch_gemv_batch(a, M, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_gemv_decode_batch_ws(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                                         int b, bl_quant_mode mode, float ln_eps, int eta_correction,
                                         const uint8_t* W_packed, const float* beta, const int32_t* rowsum,
                                         void* y, bl_dtype yt, void* ws, size_t ws_bytes, void* stream) {
  if (!x || !W_packed || !beta || !y) return BL_ERR_NULL;
  if (eta_correction && !rowsum) return BL_ERR_NULL;
  if (M <= 0 || N <= 0) return BL_ERR_SHAPE;
  bl_status st = check_kg(K, G);
  if (st != BL_OK) return st;
  if (b != 8 || !valid_dtype(xt) || !valid_dtype(yt)) return BL_ERR_UNSUPPORTED;
  if (mode != BL_ABSMAX && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (eta_correction && mode != BL_ETA) return BL_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(W_packed) || !aligned16(y)) return BL_ERR_ALIGN;
  GemvArgs a{x, xt, K, N, G, mode, ln_eps, eta_correction ? 1 : 0, W_packed, beta, rowsum, y, yt};
  if (gemv_tc_supported(M, K, N, G, eta_correction)) {
    if (!ws || ws_bytes < bitlinear_workspace_bytes(BL_OP_GEMV_DECODE_BATCH, M, N, K, G)) return BL_ERR_WORKSPACE;
    if (!aligned16(ws)) return BL_ERR_ALIGN;
    return launch_gemv_tc(a, M, ws, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
  }
  // shapes the tensor-core form does not take: the kernel of bitlinear_gemv_decode_batch; of the workspace
  // only the status word is touched (cleared, so that bitlinear_ws_status answers for this call too)
  if (ws && ws_bytes >= sizeof(uint32_t) && aligned16(ws)) a.clear_status = reinterpret_cast<uint32_t*>(ws);
  if (!gemv_batch_supported(M, K, N, G)) return BL_ERR_SHAPE;
  return launch_gemv_batch(a, M, (cudaStream_t)stream) == cudaSuccess ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_attention_causal(const void* q, const void* k, const void* v, void* o, int batch, int seq,
                                     int heads, int head_dim, int64_t ld, int64_t ld_o, void* stream) {
  if (!q || !k || !v || !o) return BL_ERR_NULL;
  if (batch <= 0 || seq <= 0 || heads <= 0 || seq % 64 != 0 || ld % 8 != 0 || ld_o % 8 != 0) return BL_ERR_SHAPE;
  if (ld < (int64_t)heads * 128 || ld_o < (int64_t)heads * 128) return BL_ERR_SHAPE;
  if (head_dim != 128) return BL_ERR_UNSUPPORTED;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return BL_ERR_ALIGN;
  return launch_attention_causal(q, k, v, o, batch, seq, heads, ld, ld_o, (cudaStream_t)stream) == cudaSuccess
             ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_block_forward(const void* x, int batch, int seq, int heads, int64_t ffn, float ln_eps,
                                  const bl_block_weights* w, const bl_block_buffers* buf, void* y, void* ws,
                                  size_t ws_bytes, void* stream) {
  if (!x || !w || !buf || !y) return BL_ERR_NULL;
  if (!w->W_q || !w->W_k || !w->W_v || !w->W_o || !w->W_up || !w->W_down) return BL_ERR_NULL;
  if (!w->beta_q || !w->beta_k || !w->beta_v || !w->beta_o || !w->beta_up || !w->beta_down) return BL_ERR_NULL;
  if (!buf->q || !buf->k || !buf->v || !buf->a || !buf->h || !buf->u) return BL_ERR_NULL;
  if (batch <= 0 || seq <= 0 || heads <= 0 || ffn <= 0 || seq % 64 != 0 || ffn % 128 != 0) return BL_ERR_SHAPE;
  const int64_t T = (int64_t)batch * seq, d = (int64_t)heads * 128;
  if (!gemm_tc_supported(T, d, d, 1) || !gemm_tc_supported(T, d, ffn, 1) || !gemm_tc_supported(T, ffn, d, 1))
    return BL_ERR_SHAPE;
  const void* ptrs[] = {x, y, buf->q, buf->k, buf->v, buf->a, buf->h, buf->u, w->W_q, w->W_k, w->W_v, w->W_o,
                        w->W_up, w->W_down};
  for (const void* p : ptrs) if (!aligned16(p)) return BL_ERR_ALIGN;
  const int64_t ld_qkv = buf->ld_qkv > 0 ? buf->ld_qkv : d;
  if (ld_qkv < d || ld_qkv % 8 != 0) return BL_ERR_SHAPE;
  const BlockWs c = carve_block(T, d, ffn);
  if (!ws || ws_bytes < c.total) return BL_ERR_WORKSPACE;
  if (!aligned16(ws)) return BL_ERR_ALIGN;
  char* base = reinterpret_cast<char*>(ws);
  cudaStream_t s = (cudaStream_t)stream;
  int8_t* codes = reinterpret_cast<int8_t*>(base + c.codes);
  float* gamma = reinterpret_cast<float*>(base + c.gamma);
  float* eta = reinterpret_cast<float*>(base + c.eta);

  // LN + per-token quantisation of `in` [T,K] (fp16), then W~ x~ rescaled into `out` [T,N] (fp16).
  // One status word for the whole block: the first kernel clears it, every later one keeps it.
  uint32_t* status = reinterpret_cast<uint32_t*>(base + c.gemm);
  bool first_kernel = true;
  auto quant = [&](const void* in, int64_t K, bl_quant_mode mode) -> bool {
    QuantArgs q{in, BL_F16, T, K, 1, mode, BL_PER_TOKEN, ln_eps, codes, gamma, eta, nullptr};
    q.status = status;
    q.keep_status = first_kernel ? 0 : 1;
    first_kernel = false;
    return launch_quant_act(q, s) == cudaSuccess;
  };
  // out [T,N] (row stride ld) = [relu] BitLinear(codes) [+ res]; beta holds one entry per beta_rows features.
  auto matmul = [&](int64_t K, int64_t N, const uint8_t* W, const float* beta, int64_t beta_rows, void* out,
                    int64_t ld, bool relu, const void* res) -> bool {
    GemmArgs g{};
    g.x_q = codes; g.M = T; g.K = K; g.N = N; g.G = 1; g.W_packed = W; g.acc = nullptr; g.y = out; g.yt = BL_F16;
    g.beta = beta; g.gamma = gamma; g.eta = eta; g.gran = BL_PER_TOKEN; g.rowsum = nullptr; g.eta_correction = 0;
    g.beta_rows = beta_rows; g.relu = relu ? 1 : 0; g.residual = res; g.ld_res = d; g.ld_y = ld;
    g.status = status; g.keep_status = 1;
    g.scratch = base + c.gemm + kStatusBytes;
    return launch_gemm_tc(g, s) == cudaSuccess;
  };
  // Q, K, V as one GEMM when the caller laid them out for it: the three packed matrices and their
  // betas back to back (one [3d, d] matrix with a beta per d rows) and q, k, v as the column
  // blocks of one [T, 3d] buffer.
  const size_t wbytes = (size_t)prefill_bytes(d, d);
  const __half* qh = reinterpret_cast<const __half*>(buf->q);
  const bool fused_qkv = ld_qkv == 3 * d && w->W_k == w->W_q + wbytes && w->W_v == w->W_k + wbytes &&
                         w->beta_k == w->beta_q + 1 && w->beta_v == w->beta_k + 1 &&
                         buf->k == (const void*)(qh + d) && buf->v == (const void*)(qh + 2 * d);
  bool ok = quant(x, d, BL_ABSMAX);
  if (fused_qkv) {
    ok = ok && matmul(d, 3 * d, w->W_q, w->beta_q, d, buf->q, ld_qkv, false, nullptr);
  } else {
    ok = ok && matmul(d, d, w->W_q, w->beta_q, 0, buf->q, ld_qkv, false, nullptr)
            && matmul(d, d, w->W_k, w->beta_k, 0, buf->k, ld_qkv, false, nullptr)
            && matmul(d, d, w->W_v, w->beta_v, 0, buf->v, ld_qkv, false, nullptr);
  }
  ok = ok && launch_attention_causal(buf->q, buf->k, buf->v, buf->a, batch, seq, heads, ld_qkv, d, s) == cudaSuccess
      && quant(buf->a, d, BL_ABSMAX) && matmul(d, d, w->W_o, w->beta_o, 0, buf->h, d, false, x)
      && quant(buf->h, d, BL_ABSMAX) && matmul(d, ffn, w->W_up, w->beta_up, 0, buf->u, ffn, true, nullptr)
      && quant(buf->u, ffn, BL_ETA) && matmul(ffn, d, w->W_down, w->beta_down, 0, y, d, false, buf->h);
  return ok ? BL_OK : BL_ERR_CUDA;
}

bl_status bitlinear_ws_status(const void* ws, void* stream) {
  if (!ws) return BL_ERR_NULL;
  uint32_t word = 0;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BL_ERR_CUDA;
  if (cudaMemcpy(&word, ws, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return BL_ERR_CUDA;
  return word == 0 ? BL_OK : BL_ERR_TIMEOUT;
}

int64_t bitlinear_debug_decode_fallbacks(void* stream) {
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return -1;
  unsigned int n = 0;
  if (gemv_decode_take_fallbacks(&n) != cudaSuccess) return -1;
  return (int64_t)n;
}

bl_status bitlinear_debug_wait_limit(int64_t polls, int meet_skew) {
  g_debug_wait_polls.store(polls < 0 ? -1 : (long long)polls, std::memory_order_relaxed);
  g_debug_meet_skew.store(meet_skew ? 1 : 0, std::memory_order_relaxed);
  return BL_OK;
}

}  // extern "C"
