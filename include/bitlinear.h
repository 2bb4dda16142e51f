/*
 * bitlinear.h - C ABI of the B200 (sm_100a) BitLinear forward library.
 *
 * BitLinear (BitNet, Sec. 2.1, Eq. 11):   y = W~ . Quant(LN(x)) . beta.gamma / Q_b
 *   step 1  LN(x) = (x - E x) / sqrt(Var x + eps)                         Eq. 12 (per group: Eq. 15)
 *   step 2  x~ = Clip(round(x^.Q_b/gamma), -(Q_b-1), Q_b-1), gamma = max|x^|   Eq. 4-5
 *           or Clip(round((x^-eta).Q_b/gamma), 0, Q_b-1), eta = min x^         Eq. 6
 *           (in this form gamma = max x^ - min x^, the range of the shifted values: a departure
 *           from Eq. 5 / 14 as printed, whose gamma = ||x||_inf would not map onto [0, Q_b];
 *           the gamma returned for BL_ETA is this range)
 *   step 3  W~ = Sign(W - alpha), alpha = mean W, beta = mean|W|          Eq. 1-3, 12 (per group: Eq. 13)
 *   step 4  acc = W~ x~ in exact integers, rescaled by beta.gamma/Q_b     Eq. 7, 11
 * Symbols follow the paper: M tokens, K input features (the contraction and the group
 * dimension), N output features, G groups along K (K_g = K/G), b = 8 bits, Q_b = 2^(b-1) = 128.
 *
 * Conventions that hold for every entry point unless it says otherwise
 *   - Every data pointer is a DEVICE pointer owned by the caller; matrices are dense row-major;
 *     base addresses are 16-byte aligned (BL_ERR_ALIGN otherwise).
 *   - The library allocates nothing and keeps no results between calls.  Scratch comes from the
 *     caller as (ws, ws_bytes); ask bitlinear_workspace_bytes() for the size.  The workspace
 *     may be reused by the next call on the same stream; it holds nothing the caller needs
 *     except the status word read by bitlinear_ws_status().  What the library does hold, per
 *     process: caches of device attributes and of per-kernel launch set-up (keyed by device
 *     ordinal), a call counter that makes the arrival tags of the cooperative LN+quant kernel
 *     unique, the setting of bitlinear_debug_wait_limit, and the fixed device array behind
 *     bitlinear_quant_act_noalloc.  None of it changes a result.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream) and never synchronise.
 *   - Errors are detected on the host before any launch and returned as a bl_status; nothing
 *     is launched when the status is not BL_OK.  Kernels never trap or print.  A device-side
 *     wait that runs out of its iteration limit records BL_ERR_TIMEOUT in the workspace
 *     status word; outputs of that call are then undefined.
 *   - Rounding to integer codes and to 16-bit outputs is round-half-to-even.
 *   - Requirements on shapes: K % (8*G) == 0, 1 <= G <= BL_MAX_GROUPS, b == 8
 *     (Sec. 2.1 leaves other widths to future work: BL_ERR_UNSUPPORTED).
 */
#ifndef BITLINEAR_H_
#define BITLINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BL_MAX_GROUPS 64

typedef enum {
  BL_OK = 0,
  BL_ERR_NULL = 1,        /* a required pointer is NULL */
  BL_ERR_SHAPE = 2,       /* a size is non-positive or breaks a divisibility rule */
  BL_ERR_ALIGN = 3,       /* a pointer is not 16-byte aligned */
  BL_ERR_UNSUPPORTED = 4, /* b != 8, unknown enum value, or layout not accepted by this call */
  BL_ERR_WORKSPACE = 5,   /* ws is NULL or smaller than bitlinear_workspace_bytes() */
  BL_ERR_CUDA = 6,        /* a CUDA runtime call (launch, attribute, tensor map) failed */
  BL_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (read via bitlinear_ws_status) */
  BL_ERR_TOO_LARGE = 8    /* the problem exceeds the built-in scratch of a *_noalloc entry point */
} bl_status;

typedef enum { BL_F32 = 0, BL_F16 = 1, BL_BF16 = 2 } bl_dtype;

/* Eq. 4-5 (signed codes in [-127,127]) or Eq. 6 (eta-shifted codes in [0,127]). */
typedef enum { BL_ABSMAX = 0, BL_ETA = 1 } bl_quant_mode;

/* Scope of gamma/eta (Sec. 2.1: per tensor in training, per token in inference).
 * PER_TENSOR: gamma, eta have G entries.  PER_TOKEN: M*G entries, index m*G + g. */
typedef enum { BL_PER_TENSOR = 0, BL_PER_TOKEN = 1 } bl_gran;

/* Storage order of the 1-bit weights W~ (bit = 1 means +1).
 *   CANONICAL  u8 [N, K/8]; weight k of row n is bit (k % 8) of byte n*K/8 + k/8.  Accepted by
 *              every entry point except gemv_decode; shapes are unrestricted.
 *   PREFILL    the same bits re-tiled for the tensor-core GEMM: blocks of 128 rows x 128
 *              weights, rows and K padded up to multiples of 128 (see bitlinear_packed_bytes and
 *              bitlinear_layout_index).  Needs K_g % 128 == 0.
 *   DECODE     the same bits re-ordered for the batch-1 GEMV.  Needs K % 256 == 0, N % 16 == 0. */
typedef enum { BL_LAYOUT_CANONICAL = 0, BL_LAYOUT_PREFILL = 1, BL_LAYOUT_DECODE = 2 } bl_layout;

typedef enum {
  BL_OP_BINARIZE_PACK = 0,
  BL_OP_QUANT_ACT = 1,
  BL_OP_FORWARD = 2,
  BL_OP_MATMUL_I32 = 3,
  BL_OP_MATMUL_DEQUANT = 4,
  BL_OP_BLOCK_FORWARD = 5,   /* M = batch * seq tokens, N = ffn width, K = model width d, G ignored (1) */
  BL_OP_FORWARD_LATENT = 6,
  BL_OP_GEMV_DECODE_BATCH = 7  /* bitlinear_gemv_decode_batch_ws; N and G ignored */
} bl_op;

/* Human-readable name of a status code (static string, never NULL). */
const char* bitlinear_status_string(bl_status st);

/* Bytes of scratch the given entry point needs for these sizes (0 on invalid sizes). */
size_t bitlinear_workspace_bytes(bl_op op, int64_t M, int64_t N, int64_t K, int G);

/* Bytes of the packed weight buffer for a layout (includes PREFILL padding); 0 if invalid. */
size_t bitlinear_packed_bytes(bl_layout layout, int64_t N, int64_t K);

/* Where weight (n, k) lives in a packed buffer of the given layout: writes the byte offset
 * and the bit number.  Host-only helper that documents the private layouts; tests use it to
 * map PREFILL/DECODE buffers back to CANONICAL.  Returns BL_ERR_SHAPE when out of range. */
bl_status bitlinear_layout_index(bl_layout layout, int64_t N, int64_t K, int64_t n, int64_t k,
                                 int64_t* byte_offset, int* bit);

/* Step 3, Eq. 1-3, 12, 13: alpha_g, beta_g over the K-slice g of all N rows, then
 * W~ = Sign(W - alpha_g) with Sign(0) = -1, packed 1 bit per weight.
 *   W         [N,K] of dtype wt (read twice).
 *   alpha_in  NULL, or G device floats used in place of the computed means (lets a caller
 *             fix alpha, e.g. to isolate the sign-and-pack step).
 *   W_packed  bitlinear_packed_bytes(layout,N,K) bytes, fully overwritten.
 *   alpha, beta  [G] fp32 outputs (the means in fp64, rounded once).
 *   rowsum    NULL or int32 [N,G]: sum over the group of W~[n,k] (used by eta_correction).
 * Sums are accumulated in fp64 in a fixed order, so results are run-to-run identical; the sign
 * test compares W against the fp64 mean exactly.  Workspace: BL_OP_BINARIZE_PACK. */
bl_status bitlinear_binarize_pack(const void* W, bl_dtype wt, int64_t N, int64_t K, int G,
                                  bl_layout layout, const float* alpha_in, uint8_t* W_packed,
                                  float* alpha, float* beta, int32_t* rowsum, void* ws,
                                  size_t ws_bytes, void* stream);

/* Steps 1-2, Eq. 12/15 then Eq. 4-6/14, b = 8.
 *   x      [M,K] of dtype xt.
 *   ln_eps LN epsilon; a negative value skips LN (codes are taken from x itself).
 *   x_q    int8 [M,K] codes.   gamma, eta: fp32, sized by gran (eta may be NULL for BL_ABSMAX).
 * gamma == 0 (constant input) yields all-zero codes, never NaN.  PER_TOKEN is one pass over x;
 * PER_TENSOR is two (statistics, then codes).  For segments of up to 8 KB that are a multiple of
 * 256 features both passes run in one cooperative kernel whose CTAs wait for one another between
 * the passes, with a limit: after a PER_TENSOR call bitlinear_ws_status(ws, stream) reports
 * BL_ERR_TIMEOUT if that wait expired (codes are then not written).  Workspace: BL_OP_QUANT_ACT.
 * PER_TOKEN needs no workspace (ws may be NULL).  Given one of at least 256 bytes, its first word
 * becomes the call's status word and segments of the shape above are fetched with bulk copies whose
 * bounded wait reports there (bitlinear_ws_status as above); the values written are the same. */
bl_status bitlinear_quant_act(const void* x, bl_dtype xt, int64_t M, int64_t K, int G, int b,
                              bl_quant_mode mode, bl_gran gran, float ln_eps, int8_t* x_q,
                              float* gamma, float* eta, void* ws, size_t ws_bytes, void* stream);

/* bitlinear_quant_act for callers that cannot provide a workspace.  (The paper has no counterpart:
 * this is a packaging variant of the entry point above, not another operation.)
 *
 * Who needs it: code that runs where device memory may not be allocated or sized at run time -
 * a plug-in called from inside another framework's stream callback or graph-building phase, a
 * real-time loop with a fixed memory budget, a host binding that only forwards pointers it was
 * given.  Such callers still own x, x_q, gamma and eta, but have nowhere to put the statistics
 * that the per-tensor path keeps between its two passes.
 *
 * The statistics go to a fixed array inside the library instead (24 bytes per segment for
 * BL_NOALLOC_MAX_SEGMENTS segments plus a 0.26 MB header, about 0.7 MB in all, resident on every
 * GPU that loads the library until the process ends).  Consequences:
 *   - BL_PER_TENSOR calls with M * G > BL_NOALLOC_MAX_SEGMENTS return BL_ERR_TOO_LARGE and launch
 *     nothing.  BL_PER_TOKEN calls keep no statistics there and have no such limit; they use the
 *     array's first word as their status word only.
 *   - All calls on one GPU share the array.  BL_PER_TENSOR calls that may overlap on the GPU
 *     (different streams) race on it and corrupt each other; keep them on one stream or order them
 *     yourself.  Overlapping BL_PER_TOKEN calls share nothing but the status word (each clears it
 *     when it starts), so their outputs are unaffected, but a timeout report of one may be wiped
 *     by the other.  A call leaves nothing behind that the next one depends on.
 *   - The first call on each device looks up the array's device address
 *     (cudaGetSymbolAddress); make that first call outside any stream capture.
 *   - No cudaMalloc, cudaFree or other allocating routine is called, now or later.
 * Arguments, results, host-side error codes and rounding are otherwise exactly those of
 * bitlinear_quant_act; the same kernels run, so the outputs are bit-identical.  The one difference
 * is where a device-side timeout is reported: the status word lives in the library's array, which
 * the caller cannot pass to bitlinear_ws_status; bitlinear_noalloc_status reads it instead. */
#define BL_NOALLOC_MAX_SEGMENTS 16384
bl_status bitlinear_quant_act_noalloc(const void* x, bl_dtype xt, int64_t M, int64_t K, int G, int b,
                                      bl_quant_mode mode, bl_gran gran, float ln_eps, int8_t* x_q,
                                      float* gamma, float* eta, void* stream);

/* Synchronises `stream`, then reads the status word that the last bitlinear_quant_act_noalloc call on
 * the current device left in the library's array (the counterpart of bitlinear_ws_status for that
 * entry point; the paper has no counterpart).  BL_OK, BL_ERR_TIMEOUT (a bounded device-side wait of
 * that call ran out: its codes were not written), or BL_ERR_CUDA.  Allocates nothing. */
bl_status bitlinear_noalloc_status(void* stream);

/* Steps 1, 2, 4, Eq. 11: y = (W~ x~) . beta_g gamma / Q_b summed over groups in ascending order.
 *   eta_correction != 0 (BL_ETA only) adds eta.beta_g.rowsum[n,g], which undoes the shift of
 *   Eq. 6 in the output; 0 is Eq. 11 as printed.
 *   W_packed  CANONICAL (any shape, plain CUDA-core kernel) or PREFILL (tcgen05 tensor-core
 *             kernel); beta [G] and rowsum [N,G] as produced by bitlinear_binarize_pack.
 *   y      [M,N] of dtype yt.
 * Workspace: BL_OP_FORWARD (holds the int8 codes, gamma, eta and the status word). */
bl_status bitlinear_forward(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                            int b, bl_quant_mode mode, bl_gran gran, float ln_eps,
                            int eta_correction, const uint8_t* W_packed, bl_layout layout,
                            const float* beta, const int32_t* rowsum, void* y, bl_dtype yt,
                            void* ws, size_t ws_bytes, void* stream);

/* The layer as it runs in training (Sec. 2.2, "mixed precision training": the latent weights are
 * binarised on the fly during the forward pass): Eq. 1-3 on the high-precision W of this step,
 * then Eq. 11, in one call.  Nothing of the packed form outlives the call except what the caller
 * asks back.
 *   W [N,K] of dtype wt (the latent weights).  Other arguments as for bitlinear_forward.
 *   alpha_out, beta_out  NULL or fp32 [G]: the alpha_g and beta_g of this step (the straight-through
 *                        backward pass needs beta).
 * The packed weights live in the workspace, in PREFILL order when the shape allows the tensor-core
 * kernel (K % 128 == 0 per group), else CANONICAL.  y is bit-identical to bitlinear_binarize_pack
 * followed by bitlinear_forward.  Workspace: BL_OP_FORWARD_LATENT. */
bl_status bitlinear_forward_latent(const void* x, bl_dtype xt, const void* W, bl_dtype wt, int64_t M, int64_t K,
                                   int64_t N, int G, int b, bl_quant_mode mode, bl_gran gran, float ln_eps,
                                   int eta_correction, float* alpha_out, float* beta_out, void* y, bl_dtype yt,
                                   void* ws, size_t ws_bytes, void* stream);

/* Step 4 alone, Eq. 7: acc[g,m,n] = sum over k in group g of W~[n,k] . x_q[m,k], exact int32.
 * The parity hook for "accumulators are bit-exact when fed given codes".
 *   x_q [M,K] int8;  acc int32 [G,M,N].  Layout CANONICAL or PREFILL as for bitlinear_forward.
 * Workspace: BL_OP_MATMUL_I32. */
bl_status bitlinear_matmul_i32(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                               const uint8_t* W_packed, bl_layout layout, int32_t* acc, void* ws,
                               size_t ws_bytes, void* stream);

/* Step 4 with the Eq. 11 rescale, for codes the caller already holds (the second half of
 * bitlinear_forward; lets one LN+Quant of x feed several weight matrices, e.g. Q, K and V).
 *   x_q [M,K] int8;  gamma, eta as written by bitlinear_quant_act for the same (mode, gran);
 *   eta may be NULL unless eta_correction != 0.  Other arguments as for bitlinear_forward.
 * The result is bit-identical to bitlinear_forward on the x that produced the codes.
 * Workspace: BL_OP_MATMUL_DEQUANT. */
bl_status bitlinear_matmul_dequant(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                                   bl_gran gran, const float* gamma, const float* eta,
                                   int eta_correction, const uint8_t* W_packed, bl_layout layout,
                                   const float* beta, const int32_t* rowsum, void* y, bl_dtype yt,
                                   void* ws, size_t ws_bytes, void* stream);

/* bitlinear_matmul_dequant with output-side options, for fusing what follows a BitLinear in the
 * decoder block (Sec. 2, Fig. 2b) into its epilogue, and for weights whose alpha / beta are taken
 * per block of output features (the partitioning of Sec. 2.1 "Model parallelism with Group
 * Quantization", Eq. 13, applied along N: each device's slice of output features carries its own
 * alpha and beta; also how W_q, W_k, W_v stacked into one [3d, d] matrix keep their own beta).
 *   beta_rows  output features per beta block: beta is [N / beta_rows, G] (block-major), rowsum
 *              stays [N, G].  0 means one block (beta [G]).  Must divide N and be a multiple of 32.
 *   relu       non-zero: y = max(y, 0), applied before the residual.
 *   residual   NULL or [M, N] of dtype yt with row stride ld_res (elements): y += residual.
 *              May alias y only if ld_res == ld_y and residual == y (each element is read by
 *              the thread that then writes it).
 *   ld_y       row stride of y in elements (0 means N), so y may be a column block of a wider buffer.
 * With epi == NULL or all-zero options the call equals bitlinear_matmul_dequant. */
typedef struct {
  int64_t beta_rows;
  int relu;
  const void* residual;
  int64_t ld_res;
  int64_t ld_y;
} bl_epilogue;
bl_status bitlinear_matmul_dequant_ex(const int8_t* x_q, int64_t M, int64_t K, int64_t N, int G,
                                      bl_gran gran, const float* gamma, const float* eta,
                                      int eta_correction, const uint8_t* W_packed, bl_layout layout,
                                      const float* beta, const int32_t* rowsum, const bl_epilogue* epi,
                                      void* y, bl_dtype yt, void* ws, size_t ws_bytes, void* stream);

/* bitlinear_binarize_pack for NB blocks of N / NB consecutive output features, each with its own
 * alpha_g and beta_g (Eq. 13 applied along N, see bitlinear_matmul_dequant_ex): block j is
 * binarised against the mean of its own rows.
 *   alpha, beta  [NB, G];  alpha_in NULL or [NB, G];  rowsum NULL or [N, G].
 *   W_packed     the blocks' packed images one after the other, which for PREFILL (N / NB a
 *                multiple of 128) and CANONICAL / DECODE layouts is the packed image of the
 *                whole [N, K] matrix.
 * Runs one pass of bitlinear_binarize_pack per block on `stream`; the workspace is that of one
 * block (BL_OP_BINARIZE_PACK), reused in stream order. */
bl_status bitlinear_binarize_pack_nsplit(const void* W, bl_dtype wt, int64_t N, int64_t K, int G, int NB,
                                         bl_layout layout, const float* alpha_in, uint8_t* W_packed,
                                         float* alpha, float* beta, int32_t* rowsum, void* ws,
                                         size_t ws_bytes, void* stream);

/* Steps 1, 2, 4 for one token (M = 1), fused in a single kernel that streams the packed
 * weights once; Eq. 11 with per-token gamma.  W_packed must be in DECODE layout.
 *   x [K] of dtype xt;  y [N] of dtype yt.  K % 256 == 0, K <= 32768, N % 16 == 0, and for G > 1
 *   K_g % 128 == 0 (BL_ERR_SHAPE otherwise).  No workspace.
 * The weights are constants of the model and are read AHEAD of stream order: the kernel starts
 * copying W_packed into shared memory while earlier work on `stream` may still be running
 * (programmatic dependent launch), so whatever wrote W_packed must have completed before this
 * call is made (a pack on the same stream: synchronise once after packing).  x, beta, rowsum
 * and y are only touched in stream order.
 * The one device-side wait (for those copies) is bounded; if it ever ran out, the affected warps
 * read their weights from global memory instead, so there is no status to collect and y is the
 * same either way. */
bl_status bitlinear_gemv_decode(const void* x, bl_dtype xt, int64_t K, int64_t N, int G, int b,
                                bl_quant_mode mode, float ln_eps, int eta_correction,
                                const uint8_t* W_packed, const float* beta,
                                const int32_t* rowsum, void* y, bl_dtype yt, void* stream);

/* bitlinear_gemv_decode for a small batch: M tokens (decode with a few sequences in flight, the
 * per-token inference of Sec. 2.1 with one weight stream shared by the batch).  Each token gets
 * its own LN statistics, gamma and eta (Eq. 12, 4-6 per token); up to 8 tokens share one pass
 * over the packed weights (tensor-core mma on bit planes of the packed words), larger M runs
 * ceil(M/8) passes with the weights served from L2.  For M >= 2 a token's result does not depend on
 * what else is in the batch (same bits); M == 1 is handed to the kernel of bitlinear_gemv_decode,
 * which is faster for one token and may differ from this one in the last bit of gamma.  W_packed
 * is read ahead of stream order, as there.
 *   x [M,K] of dtype xt;  y [M,N] of dtype yt;  W_packed in DECODE layout.
 *   K % 256 == 0, (K/G) % 256 == 0, N % 16 == 0, min(M, 8) * (K + 16) <= 155 KB (BL_ERR_SHAPE otherwise).
 * No workspace; no device-side waits for M >= 2. */
bl_status bitlinear_gemv_decode_batch(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                                      int b, bl_quant_mode mode, float ln_eps, int eta_correction,
                                      const uint8_t* W_packed, const float* beta, const int32_t* rowsum,
                                      void* y, bl_dtype yt, void* stream);

/* bitlinear_gemv_decode_batch with a workspace (Sec. 2.1, Eq. 12, 4-7, 11 per token), for G == 1,
 * eta_correction == 0, M >= 2 and K <= 12288: two kernels per call.  The first quantises the tokens
 * once (one CTA per token; LN statistics, gamma / eta, codes: the fp32 arithmetic of the kernel of
 * bitlinear_gemv_decode) into the workspace.  The second streams the packed weights once and
 * multiplies: for up to 8 tokens the bit-plane kernel of bitlinear_gemv_decode_batch, told to take
 * codes, gamma and code sums from the workspace instead of quantising every token in every CTA; for
 * more, the tcgen05 tensor cores (weight bit planes written to tensor memory as the A operand, int32
 * accumulators, exact), one pass per 32 tokens (per 16 when K > 6144), so that the time of a call
 * depends little on M up to 32.  A token's result does not depend on what else is in the batch, nor
 * on which of the two product kernels ran (same bits).  Other shapes, G > 1 and eta_correction are
 * handed to bitlinear_gemv_decode_batch's own path where it takes the shape (of the workspace only
 * the status word is used: cleared; its shape rules apply); M == 1 to the kernel of
 * bitlinear_gemv_decode, whose sums run in another order (same codes up to the tolerated ties,
 * gamma to the last bit or so).
 *   x [M,K] of dtype xt;  y [M,N] of dtype yt;  W_packed in DECODE layout, read ahead of stream
 *   order as there.  K % 256 == 0, N % 16 == 0.
 * Workspace: BL_OP_GEMV_DECODE_BATCH (device memory, 16-byte aligned; its first word is the status
 * word of bitlinear_ws_status: the tensor-core kernel's waits are bounded, and BL_ERR_TIMEOUT there
 * means y of this call is not valid).  The workspace holds the codes between the two kernels, so
 * calls that may overlap (different streams) need workspaces of their own. */
bl_status bitlinear_gemv_decode_batch_ws(const void* x, bl_dtype xt, int64_t M, int64_t K, int64_t N, int G,
                                         int b, bl_quant_mode mode, float ln_eps, int eta_correction,
                                         const uint8_t* W_packed, const float* beta, const int32_t* rowsum,
                                         void* y, bl_dtype yt, void* ws, size_t ws_bytes, void* stream);

/* Causal self-attention core of the decoder block (Sec. 2, Fig. 2b; the paper keeps it in high
 * precision): per batch and head O = softmax(Q K^T / sqrt(d_h) + causal mask) V, fp16 in and out,
 * fp32 softmax statistics and accumulators.  No positional encoding.
 *   q, k, v  fp16 [batch*seq, heads*128] with a common row stride ld (elements), so they may be
 *            column blocks of one buffer;  o fp16, same shape, row stride ld_o.
 *   head_dim must be 128, seq a multiple of 64, ld and ld_o multiples of 8. */
bl_status bitlinear_attention_causal(const void* q, const void* k, const void* v, void* o, int batch, int seq,
                                     int heads, int head_dim, int64_t ld, int64_t ld_o, void* stream);

/* One BitNet decoder block, forward (Sec. 2, Fig. 2b): every linear map is a BitLinear (its own
 * LN + per-token 8-bit quantisation in front, Eq. 11), the attention core and the residual adds
 * stay in fp16:
 *     q, k, v = BitLinear_{Q,K,V}(x)            (one LN + quant of x feeds all three)
 *     a       = causal attention(q, k, v)
 *     h       = x + BitLinear_O(a)
 *     u       = ReLU(BitLinear_up(h))
 *     y       = h + BitLinear_down(u)           (down uses the eta form of Eq. 6 on its input)
 * d = heads * 128; FFN width ffn; tokens T = batch * seq (seq % 64 == 0); d % 128 == 0, ffn % 128 == 0.
 * All weight buffers are PREFILL-packed with one group: W_q, W_k, W_v, W_o [d,d], W_up [ffn,d],
 * W_down [d,ffn]; beta_* point to one float each (as written by bitlinear_binarize_pack).
 * Every intermediate is a caller buffer (fp16, row-major), so each stage can be inspected:
 *   q, k, v [T,d] with row stride ld_qkv (0 means d);  a, h [T,d];  u [T,ffn];  y [T,d].
 * ReLU and the two residual adds run in the epilogues of the up, O and down GEMMs.  Q, K and V run
 * as ONE GEMM over a [3d, d] weight matrix when the caller lays them out for it: W_k directly
 * behind W_q and W_v behind W_k in memory (likewise beta_q, beta_k, beta_v, as written by
 * bitlinear_binarize_pack_nsplit with NB = 3), and q, k, v the three column blocks of one
 * [T, 3d] buffer (k = q + d, v = q + 2d, ld_qkv = 3d); otherwise as three GEMMs.  The values
 * written are the same either way.  9 launches in the fused layout, 11 otherwise.
 * Workspace: BL_OP_BLOCK_FORWARD (codes, gamma, eta, quant and GEMM scratch).  Asynchronous on
 * `stream`; bitlinear_ws_status(ws, stream) reports a device-side timeout of any of the block's
 * kernels (the first one clears the status word, the later ones only ever set it). */
typedef struct {
  const uint8_t *W_q, *W_k, *W_v, *W_o, *W_up, *W_down;
  const float *beta_q, *beta_k, *beta_v, *beta_o, *beta_up, *beta_down;
} bl_block_weights;
typedef struct {
  void *q, *k, *v, *a, *h, *u;
  int64_t ld_qkv;
} bl_block_buffers;
bl_status bitlinear_block_forward(const void* x, int batch, int seq, int heads, int64_t ffn, float ln_eps,
                                  const bl_block_weights* w, const bl_block_buffers* buf, void* y, void* ws,
                                  size_t ws_bytes, void* stream);

/* Synchronises `stream`, then reads the status word a previous bitlinear_forward or
 * bitlinear_matmul_i32 call left in `ws`.  BL_OK, BL_ERR_TIMEOUT, or BL_ERR_CUDA. */
bl_status bitlinear_ws_status(const void* ws, void* stream);

/* Test and diagnostic hook: caps the number of polls that the bounded device-side waits of
 * kernels launched afterwards by this process may make (bitlinear_gemv_decode's wait for its
 * weight copies; the meeting between the two passes of the cooperative per-tensor kernel of
 * bitlinear_quant_act).  polls < 0 restores the built-in limits; 0 means a single poll (for
 * bitlinear_gemv_decode: none at all, every warp reads its weights from global memory).
 * meet_skew != 0 additionally makes the cooperative kernel wait for an arrival tag that no CTA
 * publishes, so that its wait runs out by construction: the kernel then records
 * BL_ERR_TIMEOUT in the status word, writes no codes and returns (nothing hangs, traps or
 * faults).  Process-wide and not synchronised with calls in flight on other host threads; not for
 * production use.  Always returns BL_OK. */
bl_status bitlinear_debug_wait_limit(int64_t polls, int meet_skew);

/* Test and diagnostic hook: synchronises `stream`, then returns and clears the number of warps of
 * bitlinear_gemv_decode kernels (on the current device, since the last call of this function) whose
 * bounded wait for a stage of weights ran out, so that they read the stage from global memory
 * instead.  The result of such a call is still correct, only slow; a healthy run returns 0.
 * -1 on a CUDA error. */
int64_t bitlinear_debug_decode_fallbacks(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BITLINEAR_H_ */
