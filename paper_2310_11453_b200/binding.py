"""Thin Python binding of the BitLinear C ABI (include/bitlinear.h): argument marshalling only.

Every function here has the name of the C entry point it calls.  torch supplies device memory
and the current CUDA stream; every step of the computation runs in the library's kernels.
There is no CPU path: a missing or unloadable library raises at first use.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbitlinear_b200.so")

# enums of include/bitlinear.h
OK = 0
F32, F16, BF16 = 0, 1, 2
ABSMAX, ETA = 0, 1
PER_TENSOR, PER_TOKEN = 0, 1
CANONICAL, PREFILL, DECODE = 0, 1, 2
OP_BINARIZE_PACK, OP_QUANT_ACT, OP_FORWARD, OP_MATMUL_I32, OP_MATMUL_DEQUANT, OP_BLOCK_FORWARD = 0, 1, 2, 3, 4, 5
OP_FORWARD_LATENT = 6
OP_GEMV_DECODE_BATCH = 7
MAX_GROUPS = 64
NOALLOC_MAX_SEGMENTS = 16384
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_TOO_LARGE = 1, 2, 3, 4, 5, 6, 7, 8

EXPORTS = [
    "bitlinear_status_string", "bitlinear_workspace_bytes", "bitlinear_packed_bytes",
    "bitlinear_layout_index", "bitlinear_binarize_pack", "bitlinear_quant_act", "bitlinear_quant_act_noalloc",
    "bitlinear_forward", "bitlinear_matmul_i32", "bitlinear_matmul_dequant", "bitlinear_gemv_decode",
    "bitlinear_attention_causal", "bitlinear_block_forward", "bitlinear_ws_status",
    "bitlinear_matmul_dequant_ex", "bitlinear_binarize_pack_nsplit", "bitlinear_gemv_decode_batch",
    "bitlinear_forward_latent", "bitlinear_debug_wait_limit", "bitlinear_noalloc_status", "bitlinear_debug_decode_fallbacks",
    "bitlinear_gemv_decode_batch_ws",
]

_DTYPES = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
_lib = None


class BitLinearError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        super().__init__(f"{where}: {status_string(code)} (bl_status {int(code)})")


def lib():
    """Load the CUDA library (built in-tree by paper_2310_11453_b200.build); fail loudly."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2310_11453_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        i64, vp, ci, sz = C.c_int64, C.c_void_p, C.c_int, C.c_size_t
        L.bitlinear_status_string.restype = C.c_char_p
        L.bitlinear_status_string.argtypes = [ci]
        L.bitlinear_workspace_bytes.restype = sz
        L.bitlinear_workspace_bytes.argtypes = [ci, i64, i64, i64, ci]
        L.bitlinear_packed_bytes.restype = sz
        L.bitlinear_packed_bytes.argtypes = [ci, i64, i64]
        L.bitlinear_layout_index.restype = ci
        L.bitlinear_layout_index.argtypes = [ci, i64, i64, i64, i64, C.POINTER(i64), C.POINTER(ci)]
        L.bitlinear_binarize_pack.restype = ci
        L.bitlinear_binarize_pack.argtypes = [vp, ci, i64, i64, ci, ci, vp, vp, vp, vp, vp, vp, sz, vp]
        L.bitlinear_quant_act.restype = ci
        L.bitlinear_quant_act.argtypes = [vp, ci, i64, i64, ci, ci, ci, ci, C.c_float, vp, vp, vp, vp, sz, vp]
        L.bitlinear_quant_act_noalloc.restype = ci
        L.bitlinear_quant_act_noalloc.argtypes = [vp, ci, i64, i64, ci, ci, ci, ci, C.c_float, vp, vp, vp, vp]
        L.bitlinear_forward.restype = ci
        L.bitlinear_forward.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, ci, C.c_float, ci, vp, ci,
                                        vp, vp, vp, ci, vp, sz, vp]
        L.bitlinear_matmul_i32.restype = ci
        L.bitlinear_matmul_i32.argtypes = [vp, i64, i64, i64, ci, vp, ci, vp, vp, sz, vp]
        L.bitlinear_matmul_dequant.restype = ci
        L.bitlinear_matmul_dequant.argtypes = [vp, i64, i64, i64, ci, ci, vp, vp, ci, vp, ci, vp, vp, vp, ci,
                                               vp, sz, vp]
        L.bitlinear_gemv_decode.restype = ci
        L.bitlinear_gemv_decode.argtypes = [vp, ci, i64, i64, ci, ci, ci, C.c_float, ci, vp, vp, vp,
                                            vp, ci, vp]
        L.bitlinear_attention_causal.restype = ci
        L.bitlinear_attention_causal.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, i64, i64, vp]
        L.bitlinear_block_forward.restype = ci
        L.bitlinear_block_forward.argtypes = [vp, ci, ci, ci, i64, C.c_float, vp, vp, vp, vp, sz, vp]
        L.bitlinear_ws_status.restype = ci
        L.bitlinear_ws_status.argtypes = [vp, vp]
        L.bitlinear_matmul_dequant_ex.restype = ci
        L.bitlinear_matmul_dequant_ex.argtypes = [vp, i64, i64, i64, ci, ci, vp, vp, ci, vp, ci, vp, vp, vp, vp, ci,
                                                  vp, sz, vp]
        L.bitlinear_forward_latent.restype = ci
        L.bitlinear_forward_latent.argtypes = [vp, ci, vp, ci, i64, i64, i64, ci, ci, ci, ci, C.c_float, ci, vp, vp, vp,
                                               ci, vp, sz, vp]
        L.bitlinear_gemv_decode_batch.restype = ci
        L.bitlinear_gemv_decode_batch.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, C.c_float, ci, vp, vp, vp, vp,
                                                  ci, vp]
        L.bitlinear_gemv_decode_batch_ws.restype = ci
        L.bitlinear_gemv_decode_batch_ws.argtypes = [vp, ci, i64, i64, i64, ci, ci, ci, C.c_float, ci, vp, vp, vp, vp,
                                                     ci, vp, sz, vp]
        L.bitlinear_binarize_pack_nsplit.restype = ci
        L.bitlinear_binarize_pack_nsplit.argtypes = [vp, ci, i64, i64, ci, ci, ci, vp, vp, vp, vp, vp, vp, sz, vp]
        L.bitlinear_debug_decode_fallbacks.restype = i64
        L.bitlinear_debug_decode_fallbacks.argtypes = [vp]
        L.bitlinear_noalloc_status.restype = ci
        L.bitlinear_noalloc_status.argtypes = [vp]
        L.bitlinear_debug_wait_limit.restype = ci
        L.bitlinear_debug_wait_limit.argtypes = [i64, ci]
        _lib = L
    return _lib


def status_string(code) -> str:
    return lib().bitlinear_status_string(int(code)).decode()


def _check(code, where):
    if code != OK:
        raise BitLinearError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dt(t):
    try:
        return _DTYPES[t.dtype]
    except KeyError:
        raise TypeError(f"unsupported dtype {t.dtype}")


def workspace_bytes(op, M, N, K, G) -> int:
    return int(lib().bitlinear_workspace_bytes(op, M, N, K, G))


def packed_bytes(layout, N, K) -> int:
    return int(lib().bitlinear_packed_bytes(layout, N, K))


def layout_index(layout, N, K, n, k):
    off, bit = C.c_int64(0), C.c_int(0)
    _check(lib().bitlinear_layout_index(layout, N, K, n, k, C.byref(off), C.byref(bit)), "layout_index")
    return off.value, bit.value


def _ws(nbytes, device, ws=None):
    if ws is not None:
        return ws
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def binarize_pack(W, G=1, layout=CANONICAL, alpha_in=None, want_rowsum=True, out=None, ws=None):
    """bitlinear_binarize_pack.  W [N,K] on the GPU.  Returns dict(W_packed u8, alpha, beta [G] f32,
    rowsum [N,G] i32 or None).  `out` may carry preallocated tensors under the same keys."""
    N, K = W.shape
    dev = W.device
    nbytes = packed_bytes(layout, N, K)
    out = dict(out or {})
    packed = out.get("W_packed")
    if packed is None:
        packed = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=dev)
    alpha = out.get("alpha", None)
    alpha = alpha if alpha is not None else torch.empty(G, dtype=torch.float32, device=dev)
    beta = out.get("beta", None)
    beta = beta if beta is not None else torch.empty(G, dtype=torch.float32, device=dev)
    rowsum = out.get("rowsum", None)
    if rowsum is None and want_rowsum:
        rowsum = torch.empty((N, G), dtype=torch.int32, device=dev)
    ws = _ws(workspace_bytes(OP_BINARIZE_PACK, 1, N, K, G), dev, ws)
    code = lib().bitlinear_binarize_pack(_ptr(W), _dt(W), N, K, G, layout, _ptr(alpha_in), _ptr(packed),
                                         _ptr(alpha), _ptr(beta), _ptr(rowsum), _ptr(ws), ws.numel(),
                                         _stream())
    _check(code, "bitlinear_binarize_pack")
    return dict(W_packed=packed, alpha=alpha, beta=beta, rowsum=rowsum, layout=layout, N=N, K=K, G=G)


def binarize_pack_nsplit(W, NB, G=1, layout=CANONICAL, alpha_in=None, want_rowsum=True, ws=None):
    """bitlinear_binarize_pack_nsplit.  W [N,K]; NB blocks of N/NB output features, each with its own
    alpha / beta.  Returns dict(W_packed, alpha, beta [NB,G], rowsum [N,G] or None, beta_rows)."""
    N, K = W.shape
    dev = W.device
    rows = N // NB
    nbytes = NB * packed_bytes(layout, rows, K)
    packed = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=dev)
    alpha = torch.empty((NB, G), dtype=torch.float32, device=dev)
    beta = torch.empty((NB, G), dtype=torch.float32, device=dev)
    rowsum = torch.empty((N, G), dtype=torch.int32, device=dev) if want_rowsum else None
    ws = _ws(workspace_bytes(OP_BINARIZE_PACK, 1, rows, K, G), dev, ws)
    code = lib().bitlinear_binarize_pack_nsplit(_ptr(W), _dt(W), N, K, G, NB, layout, _ptr(alpha_in), _ptr(packed),
                                                _ptr(alpha), _ptr(beta), _ptr(rowsum), _ptr(ws), ws.numel(),
                                                _stream())
    _check(code, "bitlinear_binarize_pack_nsplit")
    return dict(W_packed=packed, alpha=alpha, beta=beta, rowsum=rowsum, layout=layout, N=N, K=K, G=G, NB=NB,
                beta_rows=rows)


def quant_act(x, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, b=8, out=None, ws=None):
    """bitlinear_quant_act.  x [M,K].  Returns dict(x_q i8 [M,K], gamma, eta f32).
    ws=False passes no workspace at all (allowed for PER_TOKEN only)."""
    M, K = x.shape
    dev = x.device
    out = dict(out or {})
    ns = (M, G) if gran == PER_TOKEN else (G,)
    x_q = out.get("x_q")
    x_q = x_q if x_q is not None else torch.empty((M, K), dtype=torch.int8, device=dev)
    gamma = out.get("gamma")
    gamma = gamma if gamma is not None else torch.empty(ns, dtype=torch.float32, device=dev)
    eta = out.get("eta")
    eta = eta if eta is not None else torch.zeros(ns, dtype=torch.float32, device=dev)
    if ws is False:
        ws_ptr, ws_bytes = None, 0
    else:
        ws = _ws(workspace_bytes(OP_QUANT_ACT, M, 1, K, G), dev, ws)
        ws_ptr, ws_bytes = _ptr(ws), ws.numel()
    code = lib().bitlinear_quant_act(_ptr(x), _dt(x), M, K, G, b, mode, gran, float(ln_eps), _ptr(x_q),
                                     _ptr(gamma), _ptr(eta), ws_ptr, ws_bytes, _stream())
    _check(code, "bitlinear_quant_act")
    return dict(x_q=x_q, gamma=gamma, eta=eta)


def quant_act_noalloc(x, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, b=8, out=None):
    """bitlinear_quant_act_noalloc: bitlinear_quant_act without a caller workspace (the per-tensor
    statistics go to a fixed array inside the library).  `out` must carry x_q, gamma and eta: this
    wrapper allocates nothing either.  Returns `out`."""
    M, K = x.shape
    code = lib().bitlinear_quant_act_noalloc(_ptr(x), _dt(x), M, K, G, b, mode, gran, float(ln_eps),
                                             _ptr(out["x_q"]), _ptr(out["gamma"]), _ptr(out.get("eta")),
                                             _stream())
    _check(code, "bitlinear_quant_act_noalloc")
    return out


def forward(x, W_packed, beta, N, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, layout=CANONICAL,
            rowsum=None, eta_correction=False, out_dtype=None, b=8, y=None, ws=None):
    """bitlinear_forward.  x [M,K]; returns y [M,N] of out_dtype (default: x.dtype)."""
    M, K = x.shape
    dev = x.device
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=dev)
    ws = _ws(workspace_bytes(OP_FORWARD, M, N, K, G), dev, ws)
    code = lib().bitlinear_forward(_ptr(x), _dt(x), M, K, N, G, b, mode, gran, float(ln_eps),
                                   1 if eta_correction else 0, _ptr(W_packed), layout, _ptr(beta),
                                   _ptr(rowsum), _ptr(y), _dt(y), _ptr(ws), ws.numel(), _stream())
    _check(code, "bitlinear_forward")
    return y


def matmul_i32(x_q, W_packed, N, G=1, layout=CANONICAL, acc=None, ws=None):
    """bitlinear_matmul_i32.  x_q i8 [M,K]; returns acc i32 [G,M,N]."""
    M, K = x_q.shape
    dev = x_q.device
    if acc is None:
        acc = torch.empty((G, M, N), dtype=torch.int32, device=dev)
    ws = _ws(workspace_bytes(OP_MATMUL_I32, M, N, K, G), dev, ws)
    code = lib().bitlinear_matmul_i32(_ptr(x_q), M, K, N, G, _ptr(W_packed), layout, _ptr(acc), _ptr(ws),
                                      ws.numel(), _stream())
    _check(code, "bitlinear_matmul_i32")
    return acc


def matmul_dequant(x_q, gamma, W_packed, beta, N, G=1, gran=PER_TOKEN, layout=CANONICAL, eta=None,
                   rowsum=None, eta_correction=False, out_dtype=torch.float32, y=None, ws=None):
    """bitlinear_matmul_dequant.  x_q i8 [M,K] with its gamma (and eta); returns y [M,N]."""
    M, K = x_q.shape
    dev = x_q.device
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype, device=dev)
    ws = _ws(workspace_bytes(OP_MATMUL_DEQUANT, M, N, K, G), dev, ws)
    code = lib().bitlinear_matmul_dequant(_ptr(x_q), M, K, N, G, gran, _ptr(gamma), _ptr(eta),
                                          1 if eta_correction else 0, _ptr(W_packed), layout, _ptr(beta),
                                          _ptr(rowsum), _ptr(y), _dt(y), _ptr(ws), ws.numel(), _stream())
    _check(code, "bitlinear_matmul_dequant")
    return y


def forward_latent(x, W, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, eta_correction=False, out_dtype=None,
                   b=8, y=None, ws=None):
    """bitlinear_forward_latent.  x [M,K], latent W [N,K]; returns dict(y [M,N], alpha, beta [G], ws)."""
    M, K = x.shape
    N = W.shape[0]
    dev = x.device
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=dev)
    alpha = torch.empty(G, dtype=torch.float32, device=dev)
    beta = torch.empty(G, dtype=torch.float32, device=dev)
    ws = _ws(workspace_bytes(OP_FORWARD_LATENT, M, N, K, G), dev, ws)
    code = lib().bitlinear_forward_latent(_ptr(x), _dt(x), _ptr(W), _dt(W), M, K, N, G, b, mode, gran,
                                          float(ln_eps), 1 if eta_correction else 0, _ptr(alpha), _ptr(beta),
                                          _ptr(y), _dt(y), _ptr(ws), ws.numel(), _stream())
    _check(code, "bitlinear_forward_latent")
    return dict(y=y, alpha=alpha, beta=beta, ws=ws)


class _Epilogue(C.Structure):
    _fields_ = [("beta_rows", C.c_int64), ("relu", C.c_int), ("residual", C.c_void_p), ("ld_res", C.c_int64),
                ("ld_y", C.c_int64)]


def matmul_dequant_ex(x_q, gamma, W_packed, beta, N, G=1, gran=PER_TOKEN, layout=CANONICAL, eta=None,
                      rowsum=None, eta_correction=False, beta_rows=0, relu=False, residual=None, y=None,
                      out_dtype=torch.float32, ws=None):
    """bitlinear_matmul_dequant_ex.  `y` may be a column slice of a wider row-major tensor (its row
    stride becomes ld_y), `residual` likewise.  Returns y [M,N]."""
    M, K = x_q.shape
    dev = x_q.device
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype, device=dev)
    assert y.stride(1) == 1 and (residual is None or (residual.stride(1) == 1 and residual.dtype == y.dtype))
    epi = _Epilogue(int(beta_rows), 1 if relu else 0, _ptr(residual),
                    residual.stride(0) if residual is not None else 0, y.stride(0))
    ws = _ws(workspace_bytes(OP_MATMUL_DEQUANT, M, N, K, G), dev, ws)
    code = lib().bitlinear_matmul_dequant_ex(_ptr(x_q), M, K, N, G, gran, _ptr(gamma), _ptr(eta),
                                             1 if eta_correction else 0, _ptr(W_packed), layout, _ptr(beta),
                                             _ptr(rowsum), C.byref(epi), _ptr(y), _dt(y), _ptr(ws), ws.numel(),
                                             _stream())
    _check(code, "bitlinear_matmul_dequant_ex")
    return y


def gemv_decode(x, W_packed, beta, N, G=1, mode=ABSMAX, ln_eps=1e-5, rowsum=None,
                eta_correction=False, out_dtype=None, b=8, y=None):
    """bitlinear_gemv_decode.  x [K] or [1,K]; W_packed in DECODE layout; returns y [N]."""
    K = x.numel()
    if y is None:
        y = torch.empty(N, dtype=out_dtype or x.dtype, device=x.device)
    code = lib().bitlinear_gemv_decode(_ptr(x), _dt(x), K, N, G, b, mode, float(ln_eps),
                                       1 if eta_correction else 0, _ptr(W_packed), _ptr(beta),
                                       _ptr(rowsum), _ptr(y), _dt(y), _stream())
    _check(code, "bitlinear_gemv_decode")
    return y


def gemv_decode_batch(x, W_packed, beta, N, G=1, mode=ABSMAX, ln_eps=1e-5, rowsum=None,
                      eta_correction=False, out_dtype=None, b=8, y=None):
    """bitlinear_gemv_decode_batch.  x [M,K]; W_packed in DECODE layout; returns y [M,N]."""
    M, K = x.shape
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=x.device)
    code = lib().bitlinear_gemv_decode_batch(_ptr(x), _dt(x), M, K, N, G, b, mode, float(ln_eps),
                                             1 if eta_correction else 0, _ptr(W_packed), _ptr(beta),
                                             _ptr(rowsum), _ptr(y), _dt(y), _stream())
    _check(code, "bitlinear_gemv_decode_batch")
    return y


def gemv_decode_batch_ws(x, W_packed, beta, N, G=1, mode=ABSMAX, ln_eps=1e-5, rowsum=None,
                         eta_correction=False, out_dtype=None, b=8, y=None, ws=None):
    """bitlinear_gemv_decode_batch_ws.  x [M,K]; W_packed in DECODE layout; returns y [M,N].  `ws` may carry a
    workspace of workspace_bytes(OP_GEMV_DECODE_BATCH, M, N, K, G) bytes (its first word is the status word)."""
    M, K = x.shape
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype or x.dtype, device=x.device)
    ws = _ws(workspace_bytes(OP_GEMV_DECODE_BATCH, M, N, K, G), x.device, ws)
    code = lib().bitlinear_gemv_decode_batch_ws(_ptr(x), _dt(x), M, K, N, G, b, mode, float(ln_eps),
                                                1 if eta_correction else 0, _ptr(W_packed), _ptr(beta),
                                                _ptr(rowsum), _ptr(y), _dt(y), _ptr(ws), ws.numel(), _stream())
    _check(code, "bitlinear_gemv_decode_batch_ws")
    return y


class _BlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("W_q", "W_k", "W_v", "W_o", "W_up", "W_down",
                                          "beta_q", "beta_k", "beta_v", "beta_o", "beta_up", "beta_down")]


class _BlockBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q", "k", "v", "a", "h", "u")] + [("ld_qkv", C.c_int64)]


def attention_causal(q, k, v, batch, seq, heads, head_dim=128, o=None):
    """bitlinear_attention_causal.  q, k, v fp16 [batch*seq, heads*head_dim] (may be column slices of
    one buffer with a common row stride); returns o fp16 [batch*seq, heads*head_dim]."""
    T = batch * seq
    if o is None:
        o = torch.empty((T, heads * head_dim), dtype=torch.float16, device=q.device)
    assert q.stride(1) == 1 and k.stride() == q.stride() and v.stride() == q.stride()
    code = lib().bitlinear_attention_causal(_ptr(q), _ptr(k), _ptr(v), _ptr(o), batch, seq, heads, head_dim,
                                            q.stride(0), o.stride(0), _stream())
    _check(code, "bitlinear_attention_causal")
    return o


def fuse_qkv_weights(weights):
    """Copies the packed W_q, W_k, W_v and their betas back to back (the layout that lets
    bitlinear_block_forward run them as one GEMM); returns a new weights dict sharing the rest."""
    q, k, v = (weights[n] for n in ("q", "k", "v"))
    nb = packed_bytes(PREFILL, q["N"], q["K"])
    packed = torch.cat([t["W_packed"][:nb] for t in (q, k, v)])
    beta = torch.cat([t["beta"].reshape(1) for t in (q, k, v)])
    fused = dict(weights)
    for i, n in enumerate(("q", "k", "v")):
        fused[n] = dict(weights[n], W_packed=packed[i * nb:(i + 1) * nb], beta=beta[i:i + 1])
    fused["_qkv_storage"] = (packed, beta)
    return fused


def block_forward(x, weights, batch, seq, heads, ffn, ln_eps=1e-5, ws=None, fused_qkv=False):
    """bitlinear_block_forward.  x fp16 [batch*seq, heads*128]; `weights` maps q, k, v, o, up, down to
    the dicts returned by binarize_pack(layout=PREFILL) (pass them through fuse_qkv_weights and set
    fused_qkv for the one-GEMM Q/K/V layout).  Returns dict(y, q, k, v, a, h, u): the output and every
    intermediate, all fp16 (q, k, v are column slices of one [T,3d] tensor when fused_qkv)."""
    T, d = x.shape
    dev = x.device
    f16 = dict(dtype=torch.float16, device=dev)
    out = {n: torch.empty((T, d), **f16) for n in ("a", "h", "y")}
    if fused_qkv:
        qkv = torch.empty((T, 3 * d), **f16)
        out.update(q=qkv[:, :d], k=qkv[:, d:2 * d], v=qkv[:, 2 * d:], qkv=qkv)
    else:
        out.update({n: torch.empty((T, d), **f16) for n in ("q", "k", "v")})
    out["u"] = torch.empty((T, ffn), **f16)
    w = _BlockWeights(*[weights[n]["W_packed"].data_ptr() for n in ("q", "k", "v", "o", "up", "down")],
                      *[weights[n]["beta"].data_ptr() for n in ("q", "k", "v", "o", "up", "down")])
    b = _BlockBuffers(*[out[n].data_ptr() for n in ("q", "k", "v", "a", "h", "u")], out["q"].stride(0))
    ws = _ws(workspace_bytes(OP_BLOCK_FORWARD, T, ffn, d, 1), dev, ws)
    code = lib().bitlinear_block_forward(_ptr(x), batch, seq, heads, ffn, float(ln_eps), C.byref(w), C.byref(b),
                                         _ptr(out["y"]), _ptr(ws), ws.numel(), _stream())
    _check(code, "bitlinear_block_forward")
    out["ws"] = ws
    return out


def debug_decode_fallbacks() -> int:
    """bitlinear_debug_decode_fallbacks: synchronises; warps that read weights from global memory since the last call."""
    return int(lib().bitlinear_debug_decode_fallbacks(_stream()))


def noalloc_status() -> int:
    """bitlinear_noalloc_status: synchronises the current stream; verdict of the last no-alloc call."""
    return int(lib().bitlinear_noalloc_status(_stream()))


def debug_wait_limit(polls=-1, meet_skew=False) -> None:
    """bitlinear_debug_wait_limit: test hook (poll cap of the bounded device-side waits; -1 restores)."""
    _check(lib().bitlinear_debug_wait_limit(int(polls), 1 if meet_skew else 0), "debug_wait_limit")


def ws_status(ws) -> int:
    """bitlinear_ws_status: synchronises the current stream and returns the status word's verdict."""
    return int(lib().bitlinear_ws_status(_ptr(ws), _stream()))
