"""ctypes front end of the CPU oracle (oracle/bitlinear_oracle.cpp).

Test infrastructure: only tests/, the smoke check and the CPU-baseline leg of the benchmark
import this.  Arrays are numpy, host memory, row-major.  Inputs of a 16-bit dtype are passed as
float32 holding exactly the 16-bit values.
"""
import ctypes as C

import numpy as np

from . import build as _build

ABSMAX, ETA = 0, 1
PER_TENSOR, PER_TOKEN = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a, t):
    return None if a is None else a.ctypes.data_as(C.POINTER(t))


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with code {rc}")


def binarize(W, G=1, alpha_in=None):
    """Eq. 1-3, 12, 13.  Returns dict(bits[N,K/8] u8, alpha[G], beta[G] f64, rowsum[N,G] i32)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    bits = np.zeros((N, K // 8), np.uint8)
    alpha = np.zeros(G, np.float64)
    beta = np.zeros(G, np.float64)
    rowsum = np.zeros((N, G), np.int32)
    ain = None if alpha_in is None else np.ascontiguousarray(alpha_in, dtype=np.float64)
    rc = lib().oracle_binarize(_p(W, C.c_float), C.c_int64(N), C.c_int64(K), C.c_int(G),
                               _p(ain, C.c_double), _p(bits, C.c_uint8), _p(alpha, C.c_double),
                               _p(beta, C.c_double), _p(rowsum, C.c_int32))
    _check(rc, "binarize")
    return dict(bits=bits, alpha=alpha, beta=beta, rowsum=rowsum)


def binarize_nsplit(W, NB, G=1, alpha_in=None):
    """Eq. 13 with the partition taken along the output features (Sec. 2.1, model parallelism with
    group quantisation): NB blocks of N/NB consecutive rows, each binarised against its own
    alpha_g and scaled by its own beta_g.  Returns bits [N,K/8], alpha, beta [NB,G], rowsum [N,G]."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    if N % NB != 0:
        raise ValueError("NB must divide N")
    rows = N // NB
    parts = [binarize(W[j * rows:(j + 1) * rows], G=G,
                      alpha_in=None if alpha_in is None else np.asarray(alpha_in)[j]) for j in range(NB)]
    return dict(bits=np.concatenate([p["bits"] for p in parts], axis=0),
                alpha=np.stack([p["alpha"] for p in parts]), beta=np.stack([p["beta"] for p in parts]),
                rowsum=np.concatenate([p["rowsum"] for p in parts], axis=0))


def dequant_nsplit(acc, beta, gamma, gran=PER_TOKEN, eta=None, rowsum=None, eta_correction=False):
    """Eq. 11 rescale with beta [NB,G] per block of output features.  acc [G,M,N]; returns y f64 [M,N]."""
    beta = np.asarray(beta, dtype=np.float64)
    NB = beta.shape[0]
    G, M, N = acc.shape
    rows = N // NB
    cols = []
    for j in range(NB):
        sl = slice(j * rows, (j + 1) * rows)
        cols.append(dequant(acc[:, :, sl], beta[j], gamma, gran=gran, eta=eta,
                            rowsum=None if rowsum is None else rowsum[sl], eta_correction=eta_correction))
    return np.concatenate(cols, axis=1)


def quant_act(x, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, want_xhat=False):
    """Eq. 12/15 then Eq. 4-6/14.  Returns dict(codes i8 [M,K], gamma, eta f64, xhat?)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    M, K = x.shape
    ns = M * G if gran == PER_TOKEN else G
    codes = np.zeros((M, K), np.int8)
    gamma = np.zeros(ns, np.float64)
    eta = np.zeros(ns, np.float64)
    xhat = np.zeros((M, K), np.float64) if want_xhat else None
    rc = lib().oracle_quant_act(_p(x, C.c_float), C.c_int64(M), C.c_int64(K), C.c_int(G),
                                C.c_int(mode), C.c_int(gran), C.c_double(ln_eps),
                                _p(codes, C.c_int8), _p(gamma, C.c_double), _p(eta, C.c_double),
                                _p(xhat, C.c_double))
    _check(rc, "quant_act")
    shape = (M, G) if gran == PER_TOKEN else (G,)
    out = dict(codes=codes, gamma=gamma.reshape(shape), eta=eta.reshape(shape))
    if want_xhat:
        out["xhat"] = xhat
    return out


def matmul(codes, bits, G=1):
    """Eq. 7 per group.  Returns acc i32 [G,M,N]."""
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    M, K = codes.shape
    N = bits.shape[0]
    acc = np.zeros((G, M, N), np.int32)
    rc = lib().oracle_matmul(_p(codes, C.c_int8), _p(bits, C.c_uint8), C.c_int64(M),
                             C.c_int64(N), C.c_int64(K), C.c_int(G), _p(acc, C.c_int32))
    _check(rc, "matmul")
    return acc


def matmul_samples(codes, bits, ms, ns, G=1):
    """Eq. 7 for chosen outputs only.  Returns acc i32 [len(ms), G]."""
    codes = np.ascontiguousarray(codes, dtype=np.int8)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    M, K = codes.shape
    N = bits.shape[0]
    acc = np.zeros((len(ms), G), np.int32)
    rc = lib().oracle_matmul_samples(_p(codes, C.c_int8), _p(bits, C.c_uint8), C.c_int64(M),
                                     C.c_int64(N), C.c_int64(K), C.c_int(G), _p(ms, C.c_int64),
                                     _p(ns, C.c_int64), C.c_int64(len(ms)), _p(acc, C.c_int32))
    _check(rc, "matmul_samples")
    return acc


def dequant(acc, beta, gamma, gran=PER_TOKEN, eta=None, rowsum=None, eta_correction=False):
    """Eq. 11 rescale.  acc [G,M,N]; returns y f64 [M,N]."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    G, M, N = acc.shape
    beta = np.ascontiguousarray(beta, dtype=np.float64).reshape(-1)
    gamma = np.ascontiguousarray(gamma, dtype=np.float64).reshape(-1)
    eta_a = None if eta is None else np.ascontiguousarray(eta, dtype=np.float64).reshape(-1)
    rs = None if rowsum is None else np.ascontiguousarray(rowsum, dtype=np.int32)
    y = np.zeros((M, N), np.float64)
    rc = lib().oracle_dequant(_p(acc, C.c_int32), C.c_int64(M), C.c_int64(N), C.c_int(G),
                              C.c_int(gran), _p(beta, C.c_double), _p(gamma, C.c_double),
                              _p(eta_a, C.c_double), _p(rs, C.c_int32),
                              C.c_int(1 if eta_correction else 0), _p(y, C.c_double))
    _check(rc, "dequant")
    return y


def forward(x, bits, beta, G=1, mode=ABSMAX, gran=PER_TOKEN, ln_eps=1e-5, rowsum=None,
            eta_correction=False):
    """Eq. 11, the whole layer.  Returns dict(y f64 [M,N], codes, gamma, eta, acc)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    M, K = x.shape
    N = bits.shape[0]
    ns = M * G if gran == PER_TOKEN else G
    beta = np.ascontiguousarray(beta, dtype=np.float64).reshape(-1)
    rs = None if rowsum is None else np.ascontiguousarray(rowsum, dtype=np.int32)
    codes = np.zeros((M, K), np.int8)
    gamma = np.zeros(ns, np.float64)
    eta = np.zeros(ns, np.float64)
    acc = np.zeros((G, M, N), np.int32)
    y = np.zeros((M, N), np.float64)
    rc = lib().oracle_forward(_p(x, C.c_float), C.c_int64(M), C.c_int64(K), C.c_int64(N),
                              C.c_int(G), C.c_int(mode), C.c_int(gran), C.c_double(ln_eps),
                              C.c_int(1 if eta_correction else 0), _p(bits, C.c_uint8),
                              _p(beta, C.c_double), _p(rs, C.c_int32), _p(codes, C.c_int8),
                              _p(gamma, C.c_double), _p(eta, C.c_double), _p(acc, C.c_int32),
                              _p(y, C.c_double))
    _check(rc, "forward")
    shape = (M, G) if gran == PER_TOKEN else (G,)
    return dict(y=y, codes=codes, gamma=gamma.reshape(shape), eta=eta.reshape(shape), acc=acc)


def attention_rows(q, k, v, batch, seq, heads, dh, rows):
    """Causal softmax(q k^T / sqrt(dh)) v (Sec. 2, Fig. 2b) in fp64 for the given token rows, all
    heads.  q, k, v [batch*seq, heads*dh].  Returns f64 [len(rows), heads*dh]."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    out = np.zeros((len(rows), heads * dh), np.float64)
    rc = lib().oracle_attention_rows(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float), C.c_int64(batch),
                                     C.c_int64(seq), C.c_int64(heads), C.c_int64(dh), _p(rows, C.c_int64),
                                     C.c_int64(len(rows)), _p(out, C.c_double))
    _check(rc, "attention_rows")
    return out
