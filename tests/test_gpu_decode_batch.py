"""Small-batch decode (M tokens sharing one pass over the DECODE-packed weights) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth
from tests.test_gpu_parity import check_codes, count_exact_ties
from tests.util import as_f32_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DT = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


@pytest.mark.parametrize("M,K,N,G,dtype,mode,relu", [
    (8, 4096, 16384, 1, "f16", "absmax", False),     # config c2's layer with a full batch of 8
    (1, 256, 16, 1, "f32", "absmax", False),         # smallest shape, one token
    (3, 1024, 48, 2, "bf16", "eta", True),           # groups along K, eta form
    (13, 2048, 160, 1, "f16", "absmax", False),      # two launches, ragged second batch of 5
    (5, 8192, 64, 1, "bf16", "absmax", False),       # K above two register batches of weights
    (2, 7168, 112, 7, "bf16", "eta", True),          # seven groups of 1024
    (8, 16384, 48, 2, "f16", "absmax", False),       # tokens too long to stage in shared memory: read from L2
    (7, 256, 32, 1, "f32", "absmax", False),         # one K block: the second warp of every pair has no work
])
def test_gemv_decode_batch(M, K, N, G, dtype, mode, relu):
    run_batch_case(B.gemv_decode_batch, M, K, N, G, dtype, mode, relu)


# The same call with a workspace: tokens quantised by a kernel of their own, the product on the
# tcgen05 tensor cores for G == 1 without the eta correction (other cases: the kernel above).
@pytest.mark.parametrize("M,K,N,G,dtype,mode,relu", [
    (8, 4096, 16384, 1, "f16", "absmax", False),     # config c2's layer, 8 tokens: quantising kernel + bit-plane kernel
    (9, 4096, 16384, 1, "f16", "absmax", False),     # 9 tokens: quantising kernel + tensor-core kernel, 148 CTAs of 111 rows
    (16, 4096, 16384, 1, "bf16", "absmax", False),   # a full pass of 16 tokens
    (2, 256, 16, 1, "f32", "absmax", False),         # smallest shape
    (12, 256, 16, 1, "f32", "absmax", False),        # the same on the tensor cores: one chunk (half a slot), CTAs of one row
    (9, 1024, 48, 1, "bf16", "eta", True),           # eta form without the correction; the second half of the codes is used
    (37, 2048, 160, 1, "f16", "absmax", False),      # passes of 32 tokens: a full one and a ragged one of 5
    (32, 4096, 16384, 1, "f16", "absmax", False),    # one pass of 32 tokens at config c2's layer
    (17, 6144, 256, 1, "bf16", "eta", True),         # the largest K with 32 tokens per pass; 17 tokens: three of four token blocks
    (20, 8192, 64, 1, "f16", "absmax", False),       # more than 16 tokens with K too large for 32 per pass: two passes of 16
    (11, 8192, 20480, 1, "bf16", "absmax", False),   # 160 CTAs of 128 rows: more CTAs than SMs
    (10, 12288, 64, 1, "f32", "absmax", False),      # the largest K: six pieces per thread of the quantiser
    (5, 12288, 64, 1, "f32", "eta", True),           # the same with the bit-plane kernel
    (10, 768, 3072, 1, "f32", "absmax", False),      # 125M-shaped: an odd number of chunks
    (4, 4096, 1024, 1, "f16", "absmax", False),      # few tokens, few tiles
    (9, 1024, 48, 2, "bf16", "eta", True),           # groups: the kernel without a workspace
    (8, 16384, 48, 1, "f16", "absmax", False),       # K too large for the quantising kernel: likewise
])
def test_gemv_decode_batch_ws(M, K, N, G, dtype, mode, relu):
    ws = torch.empty(B.workspace_bytes(B.OP_GEMV_DECODE_BATCH, M, N, K, G) + 256, dtype=torch.uint8, device=DEV)

    def call(*args, **kw):
        return B.gemv_decode_batch_ws(*args, ws=ws, **kw)
    # every token is quantised by the same kernel whichever product kernel follows: same bits for any batch
    run_batch_case(call, M, K, N, G, dtype, mode, relu)
    assert B.ws_status(ws) == B.OK


def run_batch_case(gemv_decode_batch, M, K, N, G, dtype, mode, relu, same_bits_from=2):
    x = synth.make_x(M, K, DT[dtype], seed=K + N + M, outliers=False, relu=relu)
    W = synth.make_w(N, K, torch.float32, seed=K)
    omode = O.ETA if mode == "eta" else O.ABSMAX
    w_ref = O.binarize(W.numpy(), G=G)
    w_gpu = B.binarize_pack(W.to(DEV), G=G, layout=B.DECODE)
    torch.cuda.synchronize()
    xd = x.to(DEV)
    # The kernel quantises the tokens itself and its codes cannot be read back, so the comparison
    # allows what the quantising kernels are allowed: a different neighbour at a rounding tie,
    # exact rational ties of the per-token eta form (either neighbour is valid) and, as for every
    # quantising kernel here, at most 1e-4 of the elements (at least one).  Each such code moves a
    # token's outputs by one quantisation step.
    q = B.quant_act(xd, G=G, mode=omode, gran=B.PER_TOKEN, ln_eps=1e-5)
    ref_q = O.quant_act(as_f32_np(x), G=G, mode=omode, gran=O.PER_TOKEN, ln_eps=1e-5)
    codes = q["x_q"].cpu().numpy()
    check_codes(codes, ref_q["codes"], x=as_f32_np(x), G=G, eta_per_token=(mode == "eta"))
    acc = O.matmul(codes, w_ref["bits"], G=G)
    for corr in ([False, True] if mode == "eta" else [False]):
        y = gemv_decode_batch(xd, w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, ln_eps=1e-5,
                              rowsum=w_gpu["rowsum"], eta_correction=corr, out_dtype=torch.float32)
        torch.cuda.synchronize()
        want = O.dequant(acc, w_gpu["beta"].cpu().numpy().astype(np.float64),
                         q["gamma"].cpu().numpy().astype(np.float64), gran=O.PER_TOKEN,
                         eta=q["eta"].cpu().numpy().astype(np.float64), rowsum=w_ref["rowsum"], eta_correction=corr)
        rms = np.sqrt((want ** 2).mean())
        gam = q["gamma"].cpu().numpy().astype(np.float64).reshape(M, G)
        step = (w_gpu["beta"].cpu().numpy().astype(np.float64)[None, :] * gam / 128.0).max(axis=1)
        ties = np.array([count_exact_ties(as_f32_np(x)[m], G) if mode == "eta" else 0 for m in range(M)])
        slack = ((max(1, int(1e-4 * K)) + ties) * step)[:, None]
        err = np.abs(y.cpu().numpy().astype(np.float64) - want)
        assert (err <= 1e-3 * rms + slack).all()
        # the typical element needs no slack (an exact tie that went the other way moves every
        # output of its token by one step, so tokens with such ties are left out)
        if (ties == 0).any():
            assert np.median(err[ties == 0]) <= 1e-3 * rms
    # 16-bit output is the rounding of the fp32 one
    y32 = gemv_decode_batch(xd, w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, out_dtype=torch.float32)
    if dtype != "f32":
        y16 = gemv_decode_batch(xd, w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, out_dtype=DT[dtype])
        assert torch.equal(y16, y32.to(DT[dtype]))
    # a token's result does not depend on what else is in the batch: the last tokens as a (smallest) batch of
    # their own give the same bits (a single token takes the single-token kernel, whose sums run in
    # another order: same codes up to the tolerated ties, gamma to the last bit or so)
    if M > same_bits_from:
        sub = same_bits_from
        y_sub = gemv_decode_batch(xd[M - sub:M].contiguous(), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode,
                                  out_dtype=torch.float32)
        assert torch.equal(y_sub, y32[M - sub:M])
    if M > 1:
        y_one = gemv_decode_batch(xd[M - 1:M].contiguous(), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode,
                                  out_dtype=torch.float32)
        d = np.abs(y_one[0].cpu().numpy().astype(np.float64) - y32[M - 1].cpu().numpy().astype(np.float64))
        assert (d <= 1e-3 * rms + slack[M - 1]).all()


def test_gemv_decode_batch_integer_definition_exactly():
    # LN skipped and gamma planted at 128 (an element equal to 128 in every token): the codes are
    # the inputs themselves, so y must equal acc * beta as computed by the oracle's integer matmul.
    M, K, N = 6, 1024, 96
    codes = synth.make_codes(M, K, seed=9)
    x = codes.to(torch.float32)
    x[:, 0] = 128.0                                                  # gamma = 128, its code clips to 127
    W = synth.make_w(N, K, torch.float32, seed=9)
    w_ref = O.binarize(W.numpy())
    w_gpu = B.binarize_pack(W.to(DEV), layout=B.DECODE)
    torch.cuda.synchronize()
    y = B.gemv_decode_batch(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, ln_eps=-1.0, out_dtype=torch.float32)
    c = codes.numpy().copy()
    c[:, 0] = 127
    acc = O.matmul(c, w_ref["bits"])[0].astype(np.float64)
    want = (acc * float(w_gpu["beta"][0])).astype(np.float32)
    assert np.allclose(y.cpu().numpy(), want, rtol=3e-7, atol=0)


@pytest.mark.parametrize("M", [6, 12, 32])
def test_gemv_decode_batch_ws_integer_definition_exactly(M):
    # As above through the workspace form: 6 tokens take the bit-plane kernel, 12 and 32 the tensor cores
    # (one pass of 16, one of 32).  With LN skipped and gamma planted at 128 the codes are the inputs, so y
    # must be the oracle's integer matmul times beta, to the last bit of the one float multiplication.
    K, N = 1024, 96
    codes = synth.make_codes(M, K, seed=9 + M)
    x = codes.to(torch.float32)
    x[:, 0] = 128.0                                                  # gamma = 128, its code clips to 127
    W = synth.make_w(N, K, torch.float32, seed=9)
    w_ref = O.binarize(W.numpy())
    w_gpu = B.binarize_pack(W.to(DEV), layout=B.DECODE)
    torch.cuda.synchronize()
    ws = torch.empty(B.workspace_bytes(B.OP_GEMV_DECODE_BATCH, M, N, K, 1), dtype=torch.uint8, device=DEV)
    y = B.gemv_decode_batch_ws(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, ln_eps=-1.0, out_dtype=torch.float32, ws=ws)
    assert B.ws_status(ws) == B.OK
    c = codes.numpy().copy()
    c[:, 0] = 127
    acc = O.matmul(c, w_ref["bits"])[0].astype(np.float64)
    want = (acc * float(w_gpu["beta"][0])).astype(np.float32)
    assert np.allclose(y.cpu().numpy(), want, rtol=3e-7, atol=0)


def test_gemv_decode_batch_argument_checks():
    x = torch.zeros((2, 384), dtype=torch.float16, device=DEV)
    w = torch.zeros(64, dtype=torch.uint8, device=DEV)
    beta = torch.ones(1, device=DEV)
    with pytest.raises(B.BitLinearError) as e:                      # K not a multiple of 256
        B.gemv_decode_batch(x, w, beta, 16)
    assert e.value.code == B.ERR_SHAPE
