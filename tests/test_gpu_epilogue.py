"""Output-side options of the dequantising GEMM and N-split groups (Eq. 13 applied to blocks of
output features), both kernels (CUDA-core CANONICAL, tensor-core PREFILL), against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth
from tests.util import as_f32_np, to_canonical

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DT = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


@pytest.mark.parametrize("N,K,NB,G,layout", [
    (384, 512, 3, 1, "prefill"), (384, 512, 3, 2, "prefill"), (96, 256, 3, 1, "canonical"),
    (512, 1024, 4, 2, "decode"), (256, 256, 1, 1, "prefill"),
])
def test_binarize_pack_nsplit(N, K, NB, G, layout):
    lay = {"prefill": B.PREFILL, "canonical": B.CANONICAL, "decode": B.DECODE}[layout]
    W = synth.make_w(N, K, torch.float32, seed=N + NB)
    # give every block its own offset and spread so that a shared alpha / beta would be wrong
    rows = N // NB
    for j in range(NB):
        W[j * rows:(j + 1) * rows] = W[j * rows:(j + 1) * rows] * (1.0 + j) + 0.01 * j
    ref = O.binarize_nsplit(W.numpy(), NB, G=G)
    got = B.binarize_pack_nsplit(W.to(DEV), NB, G=G, layout=lay)
    torch.cuda.synchronize()
    bits = to_canonical(got["W_packed"].cpu().numpy(), lay, N, K)
    assert np.array_equal(bits, ref["bits"])
    assert np.array_equal(got["rowsum"].cpu().numpy(), ref["rowsum"])
    assert np.allclose(got["alpha"].cpu().numpy(), ref["alpha"], rtol=1e-6, atol=1e-9)
    assert np.allclose(got["beta"].cpu().numpy(), ref["beta"], rtol=1e-6, atol=0)


@pytest.mark.parametrize("M,K,N,NB,G,ydtype,mode,relu,residual,wide", [
    (150, 512, 384, 3, 1, "f32", "absmax", False, False, False),     # three beta blocks (Q, K, V shape)
    (150, 512, 384, 3, 2, "f32", "eta", True, True, True),           # all options, grouped, eta correction
    (300, 1024, 768, 3, 1, "f16", "absmax", False, False, True),     # several tiles, fp16 column block output
    (70, 256, 256, 1, 1, "bf16", "absmax", True, True, False),       # ReLU then residual, one block
    (257, 384, 160, 5, 1, "f16", "absmax", False, True, True),       # ragged M and N (canonical only)
])
def test_matmul_dequant_ex(M, K, N, NB, G, ydtype, mode, relu, residual, wide):
    omode = O.ETA if mode == "eta" else O.ABSMAX
    corr = mode == "eta"
    x = synth.make_x(M, K, torch.bfloat16, seed=M + N, outliers=False, relu=(mode == "eta"))
    W = synth.make_w(N, K, torch.float32, seed=K + NB)
    rows = N // NB
    for j in range(NB):
        W[j * rows:(j + 1) * rows] *= (1.0 + 0.5 * j)
    w_ref = O.binarize_nsplit(W.numpy(), NB, G=G)
    q = B.quant_act(x.to(DEV), G=G, mode=omode, gran=B.PER_TOKEN)
    codes = q["x_q"].cpu().numpy()
    acc = O.matmul(codes, w_ref["bits"], G=G)
    gam = q["gamma"].cpu().numpy().astype(np.float64)
    eta = q["eta"].cpu().numpy().astype(np.float64)
    ydt = DT[ydtype]
    g = torch.Generator().manual_seed(5)
    res = torch.randn((M, N + 24 if wide else N), generator=g).to(ydt).to(DEV)[:, :N] if residual else None
    layouts = [B.CANONICAL]
    if rows % 128 == 0 and (K // G) % 128 == 0:
        layouts.append(B.PREFILL)
    for lay in layouts:
        w = B.binarize_pack_nsplit(W.to(DEV), NB, G=G, layout=lay)
        ybuf = torch.zeros((M, N + 40 if wide else N), dtype=ydt, device=DEV)
        y = ybuf[:, 8:8 + N] if wide else ybuf
        B.matmul_dequant_ex(q["x_q"], q["gamma"], w["W_packed"], w["beta"], N, G=G, gran=B.PER_TOKEN, layout=lay,
                            eta=q["eta"], rowsum=w["rowsum"], eta_correction=corr,
                            beta_rows=rows if NB > 1 else 0, relu=relu, residual=res, y=y)
        torch.cuda.synchronize()
        want = O.dequant_nsplit(acc, w["beta"].cpu().numpy().astype(np.float64), gam, gran=O.PER_TOKEN, eta=eta,
                                rowsum=w_ref["rowsum"], eta_correction=corr)
        rms = np.sqrt((want ** 2).mean())
        if relu:
            want = np.maximum(want, 0.0)
        if residual:
            want = want + as_f32_np(res.contiguous()).astype(np.float64)
        got = as_f32_np(y.contiguous()).astype(np.float64)
        tol = 1e-3 * rms + (0 if ydtype == "f32" else np.abs(want) * 2.0 ** (-8 if ydtype == "bf16" else -11))
        assert (np.abs(got - want) <= tol + 1e-7).all(), lay
        if wide:                                          # nothing outside the column block was written
            assert (ybuf[:, :8] == 0).all() and (ybuf[:, 8 + N:] == 0).all()
        # with no options the extended call is the plain one
        if NB == 1 and not relu and not residual and not wide:
            y0 = B.matmul_dequant(q["x_q"], q["gamma"], w["W_packed"], w["beta"].reshape(-1), N, G=G,
                                  gran=B.PER_TOKEN, layout=lay, eta=q["eta"], rowsum=w["rowsum"],
                                  eta_correction=corr, out_dtype=ydt)
            assert torch.equal(y0, y)


def test_epilogue_argument_checks():
    M, K, N = 32, 256, 256
    x = synth.make_x(M, K, torch.bfloat16, seed=1, outliers=False).to(DEV)
    W = synth.make_w(N, K, torch.float32, seed=1).to(DEV)
    w = B.binarize_pack(W, layout=B.CANONICAL)
    q = B.quant_act(x)
    with pytest.raises(B.BitLinearError) as e:          # beta block that does not divide N
        B.matmul_dequant_ex(q["x_q"], q["gamma"], w["W_packed"], w["beta"], N, beta_rows=96)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.BitLinearError) as e:          # beta block not a multiple of 32
        B.matmul_dequant_ex(q["x_q"], q["gamma"], w["W_packed"], w["beta"], N, beta_rows=16)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.BitLinearError) as e:          # NB must divide N
        B.binarize_pack_nsplit(W, 7)
    assert e.value.code == B.ERR_SHAPE


@pytest.mark.parametrize("M,K,N,G,wdtype,mode,gran", [
    (200, 512, 384, 1, "f32", "absmax", "tensor"),     # tensor-core path
    (64, 1024, 256, 2, "bf16", "eta", "token"),        # grouped, 16-bit latent weights
    (33, 1000, 70, 5, "f32", "eta", "tensor"),         # shape only the CUDA-core kernel takes
])
def test_forward_latent_is_pack_then_forward(M, K, N, G, wdtype, mode, gran):
    omode = O.ETA if mode == "eta" else O.ABSMAX
    ogran = B.PER_TOKEN if gran == "token" else B.PER_TENSOR
    x = synth.make_x(M, K, torch.bfloat16, seed=M + K, outliers=False, relu=(mode == "eta")).to(DEV)
    W = synth.make_w(N, K, DT[wdtype], seed=N).to(DEV)
    corr = mode == "eta"
    got = B.forward_latent(x, W, G=G, mode=omode, gran=ogran, eta_correction=corr, out_dtype=torch.float32)
    lay = B.PREFILL if (K // G) % 128 == 0 else B.CANONICAL
    w = B.binarize_pack(W, G=G, layout=lay)
    want = B.forward(x, w["W_packed"], w["beta"], N, G=G, mode=omode, gran=ogran, layout=lay, rowsum=w["rowsum"],
                     eta_correction=corr, out_dtype=torch.float32)
    assert torch.equal(got["y"], want)
    assert torch.equal(got["alpha"], w["alpha"]) and torch.equal(got["beta"], w["beta"])
    # and against the oracle on the same latent weights
    w_ref = O.binarize(W.float().cpu().numpy(), G=G)
    ref = O.forward(as_f32_np(x), w_ref["bits"], w_ref["beta"], G=G, mode=omode,
                    gran=O.PER_TOKEN if gran == "token" else O.PER_TENSOR, ln_eps=1e-5, rowsum=w_ref["rowsum"],
                    eta_correction=corr)
    rms = np.sqrt((ref["y"] ** 2).mean())
    err = np.abs(got["y"].cpu().numpy().astype(np.float64) - ref["y"])
    # one quantisation step of slack per code of the token that differs from the oracle's (rounding
    # ties; the codes themselves are checked in the quantisation tests)
    q = B.quant_act(x, G=G, mode=omode, gran=ogran)
    flips = np.abs(q["x_q"].cpu().numpy().astype(np.int32) - ref["codes"].astype(np.int32)).sum(axis=1)
    gam = ref["gamma"] if gran == "token" else np.broadcast_to(ref["gamma"], (M, G))
    step = (w_ref["beta"][None, :] * gam / 128.0).max(axis=1)
    assert (err <= 1e-3 * rms + (flips * step)[:, None]).all()
