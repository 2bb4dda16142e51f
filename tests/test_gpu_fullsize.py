"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times.  The oracle cannot produce every output at these sizes in seconds, so:
  * the O(MK) and O(NK) stages (binarize + pack, LN + quant) are compared in full;
  * the O(MNK) matmul is compared on sampled outputs (rows and columns drawn from every tile
    region, plus the corners), computed one by one by the oracle from the GPU's codes (bit-exact
    accumulators) and from the oracle's own codes (end-to-end tolerance)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth
from tests.util import as_f32_np, to_canonical

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FLOAT_TOL_RMS = 1e-3
CODE_FLIP_FRACTION = 1e-4


def sample_points(M, N, count, seed):
    rng = np.random.default_rng(seed)
    ms = rng.integers(0, M, count)
    ns = rng.integers(0, N, count)
    corners = [(0, 0), (0, N - 1), (M - 1, 0), (M - 1, N - 1), (127, 255), (128, 256), (255, 127), (256, 128)]
    for i, (m, n) in enumerate(corners):
        if m < M and n < N:
            ms[i], ns[i] = m, n
    return ms.astype(np.int64), ns.astype(np.int64)


def test_prefill_config_full_size():
    # config 3: x bf16 [8192, 4096] with outliers, W [4096, 4096], per-tensor absmax, y bf16
    M, K, N = 8192, 4096, 4096
    x = synth.make_x(M, K, torch.bfloat16, seed=2, outliers=True)
    W = synth.make_w(N, K, torch.float32, seed=2)
    w_ref = O.binarize(W.numpy())
    w = B.binarize_pack(W.to(DEV), layout=B.PREFILL)
    torch.cuda.synchronize()
    assert (to_canonical(w["W_packed"].cpu().numpy(), B.PREFILL, N, K) == w_ref["bits"]).all()
    assert (w["rowsum"].cpu().numpy() == w_ref["rowsum"]).all()
    q_ref = O.quant_act(as_f32_np(x), gran=O.PER_TENSOR, ln_eps=1e-5)
    xd = x.to(DEV)
    q = B.quant_act(xd, gran=B.PER_TENSOR, ln_eps=1e-5)
    y32 = B.forward(xd, w["W_packed"], w["beta"], N, gran=B.PER_TENSOR, ln_eps=1e-5, layout=B.PREFILL,
                    out_dtype=torch.float32)
    y16 = B.forward(xd, w["W_packed"], w["beta"], N, gran=B.PER_TENSOR, ln_eps=1e-5, layout=B.PREFILL,
                    out_dtype=torch.bfloat16)
    ws = torch.zeros(B.workspace_bytes(B.OP_MATMUL_I32, M, N, K, 1), dtype=torch.uint8, device=DEV)
    acc = B.matmul_i32(q["x_q"], w["W_packed"], N, layout=B.PREFILL, ws=ws)
    assert B.ws_status(ws) == B.OK
    codes = q["x_q"].cpu().numpy()
    diff = codes.astype(np.int32) - q_ref["codes"].astype(np.int32)
    assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) <= CODE_FLIP_FRACTION * diff.size
    assert abs(q["gamma"].item() - q_ref["gamma"][0]) <= 2e-6 * q_ref["gamma"][0]
    ms, ns = sample_points(M, N, 4096, seed=3)
    # accumulators: bit-exact on the GPU's own codes
    acc_s = O.matmul_samples(codes, w_ref["bits"], ms, ns)[:, 0]
    assert (acc.cpu().numpy()[0, ms, ns] == acc_s).all()
    # the layer, sampled: oracle codes -> oracle accumulators -> Eq. 11
    acc_o = O.matmul_samples(q_ref["codes"], w_ref["bits"], ms, ns)[:, 0].astype(np.float64)
    y_o = acc_o * w_ref["beta"][0] * q_ref["gamma"][0] / 128.0
    rms = np.sqrt((y_o ** 2).mean())
    step = w_ref["beta"][0] * q_ref["gamma"][0] / 128.0
    flips = np.abs(diff).sum(axis=1)[ms]
    y_g = y32.cpu().numpy()[ms, ns].astype(np.float64)
    assert (np.abs(y_g - y_o) <= FLOAT_TOL_RMS * rms + flips * step).all()
    assert torch.equal(y16, y32.to(torch.bfloat16))


def test_decode_config_full_size():
    # config 2: x fp16 [1, 4096], W [16384, 4096], per-token absmax, y fp16; every output checked
    K, N = 4096, 16384
    W = synth.make_w(N, K, torch.float32, seed=1)
    w_ref = O.binarize(W.numpy())
    w = B.binarize_pack(W.to(DEV), layout=B.DECODE)
    torch.cuda.synchronize()
    assert (to_canonical(w["W_packed"].cpu().numpy(), B.DECODE, N, K) == w_ref["bits"]).all()
    xs = synth.make_x(4, K, torch.float16, seed=1, outliers=False)
    for i in range(4):
        x = xs[i:i + 1]
        ref = O.forward(as_f32_np(x), w_ref["bits"], w_ref["beta"], gran=O.PER_TOKEN, ln_eps=1e-5)
        y = B.gemv_decode(x.to(DEV), w["W_packed"], w["beta"], N, ln_eps=1e-5, out_dtype=torch.float32)
        y16 = B.gemv_decode(x.to(DEV), w["W_packed"], w["beta"], N, ln_eps=1e-5, out_dtype=torch.float16)
        torch.cuda.synchronize()
        rms = np.sqrt((ref["y"] ** 2).mean())
        step = w_ref["beta"][0] * ref["gamma"][0, 0] / 128.0
        err = np.abs(y.cpu().numpy().astype(np.float64) - ref["y"][0])
        # only a flipped code of the token may explain more than the plain tolerance: it moves every
        # output by one step
        assert err.max() <= FLOAT_TOL_RMS * rms or err.max() <= FLOAT_TOL_RMS * rms + step
        assert torch.equal(y16, y.to(torch.float16))


def test_grouped_down_projection_full_size():
    # config 5: W fp32 [7168, 28672], G = 8 along K; x bf16 [4096, 28672] = ReLU(N(0,1)); eta mode,
    # per-group scalars over all tokens; y bf16
    M, K, N, G = 4096, 28672, 7168, 8
    W = synth.make_w(N, K, torch.float32, seed=4)
    w_ref = O.binarize(W.numpy(), G=G)
    w = B.binarize_pack(W.to(DEV), G=G, layout=B.PREFILL)
    torch.cuda.synchronize()
    assert (to_canonical(w["W_packed"].cpu().numpy(), B.PREFILL, N, K) == w_ref["bits"]).all()
    assert (w["rowsum"].cpu().numpy() == w_ref["rowsum"]).all()
    np.testing.assert_allclose(w["beta"].cpu().numpy(), w_ref["beta"], rtol=1e-6)
    del W
    x = synth.make_x(M, K, torch.bfloat16, seed=4, outliers=False, relu=True)
    q_ref = O.quant_act(as_f32_np(x), G=G, mode=O.ETA, gran=O.PER_TENSOR, ln_eps=1e-5)
    xd = x.to(DEV)
    q = B.quant_act(xd, G=G, mode=B.ETA, gran=B.PER_TENSOR, ln_eps=1e-5)
    y32 = B.forward(xd, w["W_packed"], w["beta"], N, G=G, mode=B.ETA, gran=B.PER_TENSOR, ln_eps=1e-5,
                    layout=B.PREFILL, out_dtype=torch.float32)
    ws = torch.zeros(B.workspace_bytes(B.OP_FORWARD, M, N, K, G), dtype=torch.uint8, device=DEV)
    y16 = B.forward(xd, w["W_packed"], w["beta"], N, G=G, mode=B.ETA, gran=B.PER_TENSOR, ln_eps=1e-5,
                    layout=B.PREFILL, out_dtype=torch.bfloat16, ws=ws)
    assert B.ws_status(ws) == B.OK
    codes = q["x_q"].cpu().numpy()
    diff = codes.astype(np.int32) - q_ref["codes"].astype(np.int32)
    assert np.abs(diff).max() <= 1 and np.count_nonzero(diff) <= CODE_FLIP_FRACTION * diff.size
    np.testing.assert_allclose(q["gamma"].cpu().numpy(), q_ref["gamma"], rtol=2e-6)
    np.testing.assert_allclose(q["eta"].cpu().numpy(), q_ref["eta"], rtol=2e-6, atol=1e-6)
    assert codes.min() >= 0 and codes.max() <= 127
    ms, ns = sample_points(M, N, 2048, seed=5)
    scale = w_ref["beta"] * q_ref["gamma"] / 128.0                                   # [G]
    # stage-wise: Eq. 11 from the GPU's own codes, no slack
    acc_g = O.matmul_samples(codes, w_ref["bits"], ms, ns, G=G).astype(np.float64)   # [S, G]
    y_stage = (acc_g * scale[None, :]).sum(axis=1)
    acc_o = O.matmul_samples(q_ref["codes"], w_ref["bits"], ms, ns, G=G).astype(np.float64)
    y_o = (acc_o * scale[None, :]).sum(axis=1)
    rms = np.sqrt((y_o ** 2).mean())
    y_g = y32.cpu().numpy()[ms, ns].astype(np.float64)
    assert np.abs(y_g - y_stage).max() <= FLOAT_TOL_RMS * rms
    flips = np.abs(diff).sum(axis=1)[ms]
    assert (np.abs(y_g - y_o) <= FLOAT_TOL_RMS * rms + flips * scale.max()).all()
    assert torch.equal(y16, y32.to(torch.bfloat16))
