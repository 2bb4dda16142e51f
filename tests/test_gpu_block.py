"""Decoder block (Sec. 2, Fig. 2b) on the GPU, stage by stage against the oracle.

The block chains six BitLinear layers through an fp16 attention core and fp16 residual adds, so a
double-precision oracle fed the block's own input drifts away from the fp16 path long before the
last layer.  Parity is therefore teacher-forced: every stage is checked against the oracle applied
to the input that stage actually received on the GPU (read back from the caller-visible
intermediate buffers):
  * each BitLinear: int8 codes within +-1 on <= 1e-4 of the elements; sampled outputs within 1e-3 of
    the output RMS of the oracle's Eq. 11 on the GPU's own codes, plus the fp16 rounding of the store;
  * attention: sampled rows against the fp64 definition within fp16 tolerance;
  * residual adds and ReLU (run in the GEMM epilogues): bit-exact against the fp32 projection with
    the same operation applied and one rounding to fp16;
  * Q, K, V as one [3d, d] GEMM and as three GEMMs write the same bits."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth
from tests.test_gpu_parity import check_codes
from tests.util import as_f32_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_block(d, ffn, seed):
    shapes = dict(q=(d, d), k=(d, d), v=(d, d), o=(d, d), up=(ffn, d), down=(d, ffn))
    W = {n: synth.make_w(N, K, torch.float32, seed=seed + 17 * i) for i, (n, (N, K)) in enumerate(shapes.items())}
    ref = {n: O.binarize(w.numpy()) for n, w in W.items()}
    gpu = {n: B.binarize_pack(w.to(DEV), layout=B.PREFILL) for n, w in W.items()}
    return ref, gpu


def check_bitlinear_stage(x_in, y_out, w_ref, mode, samples, seed):
    """x_in fp16 [T,K] (GPU's stage input), y_out fp16 [T,N] (GPU's stage output before any add/ReLU)."""
    x = as_f32_np(x_in)
    T, K = x.shape
    N = w_ref["bits"].shape[0]
    omode = O.ETA if mode == "eta" else O.ABSMAX
    q_ref = O.quant_act(x, mode=omode, gran=O.PER_TOKEN, ln_eps=1e-5)
    q = B.quant_act(x_in, mode=omode, gran=B.PER_TOKEN, ln_eps=1e-5)
    codes = q["x_q"].cpu().numpy()
    # exact ties of the eta form (rational pre-rounding values) are valid either way; the rest is counted
    check_codes(codes, q_ref["codes"], x=x, G=1, eta_per_token=(mode == "eta"))
    rng = np.random.default_rng(seed)
    ms, ns = rng.integers(0, T, samples), rng.integers(0, N, samples)
    acc = O.matmul_samples(codes, w_ref["bits"], ms, ns)[:, 0].astype(np.float64)
    gam = q["gamma"].cpu().numpy().astype(np.float64).reshape(-1)
    y_stage = acc * w_ref["beta"][0] * gam[ms] / 128.0
    y_gpu = y_out.cpu().float().numpy()[ms, ns].astype(np.float64)
    rms = np.sqrt((y_stage ** 2).mean())
    # fp32 result rounded to fp16 on store: half an ulp of fp16 (2^-11 relative) on top of the tolerance
    assert (np.abs(y_gpu - y_stage) <= 1e-3 * rms + np.abs(y_stage) * 2.0 ** -11 + 1e-7).all()


def run_block(batch, seq, heads, ffn, seed, attn_rows, fused_qkv):
    d = heads * 128
    T = batch * seq
    x = synth.make_x(T, d, torch.float16, seed=seed, outliers=False).to(DEV)
    w_ref, w_gpu = make_block(d, ffn, seed)
    if fused_qkv:
        w_gpu = B.fuse_qkv_weights(w_gpu)
    out = B.block_forward(x, w_gpu, batch, seq, heads, ffn, fused_qkv=fused_qkv)
    assert B.ws_status(out["ws"]) == B.OK

    def proj32(src, name, N, mode=B.ABSMAX):
        return B.forward(src, w_gpu[name]["W_packed"], w_gpu[name]["beta"], N, mode=mode, gran=B.PER_TOKEN,
                         layout=B.PREFILL, out_dtype=torch.float32)
    # stages that write their BitLinear output straight to an inspectable buffer
    for name, src, dst in (("q", x, out["q"]), ("k", x, out["k"]), ("v", x, out["v"])):
        check_bitlinear_stage(src, dst, w_ref[name], "absmax", 2000, seed)
    # attention core on the GPU's q, k, v
    rows = np.unique(np.concatenate([[0, 1, 63, 64, seq - 1, T - seq, T - 1],
                                     np.random.default_rng(seed).integers(0, T, attn_rows)])).astype(np.int64)
    rows = rows[rows < T]
    a_ref = O.attention_rows(as_f32_np(out["q"].contiguous()), as_f32_np(out["k"].contiguous()),
                             as_f32_np(out["v"].contiguous()), batch, seq, heads, 128, rows)
    a_gpu = out["a"].cpu().float().numpy()[rows].astype(np.float64)
    scale = np.abs(a_ref).max()
    assert np.abs(a_gpu - a_ref).max() <= 4e-3 * scale          # fp16 probabilities and outputs
    assert np.sqrt(((a_gpu - a_ref) ** 2).mean()) <= 1e-3 * scale
    # O projection + residual: h = x + BitLinear_O(a); recompute the projection alone for the stage check
    o_proj = proj32(out["a"], "o", d)
    check_bitlinear_stage(out["a"], o_proj.half(), w_ref["o"], "absmax", 2000, seed + 1)
    assert torch.equal(out["h"], (o_proj + x.float()).half())       # fp32 add, one rounding, bit for bit
    # up projection + ReLU
    up = proj32(out["h"], "up", ffn)
    check_bitlinear_stage(out["h"], up.half(), w_ref["up"], "absmax", 2000, seed + 2)
    assert torch.equal(out["u"], torch.relu(up).half())
    # down projection (eta form on the ReLU output) + residual
    down = proj32(out["u"], "down", d, mode=B.ETA)
    check_bitlinear_stage(out["u"], down.half(), w_ref["down"], "eta", 2000, seed + 3)
    assert torch.equal(out["y"], (down + out["h"].float()).half())
    assert torch.isfinite(out["y"]).all()
    return out


def test_block_small():
    a = run_block(batch=2, seq=128, heads=2, ffn=1024, seed=50, attn_rows=64, fused_qkv=False)
    b = run_block(batch=2, seq=128, heads=2, ffn=1024, seed=50, attn_rows=64, fused_qkv=True)
    for name in ("q", "k", "v", "a", "h", "u", "y"):
        assert torch.equal(a[name], b[name]), name


def test_block_config4_full_size():
    # d = 2048, 16 heads, FFN 8192, batch 4 x seq 2048, in the layout the benchmark times
    run_block(batch=4, seq=2048, heads=16, ffn=8192, seed=60, attn_rows=48, fused_qkv=True)


@pytest.mark.parametrize("batch,seq,heads", [(1, 256, 3), (2, 192, 2), (3, 64, 1), (1, 448, 1)])
def test_attention_alone_against_definition(batch, seq, heads):
    T, d = batch * seq, heads * 128
    g = torch.Generator().manual_seed(7)
    qkv = (torch.randn((T, 3 * d), generator=g) * 1.5).to(torch.float16).to(DEV)     # one fused buffer
    q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
    o = B.attention_causal(q, k, v, batch, seq, heads)
    rows = np.arange(T, dtype=np.int64)
    ref = O.attention_rows(as_f32_np(q.contiguous()), as_f32_np(k.contiguous()), as_f32_np(v.contiguous()),
                           batch, seq, heads, 128, rows)
    err = np.abs(o.cpu().float().numpy().astype(np.float64) - ref)
    assert err.max() <= 4e-3 * np.abs(ref).max()
    for bi in range(batch):                                                          # token 0 sees only itself
        assert torch.equal(o[bi * seq], v[bi * seq])
