"""GPU parity: every C-ABI entry point against the CPU oracle, element by element, on the same
seeded inputs.  Bars: packed bits, row sums and int32 accumulators bit-exact; int8 codes may
differ by +-1 on at most 1e-4 of the elements (fp32 vs fp64 rounding ties); float outputs
within 1e-3 of the output RMS (plus one quantisation step per flipped code of that token, and
with no allowance at all when the oracle is fed the GPU's own codes)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import synth
from tests.util import as_f32_np, to_canonical

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
DT = synth.TORCH_DTYPES
CODE_FLIP_FRACTION = 1e-4
FLOAT_TOL_RMS = 1e-3


def exact_tie_per_token_eta(x_row_seg, k):
    """Per-token eta mode in exact arithmetic: LN cancels and the pre-rounding value is
    (x - min) * 128 / (max - min), a rational number.  True when that is exactly a half-integer,
    i.e. both neighbouring codes are valid outcomes of round-half-to-even under rounding noise."""
    from fractions import Fraction
    lo, hi = Fraction(float(x_row_seg.min())), Fraction(float(x_row_seg.max()))
    if hi == lo:
        return False
    v = (Fraction(float(x_row_seg[k])) - lo) * 128 / (hi - lo)
    return v.denominator == 2


def count_exact_ties(x_row, G):
    """Number of elements of one token that are exact ties in per-token eta mode."""
    Kg = x_row.shape[0] // G
    return sum(exact_tie_per_token_eta(x_row[g * Kg:(g + 1) * Kg], k) for g in range(G) for k in range(Kg))


def self_scaled_rows(x, G, ln_eps=1e-5):
    """Per-tensor eta mode: the (token, group) segments that hold both the minimum and the maximum
    of x^ over their group's scope.  For such a segment LN cancels in (x^ - eta) / gamma exactly as
    in the per-token form, so its elements can be exact rational ties as well."""
    M, K = x.shape
    Kg = K // G
    out = set()
    for g in range(G):
        seg = x[:, g * Kg:(g + 1) * Kg].astype(np.float64)
        xh = (seg - seg.mean(axis=1, keepdims=True)) / np.sqrt(seg.var(axis=1, keepdims=True) + ln_eps)
        m_lo, m_hi = np.unravel_index(xh.argmin(), xh.shape)[0], np.unravel_index(xh.argmax(), xh.shape)[0]
        if m_lo == m_hi:
            out.add((int(m_lo), g))
    return out


TIE_EXEMPT_FRACTION = 1e-2      # cap on the elements that may be excused as exact ties
TIE_LOG = []                     # (elements, differing, excused as exact ties, of those at the even neighbour)


def check_codes(gpu_codes, ref_codes, x=None, G=1, eta_per_token=False, eta_per_tensor=False):
    """+-1 on at most 1e-4 of the elements.  Elements whose exact value is a mathematical tie
    (decidable where LN cancels and the value is rational: the per-token eta form, and in the
    per-tensor eta form the segment that holds both extremes of its scope) are valid either way
    and are not counted against that bar; their number is capped (1e-2 of the elements, at least
    4), recorded in TIE_LOG and printed, together with how many of them the GPU sent to the even
    neighbour (what round-half-to-even does when the tie survives the arithmetic).  Such ties are
    not rare with 16-bit inputs: when the segment's range max - min has few mantissa bits, every
    input whose last mantissa bit falls right is one (0.3 % of the elements in one case of the
    seeded sweep, half of which the kernel sent to the even neighbour: LN's rounding noise decides)."""
    diff = gpu_codes.astype(np.int32) - ref_codes.astype(np.int32)
    assert np.abs(diff).max() <= 1, "a code differs by more than one step"
    counted = excused = to_even = 0
    rows = self_scaled_rows(x, G) if (eta_per_tensor and x is not None and np.count_nonzero(diff)) else set()
    for m, k in zip(*np.nonzero(diff)):
        if x is not None and (eta_per_token or rows):
            Kg = x.shape[1] // G
            g = k // Kg
            if (eta_per_token or (int(m), int(g)) in rows) and \
                    exact_tie_per_token_eta(x[m, g * Kg:(g + 1) * Kg], k - g * Kg):
                excused += 1
                to_even += int(gpu_codes[m, k]) % 2 == 0
                continue
        counted += 1
    TIE_LOG.append((diff.size, int(np.count_nonzero(diff)), excused, to_even))
    if excused:
        print(f"check_codes: {excused} of {diff.size} elements excused as exact ties "
              f"({to_even} at the even neighbour), {counted} counted")
    assert excused <= max(4, int(TIE_EXEMPT_FRACTION * diff.size)), \
        f"{excused} of {diff.size} code differences claimed as exact ties"
    assert counted <= max(1, int(CODE_FLIP_FRACTION * diff.size)), f"{counted} of {diff.size} codes differ"
    return diff


def check_scalars(gpu, ref, rel=2e-6, abs_=1e-6):
    gpu = np.asarray(gpu, np.float64).reshape(-1)
    ref = np.asarray(ref, np.float64).reshape(-1)
    assert gpu.shape == ref.shape
    assert (np.abs(gpu - ref) <= rel * np.abs(ref) + abs_).all(), (gpu[:4], ref[:4])


# ---------------------------------------------------------------- step 3: binarize + pack

@pytest.mark.parametrize("N,K,G,dtype", [
    (3072, 768, 1, "f32"),        # config c1
    (37, 40, 1, "f32"),           # ragged: K % 32 != 0, N not a multiple of the rows per block
    (64, 1000, 5, "f32"),         # K_g = 200
    (130, 1024, 8, "bf16"),
    (257, 2048, 4, "f16"),
    (1, 8, 1, "f32"),
    (3, 304, 1, "f32"),           # alpha = -4.7e-7: the sum cancels to 1e-5 of sum |W|
    (64, 3000, 3, "f32"),
])
def test_binarize_pack_canonical(N, K, G, dtype):
    W = synth.make_w(N, K, DT[dtype], seed=N + K)
    if G > 1:   # give the groups different means so a whole-tensor alpha would be wrong
        W = (W.float() + torch.arange(G).repeat_interleave(K // G) * 0.003).to(DT[dtype])
    ref = O.binarize(as_f32_np(W), G=G)
    out = B.binarize_pack(W.to(DEV), G=G, layout=B.CANONICAL)
    torch.cuda.synchronize()
    bits = out["W_packed"].cpu().numpy()[: N * K // 8].reshape(N, K // 8)
    assert (bits == ref["bits"]).all()
    assert (out["rowsum"].cpu().numpy() == ref["rowsum"]).all()
    # alpha decides bits, so it must be the fp64 mean to float rounding even where the sum cancels
    # to a millionth of the weights' scale (sums with fp32 inside a chunk were off by 7e-6 there)
    assert np.allclose(out["alpha"].cpu().numpy().astype(np.float64), ref["alpha"], rtol=1.5e-7, atol=1e-30)
    check_scalars(out["beta"].cpu().numpy(), ref["beta"], rel=1e-6, abs_=0)


@pytest.mark.parametrize("layout,N,K,G", [(B.PREFILL, 256, 512, 1), (B.PREFILL, 100, 384, 3),
                                          (B.PREFILL, 300, 1024, 2), (B.DECODE, 64, 1024, 1),
                                          (B.DECODE, 48, 512, 2)])
def test_binarize_pack_private_layouts_hold_the_same_bits(layout, N, K, G):
    W = synth.make_w(N, K, torch.float32, seed=7 * N + K)
    ref = O.binarize(as_f32_np(W), G=G)
    out = B.binarize_pack(W.to(DEV), G=G, layout=layout)
    torch.cuda.synchronize()
    canon = to_canonical(out["W_packed"].cpu().numpy(), layout, N, K)
    assert (canon == ref["bits"]).all()
    assert (out["rowsum"].cpu().numpy() == ref["rowsum"]).all()


def test_binarize_pack_sign_tie_and_alpha_in():
    # entries equal to alpha must pack to 0 bits (Sign(0) = -1)
    W = torch.tensor([[-2, -1, 0, 0, 1, 2, 0, 0], [3, 0, -3, 0, 0, 0, 1, -1]], dtype=torch.float32)
    out = B.binarize_pack(W.to(DEV))
    assert out["alpha"].item() == 0.0
    assert out["W_packed"].cpu().numpy()[:2].tolist() == O.binarize(W.numpy())["bits"].reshape(-1).tolist()
    # forced alpha isolates the sign+pack step
    W = synth.make_w(64, 256, torch.float32, seed=3)
    a = torch.tensor([0.004], dtype=torch.float32)
    ref = O.binarize(W.numpy(), alpha_in=a.double().numpy())
    out = B.binarize_pack(W.to(DEV), alpha_in=a.to(DEV))
    assert (out["W_packed"].cpu().numpy()[: 64 * 32].reshape(64, 32) == ref["bits"]).all()
    assert out["alpha"].item() == a.item()


def test_binarize_pack_is_deterministic():
    W = synth.make_w(512, 2048, torch.float32, seed=11).to(DEV)
    a = B.binarize_pack(W, G=2)
    b = B.binarize_pack(W, G=2)
    assert torch.equal(a["W_packed"], b["W_packed"]) and torch.equal(a["alpha"], b["alpha"])
    assert torch.equal(a["beta"], b["beta"])


# ---------------------------------------------------------------- steps 1-2: LN + quant

QUANT_CASES = [
    # M, K, G, dtype, mode, gran, outliers, relu
    (64, 768, 1, "f32", "absmax", "tensor", True, False),    # c1
    (64, 768, 1, "f32", "absmax", "token", True, False),
    (1, 4096, 1, "f16", "absmax", "token", False, False),    # c2
    (300, 4096, 1, "bf16", "absmax", "tensor", True, False), # c3-shaped rows
    (33, 1000, 5, "f32", "eta", "token", False, True),       # ragged K_g = 200
    (33, 1000, 5, "f32", "eta", "tensor", False, True),
    (17, 28672, 8, "bf16", "eta", "tensor", False, True),    # c5-shaped rows
    (17, 28672, 8, "bf16", "absmax", "token", True, False),
    (5, 8, 1, "f32", "absmax", "token", False, False),
    (9, 8192, 1, "bf16", "absmax", "token", True, False),    # 16 KB segments: one slot per warp
    (9, 8192, 1, "f16", "eta", "tensor", False, True),
    (7, 4096, 1, "f32", "absmax", "tensor", True, False),
    (3, 2048, 1, "f32", "eta", "token", False, True),        # the longest fp32 segment with two slots per warp
    (40, 8192, 1, "f16", "eta", "token", False, True),       # more 16 KB segments than warps in a CTA
    (5, 16384, 1, "bf16", "absmax", "token", True, False),   # longer than a warp's staging area: CTA path
    (5, 16384, 1, "bf16", "eta", "tensor", False, True),
    (4, 12288, 1, "f32", "absmax", "token", False, False),   # CTA path with exactly 48 KB of dynamic shared memory
    (4, 12288, 1, "f32", "eta", "tensor", False, True),
    # per-tensor scope in one kernel: segments per CTA below, at and above what stays in shared memory
    (1, 4096, 1, "bf16", "absmax", "tensor", False, False),
    (3600, 512, 1, "bf16", "eta", "tensor", False, True),    # 24-25 segments per CTA
    (5000, 512, 2, "f16", "absmax", "tensor", True, False),  # 67-68 segments per CTA, two groups
]


@pytest.mark.parametrize("M,K,G,dtype,mode,gran,outliers,relu", QUANT_CASES)
def test_quant_act(M, K, G, dtype, mode, gran, outliers, relu):
    x = synth.make_x(M, K, DT[dtype], seed=M * 7 + K, outliers=outliers, relu=relu)
    omode = O.ETA if mode == "eta" else O.ABSMAX
    ogran = O.PER_TOKEN if gran == "token" else O.PER_TENSOR
    ref = O.quant_act(as_f32_np(x), G=G, mode=omode, gran=ogran, ln_eps=1e-5)
    out = B.quant_act(x.to(DEV), G=G, mode=omode, gran=ogran, ln_eps=1e-5)
    torch.cuda.synchronize()
    check_codes(out["x_q"].cpu().numpy(), ref["codes"], x=as_f32_np(x), G=G,
                eta_per_token=(mode == "eta" and gran == "token"),
                eta_per_tensor=(mode == "eta" and gran == "tensor"))
    check_scalars(out["gamma"].cpu().numpy(), ref["gamma"])
    if mode == "eta":
        check_scalars(out["eta"].cpu().numpy(), ref["eta"])
        assert out["x_q"].min().item() >= 0
    assert out["x_q"].abs().max().item() <= 127
    if gran == "token":
        # With a workspace the segments arrive by bulk copies whose wait reports through its first
        # word; without one, by per-lane copies.  Same values either way, and the word stays clear.
        ws = torch.full((256,), 0xA5, dtype=torch.uint8, device=DEV)
        with_ws = B.quant_act(x.to(DEV), G=G, mode=omode, gran=ogran, ln_eps=1e-5, ws=ws)
        assert B.ws_status(ws) == B.OK                 # every per-token kernel clears (or leaves clear) the word
        no_ws = B.quant_act(x.to(DEV), G=G, mode=omode, gran=ogran, ln_eps=1e-5, ws=False)
        torch.cuda.synchronize()
        for key in ("x_q", "gamma", "eta"):
            assert torch.equal(out[key], with_ws[key]) and torch.equal(out[key], no_ws[key])


def test_quant_act_per_tensor_replayed_from_a_graph_on_new_data():
    # The fused per-tensor kernel's CTAs meet over tags in the workspace.  A captured graph replays the
    # same launch parameters, so what a CTA publishes must still differ from one replay to the next (a
    # generation count in the workspace): otherwise the second replay would take the first one's tags
    # for arrivals and compute gamma from stale or half-written partial extremes.
    M, K = 600, 4096
    xa = synth.make_x(M, K, torch.bfloat16, seed=5, outliers=True)
    xb = (synth.make_x(M, K, torch.bfloat16, seed=6, outliers=False).float() * 3.0 + 0.5).to(torch.bfloat16)
    x = xa.to(DEV).clone()
    out = dict(x_q=torch.empty((M, K), dtype=torch.int8, device=DEV), gamma=torch.empty(1, device=DEV),
               eta=torch.empty(1, device=DEV))
    ws = torch.empty(B.workspace_bytes(B.OP_QUANT_ACT, M, 1, K, 1), dtype=torch.uint8, device=DEV)
    B.quant_act(x, gran=B.PER_TENSOR, out=out, ws=ws)                # warm-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        B.quant_act(x, gran=B.PER_TENSOR, out=out, ws=ws)
    for host in (xa, xb, xa, xb):
        x.copy_(host.to(DEV))
        graph.replay()
        torch.cuda.synchronize()
        assert B.ws_status(ws) == B.OK
        ref = O.quant_act(as_f32_np(host), G=1, mode=O.ABSMAX, gran=O.PER_TENSOR, ln_eps=1e-5)
        check_codes(out["x_q"].cpu().numpy(), ref["codes"], x=as_f32_np(host), G=1)
        check_scalars(out["gamma"].cpu().numpy(), ref["gamma"])


def test_quant_act_per_tensor_status_word_and_workspace_reuse():
    # The per-tensor path keeps its status word in the workspace; reusing one (uninitialised)
    # workspace for calls of different shapes must leave it clear and the results unchanged.
    ws = torch.full((B.workspace_bytes(B.OP_QUANT_ACT, 4096, 1, 4096, 2),), 0xA5, dtype=torch.uint8, device=DEV)
    for M, K, G, dtype in ((4096, 1024, 2, "bf16"), (300, 4096, 1, "f16"), (9, 8192, 1, "bf16"), (33, 1000, 5, "f32")):
        x = synth.make_x(M, K, DT[dtype], seed=M + K, outliers=True).to(DEV)
        a = B.quant_act(x, G=G, gran=B.PER_TENSOR, ws=ws)
        assert B.ws_status(ws) == B.OK
        b = B.quant_act(x, G=G, gran=B.PER_TENSOR)
        assert torch.equal(a["x_q"], b["x_q"]) and torch.equal(a["gamma"], b["gamma"])


def test_quant_act_per_tensor_from_two_streams():
    # The one-kernel per-tensor path is a cooperative launch whose CTAs wait for one another; calls
    # issued from two streams (each with its own workspace) must neither block one another nor mix.
    xs = [synth.make_x(2048, 4096, torch.bfloat16, seed=i, outliers=True).to(DEV) for i in range(2)]
    ref = [B.quant_act(x, gran=B.PER_TENSOR) for x in xs]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(2)]
    wss = [torch.empty(B.workspace_bytes(B.OP_QUANT_ACT, 2048, 1, 4096, 1), dtype=torch.uint8, device=DEV)
           for _ in range(2)]
    outs = [dict(x_q=torch.empty_like(r["x_q"]), gamma=torch.empty_like(r["gamma"]), eta=torch.zeros_like(r["eta"]))
            for r in ref]
    for _ in range(50):
        for i, st in enumerate(streams):
            with torch.cuda.stream(st):
                B.quant_act(xs[i], gran=B.PER_TENSOR, out=outs[i], ws=wss[i])
    torch.cuda.synchronize()
    for i in range(2):
        assert B.ws_status(wss[i]) == B.OK
        assert torch.equal(outs[i]["x_q"], ref[i]["x_q"]) and torch.equal(outs[i]["gamma"], ref[i]["gamma"])


def test_quant_act_ties_and_degenerate_rows():
    # LN skipped, gamma = 128 planted: scale is exactly 1, so the half-to-even ties are exact.
    vals = [0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, -3.5, 126.5, -126.5, 127.5, 128.0, 0.0, 1.0, -1.0, 2.0]
    x = torch.tensor([vals, [0.0] * 16, [3.25] * 16], dtype=torch.float32)
    ref = O.quant_act(x.numpy(), ln_eps=-1.0)
    out = B.quant_act(x.to(DEV), ln_eps=-1.0)
    assert (out["x_q"].cpu().numpy() == ref["codes"]).all()
    assert out["x_q"][0].tolist() == [0, 2, 2, 4, 0, -2, -2, -4, 126, -126, 127, 127, 0, 1, -1, 2]
    # constant rows under LN: gamma = 0, all-zero codes, nothing non-finite
    out = B.quant_act(x.to(DEV), ln_eps=1e-5)
    assert (out["x_q"][1:].cpu().numpy() == 0).all()
    assert out["gamma"][1:].abs().max().item() == 0.0 and torch.isfinite(out["gamma"]).all()
    out = B.quant_act(x.to(DEV), mode=B.ETA, gran=B.PER_TENSOR, ln_eps=-1.0)
    ref = O.quant_act(x.numpy(), mode=O.ETA, gran=O.PER_TENSOR, ln_eps=-1.0)
    check_codes(out["x_q"].cpu().numpy(), ref["codes"])


# ---------------------------------------------------------------- step 4: integer matmul

_HAVE_TC = None


def have_tensor_core_path():
    """The PREFILL (tcgen05) kernel is always compiled in: a valid tiny call must succeed, so that the
    bit-exact GEMM and forward tests can never go green on the CUDA-core kernel alone."""
    global _HAVE_TC
    if _HAVE_TC is None:
        xq = torch.zeros((128, 128), dtype=torch.int8, device=DEV)
        wp = torch.zeros(B.packed_bytes(B.PREFILL, 128, 128), dtype=torch.uint8, device=DEV)
        B.matmul_i32(xq, wp, 128, layout=B.PREFILL)         # raises if the tensor-core path refuses a valid shape
        torch.cuda.synchronize()
        _HAVE_TC = True
    return _HAVE_TC


def gemm_layouts(K, G):
    out = [B.CANONICAL]
    if K % 16 == 0 and (K // G) % 128 == 0 and have_tensor_core_path():
        out.append(B.PREFILL)
    return out


@pytest.mark.parametrize("M,N,K,G", [
    (64, 3072, 768, 1),      # c1
    (1, 16, 8, 1),
    (5, 7, 40, 1),           # nothing aligned
    (70, 130, 1000, 5),      # ragged tiles, K_g = 200
    (200, 300, 1024, 2),     # several tiles with tails, K_g = 512
    (300, 260, 3584, 1),     # K_g of config c5, tails on both sides
    (257, 129, 2048, 4),
])
def test_matmul_i32_bit_exact(M, N, K, G):
    codes = synth.make_codes(M, K, seed=M + N)
    bits = synth.make_bits(N, K, seed=K)
    ref = O.matmul(codes.numpy(), bits.numpy(), G=G)
    for layout in gemm_layouts(K, G):
        if layout == B.CANONICAL:
            packed = bits.to(DEV)
        else:
            from tests.util import from_canonical
            packed = torch.from_numpy(from_canonical(bits.numpy(), layout, N, K)).to(DEV)
        ws = torch.zeros(B.workspace_bytes(B.OP_MATMUL_I32, M, N, K, G), dtype=torch.uint8, device=DEV)
        acc = B.matmul_i32(codes.to(DEV), packed, N, G=G, layout=layout, ws=ws)
        assert B.ws_status(ws) == B.OK
        assert (acc.cpu().numpy() == ref).all(), f"layout {layout}"


def test_matmul_i32_extreme_codes():
    # all codes at +-127 and all weights +1 / -1: the largest accumulators the method allows.
    M, N, K = 130, 140, 4096
    codes = torch.full((M, K), 127, dtype=torch.int8)
    codes[1::2] = -127
    for fill in (0xFF, 0x00):
        bits = torch.full((N, K // 8), fill, dtype=torch.uint8)
        ref = O.matmul(codes.numpy(), bits.numpy())
        for layout in gemm_layouts(K, 1):
            from tests.util import from_canonical
            packed = torch.from_numpy(from_canonical(bits.numpy(), layout, N, K)).to(DEV)
            acc = B.matmul_i32(codes.to(DEV), packed, N, layout=layout)
            assert (acc.cpu().numpy() == ref).all()
    assert abs(int(ref[0, 0, 0])) == 127 * K


# ---------------------------------------------------------------- the layer, Eq. 11

def run_forward_case(M, K, N, G, dtype, ydtype, mode, gran, outliers, relu, seed, layout, eta_correction=False):
    x = synth.make_x(M, K, DT[dtype], seed=seed, outliers=outliers, relu=relu)
    W = synth.make_w(N, K, torch.float32, seed=seed)
    omode = O.ETA if mode == "eta" else O.ABSMAX
    ogran = O.PER_TOKEN if gran == "token" else O.PER_TENSOR
    w_ref = O.binarize(W.numpy(), G=G)
    w_gpu = B.binarize_pack(W.to(DEV), G=G, layout=layout)
    # fp32 output is the parity mode; the 16-bit output must be its RNE rounding
    y32 = B.forward(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, gran=ogran,
                    ln_eps=1e-5, layout=layout, rowsum=w_gpu["rowsum"], eta_correction=eta_correction,
                    out_dtype=torch.float32)
    ref = O.forward(as_f32_np(x), w_ref["bits"], w_ref["beta"], G=G, mode=omode, gran=ogran, ln_eps=1e-5,
                    rowsum=w_ref["rowsum"], eta_correction=eta_correction)
    q = B.quant_act(x.to(DEV), G=G, mode=omode, gran=ogran, ln_eps=1e-5)
    torch.cuda.synchronize()
    y_gpu = y32.cpu().numpy().astype(np.float64)
    rms = np.sqrt((ref["y"] ** 2).mean())
    # (a) end to end, with one quantisation step of slack per flipped code in the token
    diff = check_codes(q["x_q"].cpu().numpy(), ref["codes"], x=as_f32_np(x), G=G,
                       eta_per_token=(mode == "eta" and gran == "token"),
                       eta_per_tensor=(mode == "eta" and gran == "tensor"))
    gam = ref["gamma"] if gran == "token" else np.broadcast_to(ref["gamma"], (M, G))
    step = (w_ref["beta"][None, :] * gam / 128.0).max(axis=1)               # per token
    slack = (np.abs(diff).reshape(M, -1).sum(axis=1) * step)[:, None]
    assert (np.abs(y_gpu - ref["y"]) <= FLOAT_TOL_RMS * rms + slack).all()
    # (b) stage-wise: the oracle's matmul + rescale on the GPU's own codes and scales, no slack
    acc = O.matmul(q["x_q"].cpu().numpy(), w_ref["bits"], G=G)
    y_stage = O.dequant(acc, w_gpu["beta"].cpu().numpy().astype(np.float64),
                        q["gamma"].cpu().numpy().astype(np.float64), gran=ogran,
                        eta=q["eta"].cpu().numpy().astype(np.float64), rowsum=w_ref["rowsum"],
                        eta_correction=eta_correction)
    assert np.abs(y_gpu - y_stage).max() <= FLOAT_TOL_RMS * rms
    if ydtype != "f32":
        y16 = B.forward(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, gran=ogran,
                        ln_eps=1e-5, layout=layout, rowsum=w_gpu["rowsum"], eta_correction=eta_correction,
                        out_dtype=DT[ydtype])
        assert torch.equal(y16, y32.to(DT[ydtype]))
    return y32


FORWARD_CASES = [
    # M, K, N, G, x dtype, y dtype, mode, gran, outliers, relu, seed
    (64, 768, 3072, 1, "f32", "f32", "absmax", "tensor", True, False, 0),     # config c1
    (64, 768, 3072, 1, "f32", "bf16", "absmax", "token", True, False, 0),
    (70, 1000, 130, 5, "bf16", "bf16", "eta", "tensor", False, True, 21),
    (70, 1000, 130, 5, "f16", "f16", "eta", "token", False, True, 22),
    (130, 1024, 200, 2, "bf16", "bf16", "absmax", "token", True, False, 23),
    (9, 3584 * 2, 96, 2, "bf16", "bf16", "eta", "tensor", False, True, 24),   # c5-like groups
]


@pytest.mark.parametrize("M,K,N,G,dtype,ydtype,mode,gran,outliers,relu,seed", FORWARD_CASES)
def test_forward(M, K, N, G, dtype, ydtype, mode, gran, outliers, relu, seed):
    for layout in gemm_layouts(K, G):
        run_forward_case(M, K, N, G, dtype, ydtype, mode, gran, outliers, relu, seed, layout)


def test_matmul_dequant_is_the_second_half_of_forward():
    M, K, N, G = 150, 1024, 264, 2
    x = synth.make_x(M, K, torch.bfloat16, seed=41, outliers=False, relu=True).to(DEV)
    W = synth.make_w(N, K, torch.float32, seed=41).to(DEV)
    for layout in gemm_layouts(K, G):
        w = B.binarize_pack(W, G=G, layout=layout)
        for gran in (B.PER_TENSOR, B.PER_TOKEN):
            for corr in (False, True):
                y = B.forward(x, w["W_packed"], w["beta"], N, G=G, mode=B.ETA, gran=gran, layout=layout,
                              rowsum=w["rowsum"], eta_correction=corr, out_dtype=torch.float32)
                q = B.quant_act(x, G=G, mode=B.ETA, gran=gran)
                y2 = B.matmul_dequant(q["x_q"], q["gamma"], w["W_packed"], w["beta"], N, G=G, gran=gran,
                                      layout=layout, eta=q["eta"], rowsum=w["rowsum"], eta_correction=corr)
                assert torch.equal(y, y2)


def test_forward_eta_correction():
    for layout in gemm_layouts(1024, 2):
        run_forward_case(40, 1024, 72, 2, "bf16", "bf16", "eta", "token", False, True, 31, layout,
                         eta_correction=True)


def test_bounded_wait_that_runs_out_is_reported_and_the_next_call_recovers():
    # The cooperative per-tensor kernel's CTAs meet between its two passes with a bounded wait.  The
    # test hook makes them wait (a few hundred polls) for an arrival tag that nobody publishes: the
    # wait must run out, the kernel must return with BL_ERR_TIMEOUT in the status word and without
    # writing codes, and the next ordinary call on the same workspace must be clean again.
    M, K = 1024, 2048
    x = synth.make_x(M, K, torch.bfloat16, seed=77, outliers=True).to(DEV)
    ws = torch.zeros(B.workspace_bytes(B.OP_QUANT_ACT, M, 1, K, 1), dtype=torch.uint8, device=DEV)
    good = B.quant_act(x, gran=B.PER_TENSOR, ln_eps=1e-5, ws=ws)
    assert B.ws_status(ws) == B.OK
    want = good["x_q"].clone()
    out = dict(x_q=torch.full((M, K), 99, dtype=torch.int8, device=DEV),
               gamma=torch.zeros(1, device=DEV), eta=torch.zeros(1, device=DEV))
    try:
        B.debug_wait_limit(300, meet_skew=True)
        B.quant_act(x, gran=B.PER_TENSOR, ln_eps=1e-5, out=out, ws=ws)
        status = B.ws_status(ws)                       # synchronises: the kernel has returned
    finally:
        B.debug_wait_limit(-1)
    assert status == B.ERR_TIMEOUT
    assert bool((out["x_q"] == 99).all()), "codes were written although the meeting failed"
    again = B.quant_act(x, gran=B.PER_TENSOR, ln_eps=1e-5, out=out, ws=ws)
    assert B.ws_status(ws) == B.OK
    assert torch.equal(again["x_q"], want)


# ---------------------------------------------------------------- decode GEMV

def explained_by_code_flips(err, signs, step, tol, max_flips):
    """True when the output error of one token is, up to `tol`, a sum of at most `max_flips` single
    code changes of +-1: changing code k by one moves output n by W~[n,k] * step[k].  err [N];
    signs [N,K] in {-1,+1}; step [K] (the quantisation step of feature k's group).  The kernel
    quantises x itself, so its codes cannot be read back; they can be inferred this way."""
    r = np.array(err, np.float64)
    for _ in range(max_flips + 1):
        if np.abs(r).max() <= tol:
            return True
        score = (signs * r[:, None]).sum(axis=0) / (signs.shape[0] * step)       # about +-1 at a flipped code
        k = int(np.abs(score).argmax())
        r = r - np.sign(score[k]) * step[k] * signs[:, k]
    return False


@pytest.mark.parametrize("K,N,G,dtype,mode,relu", [
    (4096, 16384, 1, "f16", "absmax", False),      # config c2
    (256, 16, 1, "f32", "absmax", False),
    (1024, 48, 2, "bf16", "eta", True),
    (8192, 2048, 1, "bf16", "absmax", False),      # two K slices per row
    (28672, 112, 8, "bf16", "eta", True),          # c5-shaped K, seven slices
    (2560, 80, 1, "f16", "absmax", False),         # K not a multiple of the slice
    (1024, 40960, 1, "f16", "absmax", False),      # more weight stages than the shared-memory ring holds
    (512, 49152, 2, "bf16", "eta", True),          # the same with groups and row terms
    (32768, 32, 1, "f16", "absmax", False),        # the longest row: one row slot, eight slices
    (4096, 16384, 1, "bf16", "eta", True),         # c2-shaped, eta form (with and without the row terms)
    (12288, 4096, 1, "f16", "absmax", False),      # three slices per row
    (4096, 160000, 1, "f16", "absmax", False),     # 1082 rows per CTA: the ring is refilled many times
    (5120, 1024, 1, "bf16", "absmax", False),      # 13B-shaped width: a whole slice and a quarter of one
    (768, 3072, 1, "f32", "absmax", False),        # 125M-shaped width: a partial slice only
    (7168, 512, 1, "f16", "eta", True),            # 30B-shaped width, eta form
    (16384, 4096, 1, "f16", "absmax", False),      # the last CTA has rows in the first of its two stages only
    (1024, 4000 * 16, 2, "bf16", "eta", True),     # the same in the kernel for groups
])
def test_gemv_decode(K, N, G, dtype, mode, relu):
    x = synth.make_x(1, K, DT[dtype], seed=K + N, outliers=False, relu=relu)
    W = synth.make_w(N, K, torch.float32, seed=K)
    omode = O.ETA if mode == "eta" else O.ABSMAX
    w_ref = O.binarize(W.numpy(), G=G)
    w_gpu = B.binarize_pack(W.to(DEV), G=G, layout=B.DECODE)
    torch.cuda.synchronize()                       # the decode kernel reads the weights ahead of stream order
    signs = None
    for corr in ([False, True] if mode == "eta" else [False]):
        y = B.gemv_decode(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, ln_eps=1e-5,
                          rowsum=w_gpu["rowsum"], eta_correction=corr, out_dtype=torch.float32)
        ref = O.forward(as_f32_np(x), w_ref["bits"], w_ref["beta"], G=G, mode=omode, gran=O.PER_TOKEN,
                        ln_eps=1e-5, rowsum=w_ref["rowsum"], eta_correction=corr)
        torch.cuda.synchronize()
        rms = np.sqrt((ref["y"] ** 2).mean())
        err = y.cpu().numpy().astype(np.float64) - ref["y"][0]
        if np.abs(err).max() <= FLOAT_TOL_RMS * rms:
            continue
        # Not within the plain tolerance: the only accepted reason is that a few codes of the token
        # sit one step away from the oracle's (at most 1e-4 of K, at least one; exact ties of the
        # eta form, where either neighbour is right, on top).  No slack is granted otherwise.
        if signs is None:
            signs = 2.0 * np.unpackbits(w_ref["bits"], axis=1, bitorder="little")[:, :K].astype(np.float64) - 1.0
        step = np.repeat(w_ref["beta"] * ref["gamma"][0] / 128.0, K // G)
        ties = count_exact_ties(as_f32_np(x)[0], G) if mode == "eta" else 0
        assert explained_by_code_flips(err, signs, step, FLOAT_TOL_RMS * rms, max(1, int(CODE_FLIP_FRACTION * K)) + ties), \
            f"decode output differs from the oracle by {np.abs(err).max():.3e} (rms {rms:.3e}) and no few code flips explain it"
    y16 = B.gemv_decode(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, ln_eps=1e-5,
                        out_dtype=DT[dtype])
    y32 = B.gemv_decode(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, G=G, mode=omode, ln_eps=1e-5,
                        out_dtype=torch.float32)
    assert torch.equal(y16, y32.to(DT[dtype]))
    # every stage of weights arrived through its copy: no warp had to fall back to global loads (a
    # stage that is waited for but never copied would still give the right y, a second late per call)
    assert B.debug_decode_fallbacks() == 0


def test_gemv_decode_exact_ties_go_to_the_even_neighbour():
    # Eta form with inputs on a coarse grid: x = j / 64 for integer j in [0, 256], min 0 and max 4,
    # so (x - eta) Q_b / gamma = x * 32 = j / 2 is an exact half-integer for every odd j.  The decode
    # kernel settles such elements in exact arithmetic (Eq. 6 with round-half-to-even), so its
    # codes are known without running anything: rne(j / 2) clipped to 127.  The oracle's matmul and
    # rescale on those codes give y; no code may differ, so the plain tolerance applies.
    K, N = 4096, 256
    rng = np.random.default_rng(3)
    j = rng.integers(0, 257, size=K)
    j[0], j[1] = 0, 256
    x = torch.tensor(j / 64.0, dtype=torch.float16).reshape(1, K)
    assert (x.double().numpy()[0] * 64 == j).all()                      # exactly representable
    half = j // 2
    codes = np.where(j % 2 == 0, half, half + (half % 2)).clip(0, 127).astype(np.int8).reshape(1, K)
    assert np.count_nonzero(j % 2) > K // 3                             # ties everywhere
    W = synth.make_w(N, K, torch.float32, seed=9)
    w_ref = O.binarize(W.numpy())
    w_gpu = B.binarize_pack(W.to(DEV), layout=B.DECODE)
    torch.cuda.synchronize()
    q_ref = O.quant_act(x.float().numpy(), mode=O.ETA, gran=O.PER_TOKEN, ln_eps=1e-5)   # for gamma only
    acc = O.matmul(codes, w_ref["bits"])
    want = O.dequant(acc, w_ref["beta"], q_ref["gamma"], gran=O.PER_TOKEN)[0]
    y = B.gemv_decode(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, mode=B.ETA, ln_eps=1e-5,
                      out_dtype=torch.float32)
    torch.cuda.synchronize()
    rms = np.sqrt((want ** 2).mean())
    assert np.abs(y.cpu().numpy().astype(np.float64) - want).max() <= FLOAT_TOL_RMS * rms


def test_gemv_decode_weights_from_global_memory_when_the_wait_runs_out():
    # With the poll limit of the kernel's one bounded wait at zero every warp takes its wait to have run
    # out and reads its weights from global memory instead: same bits, same y.
    for K, N in [(4096, 16384), (1024, 40960), (8192, 2048)]:
        x = synth.make_x(1, K, torch.float16, seed=K, outliers=False).to(DEV)
        w = B.binarize_pack(synth.make_w(N, K, torch.float32, seed=K + 1).to(DEV), layout=B.DECODE)
        torch.cuda.synchronize()
        want = B.gemv_decode(x, w["W_packed"], w["beta"], N, out_dtype=torch.float32)
        assert B.debug_decode_fallbacks() == 0
        try:
            B.debug_wait_limit(0)
            got = [B.gemv_decode(x, w["W_packed"], w["beta"], N, out_dtype=torch.float32) for _ in range(3)]
        finally:
            B.debug_wait_limit(-1)
        assert B.debug_decode_fallbacks() >= 3 * 8       # every warp of every CTA took the other path
        for g in got:
            assert torch.equal(g, want)


@pytest.mark.parametrize("K,N", [(1024, 64), (4096, 160), (8192, 48)])
def test_gemv_decode_matches_integer_definition_exactly(K, N):
    # With LN skipped and gamma planted at 128 the codes are the inputs themselves, so the
    # output must equal acc * beta exactly as computed by the oracle's integer matmul.
    codes = synth.make_codes(1, K, seed=5)
    codes[0, 0] = 127
    x = codes.float()
    x[0, 1] = 128.0                    # gamma = 128 -> scale 1; this element clips to 127
    W = synth.make_w(N, K, torch.float32, seed=6)
    w_ref = O.binarize(W.numpy())
    w_gpu = B.binarize_pack(W.to(DEV), layout=B.DECODE)
    torch.cuda.synchronize()
    y = B.gemv_decode(x.to(DEV), w_gpu["W_packed"], w_gpu["beta"], N, ln_eps=-1.0, out_dtype=torch.float32)
    c = codes.clone()
    c[0, 1] = 127
    acc = O.matmul(c.numpy(), w_ref["bits"])[0, 0]
    beta32 = w_gpu["beta"].cpu().numpy()[0]
    expect = acc.astype(np.float32) * np.float32(beta32 * np.float32(128.0) * np.float32(1 / 128))
    assert (y.cpu().numpy() == expect).all()


# ---------------------------------------------------------------- argument validation: no launch

def test_invalid_arguments_return_codes():
    x = torch.zeros((4, 64), dtype=torch.float32, device=DEV)
    W = torch.zeros((8, 64), dtype=torch.float32, device=DEV)
    w = B.binarize_pack(W)
    L = B.lib()
    sp = B._stream()
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    p = B._ptr
    y = torch.zeros((4, 8), dtype=torch.float32, device=DEV)
    xq = torch.zeros((4, 64), dtype=torch.int8, device=DEV)
    g = torch.zeros(4, dtype=torch.float32, device=DEV)
    # b != 8
    assert L.bitlinear_quant_act(p(x), B.F32, 4, 64, 1, 4, 0, 1, 1e-5, p(xq), p(g), None, p(ws), ws.numel(), sp) == 4
    # NULL input
    assert L.bitlinear_quant_act(None, B.F32, 4, 64, 1, 8, 0, 1, 1e-5, p(xq), p(g), None, p(ws), ws.numel(), sp) == 1
    # K % (8 G) != 0
    assert L.bitlinear_quant_act(p(x), B.F32, 4, 64, 3, 8, 0, 1, 1e-5, p(xq), p(g), None, p(ws), ws.numel(), sp) == 2
    # workspace too small for the per-tensor path
    assert L.bitlinear_quant_act(p(x), B.F32, 4, 64, 1, 8, 0, 0, 1e-5, p(xq), p(g), None, p(ws), 8, sp) == 5
    # misaligned pointer
    xm = torch.zeros(4 * 64 + 4, dtype=torch.float32, device=DEV)[1:]
    assert L.bitlinear_quant_act(C_void(xm), B.F32, 4, 64, 1, 8, 0, 1, 1e-5, p(xq), p(g), None, p(ws), ws.numel(), sp) == 3
    # eta mode without an eta output
    assert L.bitlinear_quant_act(p(x), B.F32, 4, 64, 1, 8, 1, 1, 1e-5, p(xq), p(g), None, p(ws), ws.numel(), sp) == 1
    # forward: workspace too small, unknown layout
    assert L.bitlinear_forward(p(x), B.F32, 4, 64, 8, 1, 8, 0, 1, 1e-5, 0, p(w["W_packed"]), B.CANONICAL,
                               p(w["beta"]), None, p(y), B.F32, p(ws), 16, sp) == 5
    assert L.bitlinear_forward(p(x), B.F32, 4, 64, 8, 1, 8, 0, 1, 1e-5, 0, p(w["W_packed"]), B.DECODE,
                               p(w["beta"]), None, p(y), B.F32, p(ws), ws.numel(), sp) == 4
    # gemv: K not a multiple of 256
    assert L.bitlinear_gemv_decode(p(x), B.F32, 64, 16, 1, 8, 0, 1e-5, 0, p(w["W_packed"]), p(w["beta"]),
                                   None, p(y), B.F32, sp) == 2
    # outputs untouched by the refused calls
    torch.cuda.synchronize()
    assert y.abs().max().item() == 0 and xq.abs().max().item() == 0


def C_void(t):
    import ctypes
    return ctypes.c_void_p(t.data_ptr())


def test_output_canaries_are_not_overwritten():
    # outputs sit inside larger buffers filled with a sentinel; nothing outside may change
    M, K, N = 37, 520, 45
    x = synth.make_x(M, K, torch.float32, seed=1).to(DEV)
    W = synth.make_w(N, K, torch.float32, seed=1).to(DEV)
    w = B.binarize_pack(W)
    pad = 64
    ybuf = torch.full((M * N + 2 * pad,), 777.0, dtype=torch.float32, device=DEV)
    y = ybuf[pad:pad + M * N].view(M, N)
    B.forward(x, w["W_packed"], w["beta"], N, y=y)
    qbuf = torch.full((M * K + 2 * pad,), 55, dtype=torch.int8, device=DEV)
    xq = qbuf[pad:pad + M * K].view(M, K)
    B.quant_act(x, out=dict(x_q=xq))
    torch.cuda.synchronize()
    assert (ybuf[:pad] == 777.0).all() and (ybuf[-pad:] == 777.0).all()
    assert (qbuf[:pad] == 55).all() and (qbuf[-pad:] == 55).all()
    assert (y != 777.0).any()
