"""Pins for the CPU oracle: each test fixes a part of it to something other than itself.

Sources of truth used here: the hand-worked examples under tests/golden/ (Eq. 1-7, 11, 12),
closed forms, invariants the equations imply, brute force on tiny shapes written as explicit
Python loops over unpacked operands, and numpy's float64 matmul on a special case.
"""
import json
import math
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_examples.json")))


def unpack_pm1(bits, K):
    """bits u8 [N,K/8] -> +-1 int array [N,K]; bit k%8 of byte k/8, 1 = +1."""
    b = np.unpackbits(bits, axis=1, bitorder="little")[:, :K].astype(np.int64)
    return 2 * b - 1


# ---------------------------------------------------------------- worked examples (golden)

def test_golden_binarize():
    fx = GOLD["binarize_2x8"]
    r = O.binarize(np.array(fx["W"], np.float32))
    assert r["alpha"][0] == fx["alpha"]
    assert r["beta"][0] == fx["beta"]
    assert r["bits"].reshape(-1).tolist() == fx["bytes"]
    assert r["rowsum"].reshape(-1).tolist() == fx["rowsum"]


def test_golden_absmax_ties():
    fx = GOLD["absmax_ties_noLN"]
    r = O.quant_act(np.array([fx["x"]], np.float32), ln_eps=-1.0)
    assert r["gamma"].reshape(-1)[0] == fx["gamma"]
    assert r["codes"][0].tolist() == fx["codes"]


def test_golden_eta():
    fx = GOLD["eta_noLN"]
    r = O.quant_act(np.array([fx["x"]], np.float32), mode=O.ETA, ln_eps=-1.0)
    assert r["eta"].reshape(-1)[0] == fx["eta"]
    assert r["gamma"].reshape(-1)[0] == fx["gamma"]
    assert r["codes"][0].tolist() == fx["codes"]


def test_golden_ln_absmax():
    fx = GOLD["ln_absmax_1to8"]
    r = O.quant_act(np.array([fx["x"]], np.float32), ln_eps=fx["ln_eps"])
    assert abs(r["gamma"].reshape(-1)[0] - fx["gamma"]) < 1e-14
    assert r["codes"][0].tolist() == fx["codes"]


def test_golden_forward():
    fb, fl, ff = GOLD["binarize_2x8"], GOLD["ln_absmax_1to8"], GOLD["forward_2x8"]
    w = O.binarize(np.array(fb["W"], np.float32))
    r = O.forward(np.array([fl["x"]], np.float32), w["bits"], w["beta"], ln_eps=0.0)
    assert r["acc"].reshape(-1).tolist() == ff["acc"]
    np.testing.assert_allclose(r["y"].reshape(-1), ff["y"], rtol=1e-14)


# ---------------------------------------------------------------- binarization (Eq. 1-3, 12, 13)

def test_sign_tie_is_minus_one():
    # symmetric integer-valued W: alpha = 0 exactly; zeros must binarize to -1 (bit 0).
    W = np.array([[-2, -1, 0, 0, 1, 2, 0, 0], [3, 0, -3, 0, 0, 0, 1, -1]], np.float32)
    r = O.binarize(W)
    assert r["alpha"][0] == 0.0
    expect = np.where(W > 0, 1, -1)
    assert (unpack_pm1(r["bits"], 8) == expect).all()


def test_alpha_beta_closed_forms():
    # arithmetic progression 1..N*K: alpha = (NK+1)/2, beta the same (all positive).
    N, K = 4, 16
    W = np.arange(1, N * K + 1, dtype=np.float32).reshape(N, K)
    r = O.binarize(W)
    assert r["alpha"][0] == (N * K + 1) / 2
    assert r["beta"][0] == (N * K + 1) / 2
    # +-c checkerboard: alpha = 0, beta = c, signs follow the pattern.
    c = 0.375
    P = np.where((np.add.outer(np.arange(N), np.arange(K)) % 2) == 0, c, -c).astype(np.float32)
    r = O.binarize(P)
    assert r["alpha"][0] == 0.0 and r["beta"][0] == c
    assert (unpack_pm1(r["bits"], K) == np.sign(P)).all()
    assert (r["rowsum"] == 0).all()


def test_gaussian_closed_form_and_zero_centre():
    rng = np.random.default_rng(5)
    N, K, sigma = 512, 1024, 0.02
    W = (rng.standard_normal((N, K)) * sigma).astype(np.float32)
    r = O.binarize(W)
    nk = N * K
    assert abs(r["beta"][0] - sigma * math.sqrt(2 / math.pi)) < 4 / math.sqrt(nk) * sigma
    assert abs(r["alpha"][0]) < 5 * sigma / math.sqrt(nk)
    pm = unpack_pm1(r["bits"], K)
    assert abs(pm.sum()) <= 6 * math.sqrt(nk)                       # zero-centred
    assert (pm.sum(axis=1) == r["rowsum"][:, 0]).all()
    # beta * ||W~||_1 = ||W||_1
    l1 = np.abs(W.astype(np.float64)).sum()
    assert abs(r["beta"][0] * np.abs(pm).sum() - l1) <= 1e-12 * l1
    # mean against numpy's pairwise float64 mean
    assert abs(r["alpha"][0] - W.astype(np.float64).mean()) < 1e-15


def test_alpha_is_subtracted_not_added():
    # all weights positive, so Sign(W) would be all +1; Sign(W - alpha) splits around the mean.
    W = np.array([[1, 2, 3, 4, 5, 6, 7, 8]], np.float32)
    r = O.binarize(W)
    assert unpack_pm1(r["bits"], 8).reshape(-1).tolist() == [-1, -1, -1, -1, 1, 1, 1, 1]


def test_group_binarize_matches_slices():
    rng = np.random.default_rng(6)
    N, K, G = 8, 64, 4
    W = (rng.standard_normal((N, K)) * 0.02 + np.repeat(np.arange(G) * 0.01, K // G)).astype(np.float32)
    r = O.binarize(W, G=G)
    Kg = K // G
    for g in range(G):
        s = O.binarize(W[:, g * Kg:(g + 1) * Kg])
        assert s["alpha"][0] == r["alpha"][g] and s["beta"][0] == r["beta"][g]
        assert (s["bits"] == r["bits"][:, g * Kg // 8:(g + 1) * Kg // 8]).all()
        assert (s["rowsum"][:, 0] == r["rowsum"][:, g]).all()
    # group means really differ, so a whole-tensor alpha would give other bits
    assert not (O.binarize(W)["bits"] == r["bits"]).all()


def test_alpha_override():
    W = np.array([[1, 2, 3, 4, 5, 6, 7, 8]], np.float32)
    r = O.binarize(W, alpha_in=[6.5])
    assert unpack_pm1(r["bits"], 8).reshape(-1).tolist() == [-1] * 6 + [1, 1]
    assert r["beta"][0] == 4.5


# ---------------------------------------------------------------- LN (Eq. 12, 15)

def test_ln_moments_and_constant_row():
    rng = np.random.default_rng(7)
    M, K, eps = 5, 256, 1e-5
    x = (rng.standard_normal((M, K)) * 3 + 1.5).astype(np.float32)
    x[4] = 2.75                                                   # constant row
    r = O.quant_act(x, ln_eps=eps, want_xhat=True)
    xh = r["xhat"]
    assert np.abs(xh.mean(axis=1)).max() < 1e-12
    var = x.astype(np.float64).var(axis=1)
    np.testing.assert_allclose(xh.var(axis=1)[:4], (var / (var + eps))[:4], rtol=1e-12)
    assert (xh[4] == 0).all() and (r["codes"][4] == 0).all() and r["gamma"][4, 0] == 0.0
    assert np.isfinite(xh).all()


def test_ln_group_norm():
    rng = np.random.default_rng(8)
    M, K, G = 3, 128, 4
    x = rng.standard_normal((M, K)).astype(np.float32) * np.repeat([1, 5, 0.2, 9], K // G).astype(np.float32)
    r = O.quant_act(x, G=G, ln_eps=1e-5, want_xhat=True)
    Kg = K // G
    for g in range(G):
        s = O.quant_act(np.ascontiguousarray(x[:, g * Kg:(g + 1) * Kg]), ln_eps=1e-5, want_xhat=True)
        assert (s["xhat"] == r["xhat"][:, g * Kg:(g + 1) * Kg]).all()
        assert (s["codes"] == r["codes"][:, g * Kg:(g + 1) * Kg]).all()
        assert (s["gamma"][:, 0] == r["gamma"][:, g]).all()


# ---------------------------------------------------------------- Quant (Eq. 4-6, 14)

@pytest.mark.parametrize("gran", [O.PER_TOKEN, O.PER_TENSOR])
def test_code_bounds_saturation_and_rounding_bound(gran):
    rng = np.random.default_rng(9)
    M, K = 16, 512
    x = rng.standard_normal((M, K)).astype(np.float32)
    x[rng.random((M, K)) < 0.002] *= 20
    r = O.quant_act(x, gran=gran, ln_eps=1e-5, want_xhat=True)
    codes, xh = r["codes"].astype(np.int64), r["xhat"]
    assert np.abs(codes).max() == 127                              # |code| <= Q_b - 1, reached
    gam = r["gamma"][:, 0][:, None] if gran == O.PER_TOKEN else r["gamma"][0]
    if gran == O.PER_TOKEN:
        i = np.abs(xh).argmax(axis=1)
        assert (np.abs(codes[np.arange(M), i]) == 127).all()       # the arg-max saturates
        np.testing.assert_allclose(r["gamma"][:, 0], np.abs(xh).max(axis=1), rtol=0, atol=0)
    else:
        assert r["gamma"][0] == np.abs(xh).max()
    gam = np.broadcast_to(gam, xh.shape)
    err = np.abs(codes * gam / 128 - xh)
    unsat = np.abs(xh * 128 / gam) <= 127.5
    assert (err[unsat] <= gam[unsat] / 256 * (1 + 1e-12)).all()
    assert (err <= gam / 128 * (1 + 1e-12)).all()
    # sign of codes follows sign of xhat
    assert (np.sign(codes) * np.sign(xh) >= 0).all()


def test_eta_mode_range_and_endpoints():
    rng = np.random.default_rng(10)
    M, K = 8, 256
    x = np.maximum(rng.standard_normal((M, K)), 0).astype(np.float32)
    r = O.quant_act(x, mode=O.ETA, ln_eps=1e-5, want_xhat=True)
    codes, xh = r["codes"], r["xhat"]
    assert codes.min() == 0 and codes.max() == 127
    rows = np.arange(M)
    assert (codes[rows, xh.argmin(axis=1)] == 0).all()
    assert (codes[rows, xh.argmax(axis=1)] == 127).all()
    np.testing.assert_array_equal(r["eta"][:, 0], xh.min(axis=1))
    np.testing.assert_array_equal(r["gamma"][:, 0], xh.max(axis=1) - xh.min(axis=1))
    recon = codes * (r["gamma"][:, :1] / 128) + r["eta"][:, :1]
    assert (np.abs(recon - xh) <= r["gamma"][:, :1] / 128 * (1 + 1e-12)).all()


def test_half_to_even_ties_exact():
    # gamma = 128 planted, LN skipped -> scale exactly 1.
    vals = [0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5, -3.5, 126.5, -126.5, 127.5, 128.0, 0.0, 1.0, -1.0, 2.0]
    x = np.array([vals], np.float32)
    r = O.quant_act(x, ln_eps=-1.0)
    assert r["codes"][0].tolist() == [0, 2, 2, 4, 0, -2, -2, -4, 126, -126, 127, 127, 0, 1, -1, 2]


def test_per_tensor_gamma_is_global():
    x = np.zeros((2, 8), np.float32)
    x[0, 0], x[1, 3] = 4.0, -64.0
    r = O.quant_act(x, gran=O.PER_TENSOR, ln_eps=-1.0)
    assert r["gamma"].tolist() == [64.0]
    assert r["codes"][0, 0] == 8 and r["codes"][1, 3] == -127
    rt = O.quant_act(x, gran=O.PER_TOKEN, ln_eps=-1.0)
    assert rt["gamma"][:, 0].tolist() == [4.0, 64.0] and rt["codes"][0, 0] == 127


def test_per_tensor_eta_over_several_rows_hand_worked():
    # Eq. 6 / 14 per tensor, LN skipped, two groups of eight features over three tokens.  By hand:
    # group 0: eta = 0 (the minimum over ALL rows, found in row 1), gamma = 10 - 0 (the maximum is in
    # row 1 too), codes = rne(12.8 x); group 1: eta = -3, gamma = 5 - (-3) = 8, codes = rne(16 (x + 3)).
    # The maximum of each group reaches 128 and is clipped to 127.  gamma is the range max - min, not
    # max |x| (which would be 10 and 5).
    x = np.array([[1, 2, 3, 4, 0.5, 1.5, 2, 2, -3, -1, 1, 5, 0, 0, 0, 0],
                  [0, 5, 6, 10, 1, 1, 1, 1, 5, 5, 5, 5, 5, 5, 5, 5],
                  [7, 8, 9, 2.5, 3, 3, 3, 3, -3, 0, 2, 3, 1, 1, 1, 1]], np.float32)
    r = O.quant_act(x, G=2, mode=O.ETA, gran=O.PER_TENSOR, ln_eps=-1.0)
    assert r["eta"].tolist() == [0.0, -3.0]
    assert r["gamma"].tolist() == [10.0, 8.0]
    assert r["codes"].tolist() == [
        [13, 26, 38, 51, 6, 19, 26, 26, 0, 32, 64, 127, 48, 48, 48, 48],
        [0, 64, 77, 127, 13, 13, 13, 13, 127, 127, 127, 127, 127, 127, 127, 127],
        [90, 102, 115, 32, 38, 38, 38, 38, 0, 48, 80, 96, 64, 64, 64, 64]]
    # per token the same input has its own eta and gamma per row and group
    rt = O.quant_act(x, G=2, mode=O.ETA, gran=O.PER_TOKEN, ln_eps=-1.0)
    assert rt["eta"].tolist() == [[0.5, -3.0], [0.0, 5.0], [2.5, -3.0]]
    assert rt["gamma"].tolist() == [[3.5, 8.0], [10.0, 0.0], [6.5, 6.0]]
    assert rt["codes"][1, 8:].tolist() == [0] * 8                 # a constant segment: gamma = 0, codes 0


def test_zero_input_gives_zero_codes():
    r = O.quant_act(np.zeros((2, 16), np.float32), ln_eps=1e-5)
    assert (r["codes"] == 0).all() and (r["gamma"] == 0).all()
    r = O.quant_act(np.zeros((2, 16), np.float32), mode=O.ETA, ln_eps=-1.0)
    assert (r["codes"] == 0).all()


# ---------------------------------------------------------------- matmul (Eq. 7)

@pytest.mark.parametrize("M,N,K,G", [(1, 1, 8, 1), (3, 5, 16, 1), (4, 8, 64, 1), (2, 3, 64, 4)])
def test_matmul_brute_force(M, N, K, G):
    rng = np.random.default_rng(100 + K + G)
    codes = rng.integers(-127, 128, (M, K)).astype(np.int8)
    bits = rng.integers(0, 256, (N, K // 8)).astype(np.uint8)
    acc = O.matmul(codes, bits, G=G)
    Kg = K // G
    for g in range(G):
        for m in range(M):
            for n in range(N):
                s = 0
                for k in range(g * Kg, (g + 1) * Kg):
                    bit = (int(bits[n, k // 8]) >> (k % 8)) & 1
                    s += (1 if bit else -1) * int(codes[m, k])
                assert acc[g, m, n] == s


def test_matmul_all_plus_all_minus_and_one_hot():
    rng = np.random.default_rng(11)
    M, N, K = 4, 6, 64
    codes = rng.integers(-127, 128, (M, K)).astype(np.int8)
    plus = np.full((N, K // 8), 0xFF, np.uint8)
    assert (O.matmul(codes, plus)[0] == codes.astype(np.int64).sum(axis=1)[:, None]).all()
    assert (O.matmul(codes, np.zeros_like(plus))[0] == -codes.astype(np.int64).sum(axis=1)[:, None]).all()
    # one-hot code rows read back W~[n,k]*127 for every k: pins bit order and K-major packing.
    bits = rng.integers(0, 256, (N, K // 8)).astype(np.uint8)
    onehot = (np.eye(K) * 127).astype(np.int8)
    acc = O.matmul(onehot, bits)[0]                                 # [K, N]
    assert (acc.T == 127 * unpack_pm1(bits, K)).all()


def test_matmul_against_float64_gemm_and_samples():
    rng = np.random.default_rng(12)
    M, N, K, G = 33, 70, 256, 2
    codes = rng.integers(-127, 128, (M, K)).astype(np.int8)
    bits = rng.integers(0, 256, (N, K // 8)).astype(np.uint8)
    acc = O.matmul(codes, bits, G=G)
    pm = unpack_pm1(bits, K).astype(np.float64)
    Kg = K // G
    for g in range(G):
        ref = codes[:, g * Kg:(g + 1) * Kg].astype(np.float64) @ pm[:, g * Kg:(g + 1) * Kg].T
        assert (acc[g] == ref).all()
    ms = rng.integers(0, M, 50)
    ns = rng.integers(0, N, 50)
    s = O.matmul_samples(codes, bits, ms, ns, G=G)
    for g in range(G):
        assert (s[:, g] == acc[g, ms, ns]).all()


def test_matmul_is_not_transposed():
    # M != N and an asymmetric pattern: swapping operands or indices cannot pass.
    codes = np.zeros((2, 8), np.int8)
    codes[0, 0], codes[1, 7] = 5, 9
    bits = np.zeros((3, 1), np.uint8)
    bits[1, 0] = 0x01      # row 1: +1 at k = 0
    bits[2, 0] = 0x80      # row 2: +1 at k = 7
    acc = O.matmul(codes, bits)[0]
    assert acc.shape == (2, 3)
    assert acc.tolist() == [[-5, 5, -5], [-9, -9, 9]]


# ---------------------------------------------------------------- dequant / forward (Eq. 11)

def test_forward_equals_staged_and_linearity_bound():
    rng = np.random.default_rng(13)
    M, N, K = 16, 48, 1024
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w = O.binarize(W)
    f = O.forward(x, w["bits"], w["beta"], ln_eps=1e-5)
    q = O.quant_act(x, ln_eps=1e-5, want_xhat=True)
    acc = O.matmul(q["codes"], w["bits"])
    y = O.dequant(acc, w["beta"], q["gamma"])
    assert (f["y"] == y).all() and (f["codes"] == q["codes"]).all()
    # Eq. 11 written out with numpy on the oracle's own integer results
    y_np = acc[0].astype(np.float64) * w["beta"][0] * q["gamma"] / 128.0
    np.testing.assert_allclose(y, y_np, rtol=1e-14)
    # y approximates beta * W~ xhat with uniform-quantisation-noise error
    pm = unpack_pm1(w["bits"], K).astype(np.float64)
    exact = w["beta"][0] * q["xhat"] @ pm.T
    rms_err = np.sqrt(((y - exact) ** 2).mean())
    bound = (q["gamma"].max() / (128 * math.sqrt(12))) * w["beta"][0] * math.sqrt(K) * 1.2
    assert rms_err <= bound
    assert rms_err >= 0.5 * (q["gamma"].min() / (128 * math.sqrt(12))) * w["beta"][0] * math.sqrt(K)


def test_variance_argument():
    # Eq. 8-10: Var(y) ~ K * beta^2 * E[xhat_q^2]; with LN that is ~ K beta^2.
    rng = np.random.default_rng(14)
    M, N, K = 32, 256, 4096
    x = rng.standard_normal((M, K)).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w = O.binarize(W)
    f = O.forward(x, w["bits"], w["beta"], ln_eps=1e-5)
    rms = np.sqrt((f["y"] ** 2).mean())
    assert abs(rms / (w["beta"][0] * math.sqrt(K)) - 1.0) < 0.05


def test_group_forward_is_sum_of_slices():
    rng = np.random.default_rng(15)
    M, N, K, G = 6, 10, 256, 4
    x = np.maximum(rng.standard_normal((M, K)), 0).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    Kg = K // G
    for mode in (O.ABSMAX, O.ETA):
        for gran in (O.PER_TOKEN, O.PER_TENSOR):
            w = O.binarize(W, G=G)
            f = O.forward(x, w["bits"], w["beta"], G=G, mode=mode, gran=gran, ln_eps=1e-5)
            total = np.zeros((M, N))
            for g in range(G):
                ws = O.binarize(W[:, g * Kg:(g + 1) * Kg])
                fs = O.forward(np.ascontiguousarray(x[:, g * Kg:(g + 1) * Kg]), ws["bits"], ws["beta"],
                               mode=mode, gran=gran, ln_eps=1e-5)
                assert (fs["acc"][0] == f["acc"][g]).all()
                total += fs["y"]
            np.testing.assert_allclose(f["y"], total, rtol=1e-13, atol=1e-15)
    # G = 1 is the ungrouped layer
    w1 = O.binarize(W, G=1)
    assert (O.forward(x, w1["bits"], w1["beta"], G=1)["y"] == O.forward(x, w1["bits"], w1["beta"])["y"]).all()


def test_eta_correction_restores_unshifted_product():
    rng = np.random.default_rng(16)
    M, N, K = 4, 12, 512
    x = np.maximum(rng.standard_normal((M, K)), 0).astype(np.float32)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    w = O.binarize(W)
    lit = O.forward(x, w["bits"], w["beta"], mode=O.ETA, ln_eps=1e-5)
    cor = O.forward(x, w["bits"], w["beta"], mode=O.ETA, ln_eps=1e-5, rowsum=w["rowsum"], eta_correction=True)
    diff = cor["y"] - lit["y"]
    expect = lit["eta"][:, :1] * w["beta"][0] * w["rowsum"][:, 0][None, :]
    np.testing.assert_allclose(diff, expect, rtol=1e-12, atol=1e-15)
    q = O.quant_act(x, mode=O.ETA, ln_eps=1e-5, want_xhat=True)
    exact = w["beta"][0] * q["xhat"] @ unpack_pm1(w["bits"], K).astype(np.float64).T
    assert np.sqrt(((cor["y"] - exact) ** 2).mean()) < 0.02 * np.sqrt((exact ** 2).mean())


def test_dequant_scale_is_qb_128_not_127():
    acc = np.array([[[128]]], np.int32)
    y = O.dequant(acc, [0.5], [[2.0]])
    assert y[0, 0] == 128 * 0.5 * 2.0 / 128


def test_bad_shapes_are_rejected():
    with pytest.raises(ValueError):
        O.binarize(np.zeros((2, 12), np.float32))            # K % 8 != 0
    with pytest.raises(ValueError):
        O.quant_act(np.zeros((2, 16), np.float32), G=4)      # K % (8 G) != 0


# ---------------------------------------------------------------- attention core of the block (Sec. 2)

def _attn_inputs(B, S, H, D, seed):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((B * S, H * D)).astype(np.float32) for _ in range(3)]


def test_attention_matches_library_routine():
    # special case that reduces to a library routine: torch's CPU scaled_dot_product_attention in fp64
    import torch
    B, S, H, D = 2, 80, 3, 16
    q, k, v = _attn_inputs(B, S, H, D, 0)
    out = O.attention_rows(q, k, v, B, S, H, D, np.arange(B * S))

    def heads_first(a):
        return torch.from_numpy(a).double().view(B, S, H, D).permute(0, 2, 1, 3)

    ref = torch.nn.functional.scaled_dot_product_attention(heads_first(q), heads_first(k), heads_first(v), is_causal=True)
    ref = ref.permute(0, 2, 1, 3).reshape(B * S, H * D).numpy()
    assert np.abs(out - ref).max() < 1e-12


def test_attention_closed_forms():
    B, S, H, D = 2, 33, 2, 8
    q, k, v = _attn_inputs(B, S, H, D, 1)
    rows = np.arange(B * S)
    out = O.attention_rows(q, k, v, B, S, H, D, rows)
    # the first token of every sequence attends only itself
    assert np.array_equal(out[0], v[0].astype(np.float64)) and np.array_equal(out[S], v[S].astype(np.float64))
    # zero queries give uniform weights: the running mean of v over the causal prefix
    out0 = O.attention_rows(np.zeros_like(q), k, v, B, S, H, D, rows)
    for b in range(B):
        prefix_mean = np.cumsum(v[b * S:(b + 1) * S].astype(np.float64), axis=0) / np.arange(1, S + 1)[:, None]
        assert np.abs(out0[b * S:(b + 1) * S] - prefix_mean).max() < 1e-12
    # outputs are convex combinations of the value rows seen so far, head by head
    for t in (5, S + 7):
        b, tt = divmod(t, S)
        for h in range(H):
            vs = v[b * S:b * S + tt + 1, h * D:(h + 1) * D]
            assert (out[t, h * D:(h + 1) * D] <= vs.max(axis=0) + 1e-12).all()
            assert (out[t, h * D:(h + 1) * D] >= vs.min(axis=0) - 1e-12).all()
    # a future token never matters: changing k, v after position t leaves row t unchanged
    k2, v2 = k.copy(), v.copy()
    k2[20:S] += 3.0
    v2[20:S] -= 2.0
    out2 = O.attention_rows(q, k2, v2, B, S, H, D, np.arange(0, 20))
    assert np.array_equal(out2, out[:20])
    # a sharp query picks one key: q = c * k_s with large c selects v_s (s <= t)
    q3 = np.zeros_like(q)
    q3[10, :D] = 200.0 * k[4, :D] / (np.linalg.norm(k[4, :D]) ** 2) * np.sqrt(D) * 40
    o3 = O.attention_rows(q3, k, v, B, S, H, D, np.array([10]))
    scores = (q3[10, :D].astype(np.float64) @ k[:11, :D].astype(np.float64).T) / np.sqrt(D)
    assert np.abs(o3[0, :D] - v[int(np.argmax(scores)), :D]).max() < 1e-6


# ---------------------------------------------------------------- N-split groups (Eq. 13 along N)

def test_binarize_nsplit_blocks_have_their_own_alpha_and_beta():
    rng = np.random.default_rng(7)
    N, K, NB, G = 24, 64, 3, 2
    # blocks with clearly different means and spreads
    W = np.concatenate([rng.normal(m, s, size=(N // NB, K)) for m, s in ((0.5, 0.1), (-0.2, 1.0), (0.0, 0.01))])
    W = W.astype(np.float32)
    r = O.binarize_nsplit(W, NB, G=G)
    rows, Kg = N // NB, K // G
    for j in range(NB):
        for g in range(G):
            blk = W[j * rows:(j + 1) * rows, g * Kg:(g + 1) * Kg].astype(np.float64)
            assert abs(r["alpha"][j, g] - blk.mean()) < 1e-12
            assert abs(r["beta"][j, g] - np.abs(blk).mean()) < 1e-12
            want = (blk > blk.mean())
            got = np.unpackbits(r["bits"][j * rows:(j + 1) * rows], axis=1, bitorder="little")[:, g * Kg:(g + 1) * Kg]
            assert np.array_equal(got.astype(bool), want)
    # one block is the plain per-matrix binarisation
    one = O.binarize_nsplit(W, 1, G=G)
    ref = O.binarize(W, G=G)
    assert np.array_equal(one["bits"], ref["bits"]) and np.array_equal(one["alpha"][0], ref["alpha"])


def test_dequant_nsplit_scales_each_block_by_its_beta():
    rng = np.random.default_rng(8)
    G, M, N, NB = 2, 5, 12, 3
    acc = rng.integers(-1000, 1000, size=(G, M, N)).astype(np.int32)
    beta = rng.uniform(0.1, 2.0, size=(NB, G))
    gamma = rng.uniform(1.0, 5.0, size=(M, G))
    y = O.dequant_nsplit(acc, beta, gamma, gran=O.PER_TOKEN)
    want = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            want[m, n] = sum(acc[g, m, n] * beta[n // (N // NB), g] * gamma[m, g] / 128.0 for g in range(G))
    assert np.allclose(y, want, rtol=1e-13, atol=0)
