"""Seeded sweep over random shapes, dtypes, modes and group counts: every draw runs one of the parity
cases of the other GPU test files (same oracle, same bars) on a shape nobody picked by hand.
Shapes outside an entry point's documented limits must come back as a status code, never as a
wrong result."""
import random

import pytest

from paper_2310_11453_b200 import binding as B
from tests import test_gpu_decode_batch as TB
from tests import test_gpu_epilogue as TE
from tests import test_gpu_parity as TP

pytestmark = pytest.mark.gpu
DRAWS_PER_SEED = 100


def draw(rng):
    G = rng.choice([1, 1, 1, 2, 3, 4, 8])
    kind = rng.choice(["quant", "quant", "forward", "gemv", "batch", "i32", "pack", "ex"])
    dtype = rng.choice(["f32", "f16", "bf16"])
    mode = rng.choice(["absmax", "eta"])
    gran = rng.choice(["tensor", "token"])
    relu = mode == "eta" and rng.random() < 0.7
    outliers = rng.random() < 0.5
    if kind == "quant":
        Kg = rng.choice([256 * rng.randint(1, 16), 128 * rng.randint(1, 20), 8 * rng.randint(1, 300)])
        M = rng.choice([1, 2, 7, 33, 129, 300, 600, 3553])
        M = max(1, min(M, 2_000_000 // (Kg * G)))
        return lambda: TP.test_quant_act(M, Kg * G, G, dtype, mode, gran, outliers, relu)
    if kind == "forward":
        Kg = rng.choice([128 * rng.randint(1, 12), 8 * rng.randint(1, 100)])
        M, N = rng.choice([1, 7, 64, 129, 257, 300]), rng.choice([1, 8, 17, 130, 256, 300])
        ydt, seed = rng.choice(["f32", "f16", "bf16"]), rng.randint(0, 1000)
        corr = mode == "eta" and rng.random() < 0.5

        def run():
            for layout in TP.gemm_layouts(Kg * G, G):
                TP.run_forward_case(M, Kg * G, N, G, dtype, ydt, mode, gran, outliers, relu, seed, layout,
                                    eta_correction=corr)
        return run
    if kind == "gemv":
        K = 256 * G * rng.randint(1, max(1, 32 // G))
        return lambda: TP.test_gemv_decode(K, 16 * rng.randint(1, 16), G, "f16" if dtype == "f32" else dtype, mode, relu)
    if kind == "batch":
        K = 256 * G * rng.randint(1, max(1, 32 // G))
        return lambda: TB.test_gemv_decode_batch(rng.choice([1, 2, 3, 5, 8, 9, 16]), K, 16 * rng.randint(1, 16), G,
                                                 dtype, mode, relu)
    if kind == "i32":
        Kg = rng.choice([128 * rng.randint(1, 12), 8 * rng.randint(1, 100)])
        M = rng.choice([1, 5, 127, 128, 129, 255, 256, 257, 513, 700])
        N = rng.choice([1, 7, 127, 128, 130, 255, 256, 257, 384, 520])
        return lambda: TP.test_matmul_i32_bit_exact(M, N, Kg * G, G)
    if kind == "pack":
        return lambda: TP.test_binarize_pack_canonical(rng.choice([1, 3, 37, 130, 257, 600]), 8 * G * rng.randint(1, 200),
                                                       G, dtype)
    NB, rows = rng.choice([1, 2, 3]), 32 * rng.randint(1, 8)
    return lambda: TE.test_matmul_dequant_ex(rng.choice([1, 33, 128, 150, 257, 400]), 128 * G * rng.randint(1, 6),
                                             rows * NB, NB, G, rng.choice(["f32", "f16", "bf16"]), mode,
                                             rng.random() < 0.5, rng.random() < 0.5, rng.random() < 0.5)


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_shapes_against_the_oracle(seed):
    rng = random.Random(seed)
    ran = 0
    for _ in range(DRAWS_PER_SEED):
        case = draw(rng)
        try:
            case()
            ran += 1
        except B.BitLinearError as e:
            assert e.code in (B.ERR_SHAPE, B.ERR_UNSUPPORTED), e   # outside the documented limits: refused, not wrong
    assert ran >= DRAWS_PER_SEED // 2


@pytest.mark.parametrize("seed", [21, 22])
def test_random_shapes_decode_batch_with_a_workspace(seed):
    # The tensor-core form (8 or more tokens, one group, K up to 12288) and the hand-over to the other
    # decode kernels around it: token counts on both sides of 8, 16 and 32, chunk counts odd and even,
    # K on both sides of the 32-tokens-per-pass limit, row counts that leave the last CTA short.
    rng = random.Random(seed)
    ran = 0
    for _ in range(30):
        G = rng.choice([1, 1, 1, 1, 2])
        M = rng.choice([2, 7, 8, 9, 15, 16, 17, 24, 31, 32, 33, 40])
        K = 256 * G * rng.randint(1, 48 // G)
        N = 16 * rng.choice([1, 2, 7, 9, 10, 37, 148, 149, 300])
        dtype, mode = rng.choice(["f32", "f16", "bf16"]), rng.choice(["absmax", "eta"])
        try:
            TB.test_gemv_decode_batch_ws(M, K, N, G, dtype, mode, mode == "eta" and rng.random() < 0.7)
            ran += 1
        except B.BitLinearError as e:
            assert e.code in (B.ERR_SHAPE, B.ERR_UNSUPPORTED), e
    assert ran >= 20
