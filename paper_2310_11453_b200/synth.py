"""Seeded synthetic inputs shaped like the paper's 125M-30B models (Appendix A, model table).

This module holds none of the method's arithmetic: it only draws random tensors.  The same
arrays are handed to the CUDA path and to the CPU checker by the tests and the benchmark.
Everything is drawn on the CPU with torch.Generator so that results do not depend on the GPU.
"""
import torch

OUTLIER_PROB = 0.001   # fraction of activation entries scaled up
OUTLIER_SCALE = 20.0
W_STD = 0.02           # "N(0, 0.02)": 0.02 is the standard deviation (GPT-style init)


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def make_x(M: int, K: int, dtype=torch.float32, seed: int = 0, outliers: bool = True,
           relu: bool = False) -> torch.Tensor:
    """Activations ~N(0,1); optionally 0.1 % of entries x20; optionally ReLU'd; cast to dtype."""
    g = _gen(seed)
    x = torch.randn(M, K, generator=g, dtype=torch.float32)
    if outliers:
        mask = torch.rand(M, K, generator=g) < OUTLIER_PROB
        x = torch.where(mask, x * OUTLIER_SCALE, x)
    if relu:
        x = torch.relu(x)
    return x.to(dtype).contiguous()


def make_w(N: int, K: int, dtype=torch.float32, seed: int = 0) -> torch.Tensor:
    """Latent weights ~N(0, 0.02^2), row-major [N, K]."""
    g = _gen(seed + 1_000_003)
    w = torch.randn(N, K, generator=g, dtype=torch.float32) * W_STD
    return w.to(dtype).contiguous()


def make_codes(M: int, K: int, seed: int = 0, lo: int = -127, hi: int = 127) -> torch.Tensor:
    """Uniform int8 codes in [lo, hi] for integer-only matmul checks."""
    g = _gen(seed + 2_000_003)
    return torch.randint(lo, hi + 1, (M, K), generator=g, dtype=torch.int16).to(torch.int8)


def make_bits(N: int, K: int, seed: int = 0) -> torch.Tensor:
    """Uniform random packed sign bits, u8 [N, K/8]."""
    g = _gen(seed + 3_000_003)
    return torch.randint(0, 256, (N, K // 8), generator=g, dtype=torch.int16).to(torch.uint8)


# The benchmark configurations (name -> shapes and flags); sizes follow the model table's
# hidden widths with FFN = 4 x hidden.
CONFIGS = {
    "c1": dict(M=64, K=768, N=3072, G=1, xdtype="f32", ydtype="f32", mode="absmax",
               gran="tensor", seed=0, outliers=True, relu=False),
    "c2": dict(M=1, K=4096, N=16384, G=1, xdtype="f16", ydtype="f16", mode="absmax",
               gran="token", seed=1, outliers=False, relu=False),
    "c3": dict(M=8192, K=4096, N=4096, G=1, xdtype="bf16", ydtype="bf16", mode="absmax",
               gran="tensor", seed=2, outliers=True, relu=False),
    "c5": dict(M=4096, K=28672, N=7168, G=8, xdtype="bf16", ydtype="bf16", mode="eta",
               gran="tensor", seed=4, outliers=False, relu=True),
}

TORCH_DTYPES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}
