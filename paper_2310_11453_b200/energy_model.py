"""Arithmetic-energy estimate of the matrix multiplications of a decoder-only Transformer and of
its BitNet counterpart (Sec. 2.3 "Computational Efficiency", Table 1 from Table 2).

Host-side calculator, no GPU work: it turns model shapes into operation counts and multiplies
them by the per-operation energies of Table 2.

What is counted, per input sequence of m tokens (the paper reports m = 512):
  * the linear maps of every block: Q, K, V, O (d x d each), FFN up (d x 4d) and down (4d x d);
  * the two attention matmuls of every block, per head: scores (m x d_h)(d_h x m) and
    values (m x m)(m x d_h), unmasked.
For an (m x n)(n x p) product the paper's count is m(n-1)p additions and mnp multiplications.
In BitNet the linear maps run on 1-bit weights and 8-bit activations: their additions are INT8
additions and their only multiplications are the output rescale by beta and gamma/Q_b,
mp + mn of them; the attention matmuls stay in FP16.  Embeddings and the output head are not
counted (the printed table does not include them: see the test that pins this module to it).

The precision of the mp + mn rescale multiplications is not stated in the paper; FP16 is used
here, the format of the half-precision comparison (with FP32 two printed digits of Table 1 would
come out one unit higher).
"""
from __future__ import annotations

from dataclasses import dataclass

# Table 2: energy per operation in pJ, (ADD, MUL), by number format and process node.
ENERGY_PJ = {
    ("fp32", "45nm"): (0.9, 3.7), ("fp32", "7nm"): (0.38, 1.31),
    ("fp16", "45nm"): (0.4, 1.1), ("fp16", "7nm"): (0.16, 0.34),
    ("int8", "45nm"): (0.03, 0.2), ("int8", "7nm"): (0.007, 0.07),
}

# Model shapes of the scaling experiments (appendix table of hyper-parameters).
MODEL_SHAPES = {
    "125M": (768, 12, 12), "350M": (1024, 24, 16), "760M": (1536, 24, 16), "1.3B": (2048, 24, 32),
    "2.7B": (2560, 32, 32), "6.7B": (4096, 32, 32), "13B": (5120, 40, 40), "30B": (7168, 48, 56),
}  # name -> (hidden d, layers, heads)


@dataclass(frozen=True)
class OpCount:
    adds: float = 0.0
    muls: float = 0.0

    def __add__(self, other: "OpCount") -> "OpCount":
        return OpCount(self.adds + other.adds, self.muls + other.muls)

    def scaled(self, k: float) -> "OpCount":
        return OpCount(self.adds * k, self.muls * k)


def matmul_ops(m: int, n: int, p: int) -> OpCount:
    """(m x n)(n x p) in a vanilla Transformer: m(n-1)p additions, mnp multiplications."""
    return OpCount(adds=float(m) * (n - 1) * p, muls=float(m) * n * p)


def bitlinear_ops(m: int, n: int, p: int) -> OpCount:
    """The same product in BitLinear: additions only, plus mp + mn rescale multiplications."""
    return OpCount(adds=float(m) * (n - 1) * p, muls=float(m) * p + float(m) * n)


def block_linear_shapes(d: int, ffn_mult: int = 4):
    """(n, p) of the six linear maps of one block."""
    return [(d, d)] * 4 + [(d, ffn_mult * d), (ffn_mult * d, d)]


def attention_ops(m: int, d: int, heads: int) -> OpCount:
    dh = d // heads
    per_head = matmul_ops(m, dh, m) + matmul_ops(m, m, dh)
    return per_head.scaled(heads)


def energy_joule(ops: OpCount, fmt: str, node: str):
    e_add, e_mul = ENERGY_PJ[(fmt, node)]
    return ops.adds * e_add * 1e-12, ops.muls * e_mul * 1e-12


def model_energy(d: int, layers: int, heads: int, seq_len: int, wbits: int, node: str):
    """(E_add, E_mul) in joules for one sequence.  wbits 32 / 16: Transformer in that format;
    wbits 1: BitNet (W1A8 linear maps, FP16 attention)."""
    attn = attention_ops(seq_len, d, heads).scaled(layers)
    if wbits in (32, 16):
        fmt = "fp32" if wbits == 32 else "fp16"
        lin = OpCount()
        for n, p in block_linear_shapes(d):
            lin = lin + matmul_ops(seq_len, n, p)
        return energy_joule(lin.scaled(layers) + attn, fmt, node)
    if wbits != 1:
        raise ValueError("wbits must be 32, 16 or 1")
    lin = OpCount()
    for n, p in block_linear_shapes(d):
        lin = lin + bitlinear_ops(seq_len, n, p)
    lin = lin.scaled(layers)
    add_lin, _ = energy_joule(OpCount(adds=lin.adds), "int8", node)
    _, mul_lin = energy_joule(OpCount(muls=lin.muls), "fp16", node)
    add_attn, mul_attn = energy_joule(attn, "fp16", node)
    return add_lin + add_attn, mul_lin + mul_attn


def table1(seq_len: int = 512, sizes=("6.7B", "13B", "30B")):
    """Rows of Table 1: (size, wbits, 7nm MUL, 7nm ADD, 45nm MUL, 45nm ADD) in joules."""
    rows = []
    for size in sizes:
        d, layers, heads = MODEL_SHAPES[size]
        for wbits in (32, 16, 1):
            a7, m7 = model_energy(d, layers, heads, seq_len, wbits, "7nm")
            a45, m45 = model_energy(d, layers, heads, seq_len, wbits, "45nm")
            rows.append((size, wbits, m7, a7, m45, a45))
    return rows


if __name__ == "__main__":
    print(f"{'size':>5} {'WBits':>5} {'7nm MUL':>9} {'7nm ADD':>9} {'45nm MUL':>9} {'45nm ADD':>9}   (J per 512-token sequence)")
    for size, wbits, m7, a7, m45, a45 in table1():
        print(f"{size:>5} {wbits:>5} {m7:9.3f} {a7:9.3f} {m45:9.3f} {a45:9.3f}")
