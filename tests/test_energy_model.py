"""The energy-model calculator against the numbers the paper prints (Table 1) and against the
closed forms of its operation counts (Sec. 2.3)."""
import os

import pytest

from paper_2310_11453_b200 import energy_model as E

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_energy.txt")


def printed_rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        size, wbits, *vals = line.split()
        rows.append((size, int(wbits), [float(v) for v in vals]))
    return rows


def test_table1_matches_the_printed_values():
    model = {(size, wbits): vals for size, wbits, *vals in E.table1()}
    # One printed entry the stated model does not reproduce: BitNet 6.7B, 7 nm ADD is printed
    # as 0.04 J, while INT8 additions of the linear maps (0.0231 J) plus FP16 additions of the
    # attention matmuls (0.0110 J) give 0.034 J; the same sum reproduces the 13B and 30B rows
    # and the 45 nm column of this row.
    known_off = {("6.7B", 1, 1)}
    checked = 0
    for size, wbits, vals in printed_rows():
        got = model[(size, wbits)]
        for col, (want, have) in enumerate(zip(vals, got)):
            tol = 0.0105 if (size, wbits, col) in known_off else 0.0056   # half a printed digit
            assert abs(have - want) <= tol, (size, wbits, col, want, have)
            checked += 1
    assert checked == 36


def test_operation_counts_closed_forms():
    assert E.matmul_ops(3, 5, 7) == E.OpCount(adds=3 * 4 * 7, muls=3 * 5 * 7)
    assert E.bitlinear_ops(3, 5, 7) == E.OpCount(adds=3 * 4 * 7, muls=3 * 7 + 3 * 5)
    # a block's linear maps hold 12 d^2 weights
    d = 64
    assert sum(n * p for n, p in E.block_linear_shapes(d)) == 12 * d * d
    # attention: 2 m^2 d multiplications per block, whatever the number of heads
    for heads in (1, 4, 8):
        assert E.attention_ops(16, d, heads).muls == 2 * 16 * 16 * d


def test_bitnet_saves_energy_at_every_size_and_node():
    for size, (d, layers, heads) in E.MODEL_SHAPES.items():
        for node in ("7nm", "45nm"):
            a1, m1 = E.model_energy(d, layers, heads, 512, 1, node)
            a16, m16 = E.model_energy(d, layers, heads, 512, 16, node)
            assert a1 < a16 and m1 < m16


def test_rejects_other_weight_widths():
    with pytest.raises(ValueError):
        E.model_energy(768, 12, 12, 512, 8, "7nm")
