"""CPU-only checks of the boundary: the library loads, exports what the header declares, and
its host-side helpers (sizes, layout maps, status strings) behave.  No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2310_11453_b200 import binding as B
from paper_2310_11453_b200 import build as bl_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    bl_build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bitlinear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bitlinear_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 9
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in bitlinear.h but not exported"
    assert sorted(B.EXPORTS) == names


def test_status_strings():
    seen = {B.status_string(c) for c in range(8)}
    assert len(seen) == 8 and B.status_string(0) == "ok"
    assert B.status_string(99) == "unknown status"


def test_packed_and_workspace_sizes():
    assert B.packed_bytes(B.CANONICAL, 3072, 768) == 3072 * 96
    assert B.packed_bytes(B.PREFILL, 4096, 4096) == 4096 * 512
    assert B.packed_bytes(B.PREFILL, 100, 144) == 128 * 256 // 8      # padded to 128 x 256
    assert B.packed_bytes(B.PREFILL, 100, 136) == 0                    # K % 16 != 0
    assert B.packed_bytes(B.DECODE, 16384, 4096) == 16384 * 512
    assert B.packed_bytes(B.DECODE, 16384, 4000) == 0
    assert B.packed_bytes(B.CANONICAL, 4, 12) == 0
    assert B.workspace_bytes(B.OP_BINARIZE_PACK, 1, 8, 64, 1) > 0
    assert B.workspace_bytes(B.OP_FORWARD, 64, 3072, 768, 1) >= 64 * 768
    assert B.workspace_bytes(B.OP_FORWARD, 64, 3072, 768, 5) == 0      # K % (8 G) != 0
    assert B.workspace_bytes(B.OP_QUANT_ACT, 64, 1, 768, 65) == 0      # G too large
    # small-batch decode with a workspace: a status block, then per pass of up to 32 tokens their codes
    # (K bytes per token), gamma and the sum of the codes; enough for passes of 16 as well
    for M, K in [(8, 4096), (16, 4096), (17, 4096), (32, 6144), (33, 8192), (40, 12288)]:
        need = B.workspace_bytes(B.OP_GEMV_DECODE_BATCH, M, 16384, K, 1)
        assert need % 256 == 0
        assert need >= 256 + -(-M // 32) * 32 * (K + 8)
        assert need >= 256 + -(-M // 16) * 16 * (K + 8)
        assert need <= 512 + -(-M // 32) * 32 * (K + 8) + 256
    assert B.workspace_bytes(B.OP_GEMV_DECODE_BATCH, 8, 16384, 4100, 1) == 0     # K % 8 != 0


@pytest.mark.parametrize("layout,N,K", [(B.CANONICAL, 5, 40), (B.PREFILL, 130, 144), (B.PREFILL, 256, 256),
                                        (B.DECODE, 16, 256), (B.DECODE, 32, 512)])
def test_layout_index_is_a_bijection(layout, N, K):
    total = B.packed_bytes(layout, N, K) * 8
    seen = set()
    for n in range(N):
        for k in range(K):
            off, bit = B.layout_index(layout, N, K, n, k)
            assert 0 <= bit < 8 and 0 <= off * 8 + bit < total
            seen.add(off * 8 + bit)
    assert len(seen) == N * K
    with pytest.raises(B.BitLinearError):
        B.layout_index(layout, N, K, N, 0)


def test_canonical_layout_definition():
    assert B.layout_index(B.CANONICAL, 4, 64, 2, 13) == (2 * 8 + 1, 5)


def test_round_trip_helpers():
    from tests.util import from_canonical, to_canonical
    rng = np.random.default_rng(0)
    for layout, N, K in [(B.PREFILL, 130, 272), (B.DECODE, 16, 512)]:
        canon = rng.integers(0, 256, (N, K // 8)).astype(np.uint8)
        packed = from_canonical(canon, layout, N, K)
        assert (to_canonical(packed, layout, N, K) == canon).all()
