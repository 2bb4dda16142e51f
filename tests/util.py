"""Helpers shared by the tests (no arithmetic of the method lives here)."""
import numpy as np
import torch

from paper_2310_11453_b200 import binding as B


def to_canonical(packed: np.ndarray, layout: int, N: int, K: int) -> np.ndarray:
    """Map a packed weight buffer of any layout to CANONICAL u8 [N, K/8] through
    bitlinear_layout_index (element by element for small shapes; for large ones the map of one
    128x128 tile / one 32-weight word is computed once and repeated, which is how the layouts are
    defined)."""
    packed = np.ascontiguousarray(packed).reshape(-1)
    if layout == B.CANONICAL:
        return packed[: N * K // 8].reshape(N, K // 8).copy()
    bits = np.zeros((N, K), np.uint8)
    if N * K <= 1 << 16:
        for n in range(N):
            for k in range(K):
                off, bit = B.layout_index(layout, N, K, n, k)
                bits[n, k] = (packed[off] >> bit) & 1
    else:
        pn, pk = (128, 128) if layout == B.PREFILL else (1, 32)
        off0, _ = B.layout_index(layout, N, K, 0, 0)
        rel = np.zeros((pn, pk), np.int64)
        bit = np.zeros((pn, pk), np.int64)
        for i in range(min(pn, N)):
            for j in range(min(pk, K)):
                o, b = B.layout_index(layout, N, K, i, j)
                rel[i, j], bit[i, j] = o - off0, b
        for n0 in range(0, N, pn):
            for k0 in range(0, K, pk):
                base, _ = B.layout_index(layout, N, K, n0, k0)
                h, w = min(pn, N - n0), min(pk, K - k0)
                idx = base + rel[:h, :w]
                bits[n0:n0 + h, k0:k0 + w] = (packed[idx] >> bit[:h, :w]) & 1
    return np.packbits(bits, axis=1, bitorder="little")


def from_canonical(canon: np.ndarray, layout: int, N: int, K: int) -> np.ndarray:
    """Inverse of to_canonical for small shapes: CANONICAL u8 [N,K/8] -> packed buffer."""
    out = np.zeros(B.packed_bytes(layout, N, K), np.uint8)
    bits = np.unpackbits(canon, axis=1, bitorder="little")[:, :K]
    if layout == B.CANONICAL:
        return canon.reshape(-1).copy()
    pn, pk = (128, 128) if layout == B.PREFILL else (1, 32)
    off0, _ = B.layout_index(layout, N, K, 0, 0)
    rel = np.zeros((pn, pk), np.int64)
    bit = np.zeros((pn, pk), np.int64)
    for i in range(min(pn, N)):
        for j in range(min(pk, K)):
            o, b = B.layout_index(layout, N, K, i, j)
            rel[i, j], bit[i, j] = o - off0, b
    for n0 in range(0, N, pn):
        for k0 in range(0, K, pk):
            base, _ = B.layout_index(layout, N, K, n0, k0)
            h, w = min(pn, N - n0), min(pk, K - k0)
            np.bitwise_or.at(out, (base + rel[:h, :w]).reshape(-1),
                             (bits[n0:n0 + h, k0:k0 + w].astype(np.uint8) << bit[:h, :w].astype(np.uint8)).reshape(-1))
    return out


def as_f32_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()
