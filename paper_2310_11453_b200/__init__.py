"""B200-native BitLinear forward (BitNet, Sec. 2.1): thin Python binding over the C-ABI library.

The CUDA shared library is loaded on first use by `paper_2310_11453_b200.binding`; there is no
CPU fallback.  `paper_2310_11453_b200.synth` only draws seeded inputs and needs no GPU.
"""
__all__ = ["binding", "synth"]
