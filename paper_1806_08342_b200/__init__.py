"""B200-native integer-only quantized convolution (uniform affine quantization).

``paper_1806_08342_b200.qtz`` is the thin binding over the C-ABI CUDA library;
``paper_1806_08342_b200.synth`` draws the seeded synthetic workloads.  Nothing is
loaded at import time: the CUDA library is opened on first use and its absence
is an error, never a fallback.
"""
__all__ = ["qtz", "synth"]
