"""B200-native alternating multi-bit quantization: row quantizer, bit-plane packing, binary
GEMV/GEMM and quantized LSTM/GRU steps, as hand-written CUDA for sm_100a behind a C-ABI library.

`paper_1802_00150_b200.amq` is the Python binding (it loads the CUDA library on import and raises
if the library is missing: there is no CPU fallback).  `paper_1802_00150_b200.synth` holds the seeded
synthetic inputs and imports nothing else.
"""
__all__ = ["amq", "synth"]
