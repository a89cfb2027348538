"""B200-native fake-quantization hot path (NVFP4 / MXFP4 / Q4_K quantize-dequantize, the BF16
matmul on fake-quantized operands, and the straight-through backward) behind a C-ABI library.

``paper_2609_39223_b200.api`` is the thin ctypes binding over ``libqf.so``;
``paper_2609_39223_b200.synth`` draws the seeded synthetic workloads.
"""
__all__ = ["api", "replicas", "synth"]
