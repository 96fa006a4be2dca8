"""B200-native FP8 in-context-learning attention (per-head absmax e4m3
quantization of Q/K/V plus fused train->train / test->train attention).

``paper_2609_13031_b200.api`` is the Python binding of the C-ABI library
(``include/fp8attn.h``); it loads the CUDA library on first use and raises if
it has not been built.  ``paper_2609_13031_b200.workloads`` draws the seeded
synthetic inputs.  There is no CPU fallback.
"""
__all__ = ["api", "workloads"]
