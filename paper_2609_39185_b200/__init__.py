"""B200-native quantized selective-state-update decode step (fp16 / bf16 / fp8-e4m3 state store with
round-to-nearest, Philox stochastic rounding or the golden-ratio Weyl dither).

``paper_2609_39185_b200.ssdq`` is the thin ctypes binding of the C-ABI CUDA library declared in
``include/ssdq.h``; ``paper_2609_39185_b200.workloads`` generates the seeded synthetic inputs.
The library is loaded on first use and there is no CPU fallback: without the compiled CUDA
extension every call raises.
"""
__all__ = ["workloads"]
