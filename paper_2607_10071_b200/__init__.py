"""B200-native fused Sampling-VT (FlashBEV gather-reduction).

``paper_2607_10071_b200.binding`` is the thin ctypes layer over the C-ABI CUDA
library; ``paper_2607_10071_b200.workloads`` generates seeded synthetic inputs.
Nothing is imported eagerly so that the input generator can be used without the
CUDA library being built.
"""
__all__ = ["binding", "workloads", "build"]
__version__ = "0.1.0"
