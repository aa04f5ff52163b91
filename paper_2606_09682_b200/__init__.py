"""B200-native single-kernel Llama decode step (batch 1), after the AutoMegaKernel paper.

``paper_2606_09682_b200.binding`` is the thin ctypes layer over the C-ABI library (``include/amk.h``);
``paper_2606_09682_b200.inputs`` draws the seeded synthetic workloads.  Importing the package loads
neither CUDA nor the shared library; the binding does, and raises if the library is missing.
"""
__all__ = ["inputs"]
