"""B200-native fused codistillation objective (loss forward + gradient w.r.t. the logits).

``paper_2010_02838_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/codistill.h``); ``paper_2010_02838_b200.synth`` generates the seeded synthetic
workloads.  Importing the package does not load the CUDA library; the first call into the
binding does, and raises if the library has not been built.
"""
__all__ = ["binding", "synth", "build"]
