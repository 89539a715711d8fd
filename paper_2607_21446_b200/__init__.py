"""KroQuant online activation quantizer for NVIDIA B200 (sm_100a).

``binding`` is the thin Python layer over the C-ABI CUDA library
(``include/kroquant.h``); ``workloads`` draws the seeded synthetic inputs;
``build`` compiles the library in-tree.  Importing this package does not load the
CUDA library; the first call into ``binding`` does, and fails loudly if it is
missing.
"""
__all__ = ["binding", "workloads", "build"]
