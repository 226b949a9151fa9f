"""B200-native LOTFormer attention forward (arXiv 2509.23436, Section "Method").

The product is the CUDA library under ``csrc/`` behind the C ABI declared in
``include/lot.h``; ``binding`` marshals torch device tensors into those calls and
does no arithmetic of its own.  ``synth`` draws the seeded benchmark inputs.
Importing the package does not load the library; the first call does, and raises
if it is missing.
"""
__all__ = ["binding", "synth"]
